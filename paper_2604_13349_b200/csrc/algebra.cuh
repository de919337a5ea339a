// Per-head dense algebra of Orthogonal BackFill (Eq. 2-6), one thread block per
// (cache, layer, KV head), everything in fp32 in shared memory.
//
// Inputs (from the streaming pass): Gram of the deleted values G_del, Gram of the
// retained values G_keep (only when k_eff >= d), u = sum_del A_j v_j, the demand
// sums, and the retained rows themselves (read back from v_out).  The tuned streaming
// pass delivers G and u over ALL rows instead (it runs before the selection is known):
// P G_all P = P G_del P because P annihilates the retained rows; the retained rows'
// share of u and of the trace of G is subtracted here, while they are read for the basis.
//
//   1. k_eff >= d: k_span_test has factorised G_keep (Cholesky).  If every pivot
//      stayed above 1e-3 of its diagonal entry the retained values span R^d, the
//      residual of Eq. 3 is identically zero and delta = 0.
//   2. Otherwise: orthonormal basis Q of span(V_keep) (Eq. 2) by Gram-Schmidt over
//      the retained rows, iterated a second time for a row that lost more than half
//      of its squared norm in the first pass; a row adds a direction when what is
//      left of it exceeds 1e-4 of its own norm.
//   3. M = P G P = R^T R with P = I - Q^T Q (Eq. 3 in Gram form, App. H), formed without P as two rank-m
//      updates with the m basis rows in Q: X <- X - Q^T (Q X) from the left, then the same from the right
//      (8 m d^2 flops instead of the 4 d^3 of two full products),
//      r_bar = P u / (A_del + eps) = (u - Q^T (Q u)) / (A_del + eps)  (Eq. 4).
//   4. C = eigenvectors of the `rank` largest eigenvalues of M above 1e-5 of the
//      largest.  For rank <= ALG_TRI_MAX_RANK: Householder reduction of M to
//      tridiagonal form (two block barriers per column), the rank + 1 largest
//      eigenvalues by 33-way multisection on Sturm counts, their vectors by inverse
//      iteration (neighbours closer than 1e-3 of the largest eigenvalue are kept
//      orthogonal during the iteration), mapped back through the reflectors two at a
//      time.  For larger ranks: full eigen-decomposition by
//      parallel-order Jacobi rotations run to convergence.
//   5. Delta = C^T C r_bar (Eq. 5), delta = A_del / (A_keep + eps) * Delta (Eq. 6), projected once more off the
//      basis rows (the subtractions that form M leave rounding noise of the size of G's largest entries),
//      V_out = V_keep + delta on the head's retained rows (Eq. 7).
//
// Shared memory: M (d x d) plus a region sized by the number of basis rows any head of the call can have
// (min(k_eff, d)): with budgets below d two blocks share a multiprocessor, which is what the latency-bound
// steps of the eigen-solver need.  That caps the kernel at 64 registers per thread: the loops below are written
// for few live values and few instructions (thread maps that keep a warp's 32 lanes on 32 banks of the
// 129-float rows, whole rows and column groups skipped rather than predicated off), which is what its time is
// made of.
#pragma once

#include "common.cuh"
#include "span_test.cuh"

namespace obf {

constexpr int ALG_NT = 512;
constexpr float SPAN_ROW_TOL = 1e-4f;
constexpr float RCR_SKIP_TOL = 1e-6f;
constexpr float EIG_RANK_TOL = 1e-5f;
constexpr int JACOBI_MAX_SWEEPS = 30;
constexpr int ALG_TRI_MAX_RANK = 8;     // up to this rank only rank + 1 eigenpairs are computed
constexpr int ALG_TRI_NE = ALG_TRI_MAX_RANK + 1;
constexpr float EIG_CLUSTER_TOL = 1e-3f; // eigenvalues closer than this (relative to the largest) are orthogonalised explicitly

// Number of eigenvalues of the symmetric tridiagonal matrix (diagonal a, off-diagonal b) that are smaller than x:
// the negative pivots of the LDL^T factorisation of T - x I.
template <int D>
__device__ __forceinline__ int sturm_count(const float *a, const float *b, float x, float pivmin)
{
    float q = a[0] - x;
    int cnt = q < 0.f ? 1 : 0;
#pragma unroll 4
    for (int i = 1; i < D; ++i) {
        if (fabsf(q) < pivmin) q = -pivmin;
        // the quotient need not be rounded correctly: an error of a few ulp moves the count's switching point by as much
        q = a[i] - x - __fdividef(b[i - 1] * b[i - 1], q);
        cnt += q < 0.f ? 1 : 0;
    }
    return cnt;
}

// Floats of the eigen-solver's workspace: tridiagonal form (diagonal, off-diagonal, eigenvalues, rank + 1 vectors
// with five factor arrays each), or the d x d eigenvector matrix of the Jacobi route, or two row blocks of the
// fixed-iteration route.
template <int D>
__host__ __device__ constexpr int algebra_eig_floats(int rank, int fast_iters)
{
    const int ne = (rank < D ? rank : D) + 1;
    const int tri = 2 * D + 16 + ne * D + ne * 5 * D;
    const int jac = D * (D + 1);
    const int fast = 2 * (rank < D ? rank : D) * (D + 1);
    return fast_iters > 0 ? fast : (rank <= ALG_TRI_MAX_RANK ? tri : jac);
}

// mcap: basis rows any head of the call can have, min(largest k_eff, D).
template <int D>
__host__ __device__ constexpr int algebra_region_floats(int mcap, int rank, int fast_iters)
{
    const int thin = mcap * (D + 1);                                // Q X of a projection
    const int eig = algebra_eig_floats<D>(rank, fast_iters);
    return mcap * (D + 1) + (thin > eig ? thin : eig);
}

template <int D>
inline size_t algebra_smem_bytes(int mcap, int rank, int fast_iters)
{
    return (size_t)(D * (D + 1) + 6 * D + 64 + algebra_region_floats<D>(mcap, rank, fast_iters)) * sizeof(float) +
           2 * D * sizeof(int);
}

template <typename TIN, int D>
__global__ void __launch_bounds__(ALG_NT, 2) k_obf_algebra(const __grid_constant__ CallDev p)
{
    constexpr int LD = D + 1;
    extern __shared__ float sm[];
    const int mcap = p.alg_rows;                   // basis rows any head of this call can have
    float *B2 = sm;                                // d x d: G, then M, then the reflectors in M's dead columns
    float *vw = B2 + D * LD, *vc = vw + D, *vu = vc + D, *vl = vu + D, *vcs = vl + D;  // vcs: 2*D/2 floats (c,s)
    float *red = vcs + D;                          // 32 floats
    float *misc = red + 32;                        // 32 floats
    int *ipq = reinterpret_cast<int *>(misc + 32); // D ints: pairs (p,q); then D ints: selected eigen-columns
    int *isel = ipq + D;
    float *Qb = reinterpret_cast<float *>(isel + D);   // basis rows of span(V_keep), mcap x LD; stays to the end
    float *Bm = Qb + mcap * LD;                    // Q X (m x d) of the two projections; the eigen-solvers reuse this
    float *WS = Bm;                                // workspace of the eigen-solvers

    const int g = blockIdx.x, tid = threadIdx.x;
    int ci, lh;
    locate(p, g, ci, lh);
    const CacheDev &c = p.c[ci];
    const int T = c.T, k = c.k_eff, S = p.gram_slots;
    const int n_del = gram_partial_count(p, c, lh);
    const float a_keep = p.sums[(size_t)g * 4], a_del = p.sums[(size_t)g * 4 + 1];
    const float alpha = a_del / (a_keep + p.eps);

    if (tid < D) {
        p.delta[(size_t)g * D + tid] = 0.f;
        if (c.delta_out) c.delta_out[(size_t)lh * D + tid] = 0.f;
    }
    const uint32_t hflag_in = p.hflag[g];          // written by k_span_test
    __syncthreads();
    if (tid == 0) p.hflag[g] = 0u;
    if (T - k == 0 || p.rank <= 0) return;

    uint32_t status = 0u;
    int m = 0;
    // c = Q x (vc) and x -= Q^T c for a vector x of d floats in shared memory: four threads per basis row / per
    // channel.  The thread's share of the row is cut so that the 32 lanes of a warp meet 32 different banks (rows are
    // d + 1 floats apart: lanes of neighbouring rows are one bank apart, the four threads of a row eight).
    auto q_dot = [&](const float *x, int rows) {
        const int j = tid >> 2, part = tid & 3;
        float sacc = 0.f;
        if (j < rows) {
            const float *qj = Qb + j * LD;
#pragma unroll 8
            for (int e = 0; e < D / 4; ++e) {
                const int cc = ((e >> 3) << 5) + part * 8 + (e & 7);
                sacc = fmaf(qj[cc], x[cc], sacc);
            }
        }
        sacc += __shfl_xor_sync(0xffffffffu, sacc, 1);
        sacc += __shfl_xor_sync(0xffffffffu, sacc, 2);
        if (part == 0 && j < rows) vc[j] = sacc;
    };
    auto q_minus = [&](float *x, int rows) {
        const int cc = tid >> 2, part = tid & 3;
        float sacc = 0.f;
        if (cc < D) {
            const int n_e = ((rows + 31) >> 5) << 3;
            for (int e = 0; e < n_e; ++e) {
                const int j = ((e >> 3) << 5) + part * 8 + (e & 7);
                if (j < rows) sacc = fmaf(vc[j], Qb[j * LD + cc], sacc);
            }
        }
        sacc += __shfl_xor_sync(0xffffffffu, sacc, 1);
        sacc += __shfl_xor_sync(0xffffffffu, sacc, 2);
        if (part == 0 && cc < D) x[cc] -= sacc;
    };
    float rcr = 0.f, lam1 = 0.f, lam_rho = 0.f, lam_next = 0.f, dnorm = 0.f, revr = 0.f, pc = 0.f;
    int rho = 0;
    bool done = false;

    // ---- 1. k_eff >= d: the span test kernel has already factorised G_keep --
    if (k >= D && (hflag_in & HFLAG_SPAN_FULL)) { m = D; done = true; pc = 1.f; status |= OBF_DEV_SKIPPED | OBF_DEV_SPAN_FULL; }

    // ---- 2. orthonormal basis of span(V_keep), Eq. 2 ------------------------
    float u_keep[U_LEVELS], sq_keep = 0.f;         // retained rows' share of u (channel tid, per mass level) and of tr G
#pragma unroll
    for (int l = 0; l < U_LEVELS; ++l) u_keep[l] = 0.f;
    if (!done) {
        const TIN *vk = reinterpret_cast<const TIN *>(c.v_out) + (size_t)lh * k * D;
        const float *A = p.scores + c.tok_off + (size_t)lh * T;
        const int32_t *idx = c.idx_out + (size_t)lh * k;
        // the next row and its mass are asked for while the current row is worked on
        float v_next = 0.f, a_next = 0.f;
        if (tid < D && k > 0) {
            v_next = to_f32(vk[tid]);
            if (p.gram_all) a_next = A[idx[0]];
        }
#pragma unroll 1
        for (int i = 0; i < k && m < D; ++i) {
            if (tid < D) {
                const float v = v_next, a = a_next;
                if (i + 1 < k) {
                    v_next = to_f32(vk[(size_t)(i + 1) * D + tid]);
                    if (p.gram_all) a_next = A[idx[i + 1]];
                }
                vw[tid] = v;
                if (p.gram_all) {
                    const int lev = u_level(a);
#pragma unroll
                    for (int l = 0; l < U_LEVELS; ++l)
                        if (l == lev) u_keep[l] = fmaf(a, v, u_keep[l]);
                }
            }
            __syncthreads();
            // the norms of a row are taken by every warp for itself (same sum, same order): no block reduction
            float np0 = 0.f;
            for (int cc = (tid & 31); cc < D; cc += 32) np0 = fmaf(vw[cc], vw[cc], np0);
            const float n0sq = warp_sum(np0);
            sq_keep += n0sq;
            const float n0 = sqrtf(n0sq);
            // Gram-Schmidt against the basis so far, a second time only when the first pass took away more than half of
            // the row's squared norm: what is left of a row that keeps more than that is orthogonal to the basis to
            // rounding already ("twice is enough", and once where nothing cancels)
            float n1 = 0.f;
            for (int pass = 0; pass < 2; ++pass) {
                q_dot(vw, m);
                __syncthreads();
                q_minus(vw, m);
                __syncthreads();
                float np1 = 0.f;
                for (int cc = (tid & 31); cc < D; cc += 32) np1 = fmaf(vw[cc], vw[cc], np1);
                const float n1sq = warp_sum(np1);
                n1 = sqrtf(n1sq);
                if (n1sq > 0.5f * n0sq) break;                      // the same in every thread
            }
            const float w1 = tid < D ? vw[tid] : 0.f;
            if (n1 > SPAN_ROW_TOL * n0 && n1 > 0.f) {
                // a head can only have more basis rows than the call's layout holds if they reach d (span full)
                if (m < mcap && tid < D) Qb[m * LD + tid] = w1 / n1;
                ++m;
            }
            __syncthreads();
        }
        if (m >= D) { done = true; pc = 1.f; status |= OBF_DEV_SKIPPED | OBF_DEV_SPAN_FULL; }
        else if (m > mcap) { done = true; status |= OBF_DEV_INTERNAL | OBF_DEV_SKIPPED; }   // cannot happen: m <= min(k, d)
    }

    if (!done) {
        // ---- 3. G, u; M = P G P and r_bar without forming P -----------------------
        for (int e = tid; e < D * D; e += ALG_NT) {
            float s = 0.f;
            for (int sp = 0; sp < n_del; ++sp) s += p.gram_d[((size_t)g * S + sp) * D * D + e];
            B2[(e / D) * LD + (e % D)] = s;
        }
        if (tid < D) {
            // per level: what the pass over V added up minus the retained rows' share; smallest masses first
            float s = 0.f;
            for (int l = 0; l < p.u_levels; ++l) {
                float sl = 0.f;
                for (int sp = 0; sp < n_del; ++sp) sl += p.uvec[(((size_t)g * S + sp) * p.u_levels + l) * D + tid];
                if (p.gram_all) {
#pragma unroll
                    for (int l2 = 0; l2 < U_LEVELS; ++l2)
                        if (l2 == l) sl -= u_keep[l2];
                }
                s += sl;
            }
            vu[tid] = s;
            if (c.diag) vw[tid] = p.svec[(size_t)g * D + tid];
        }
        __syncthreads();
        // x -> P x = x - Q^T (Q x) for the vector in `x` (d floats in shared memory), in place; vc is scratch
        auto project = [&](float *x) {
            q_dot(x, m);
            __syncthreads();
            q_minus(x, m);
            __syncthreads();
        };
        if (c.diag) {
            // projection cosine: s = sum of the deleted values, its part inside span(V_keep) is s - P s
            const float sv = tid < D ? vw[tid] : 0.f;
            project(vw);
            const float par = tid < D ? sv - vw[tid] : 0.f;
            const float ss = block_sum<ALG_NT>(sv * sv, red), pp = block_sum<ALG_NT>(par * par, red);
            const float sp = block_sum<ALG_NT>(sv * par, red);
            pc = (ss > 0.f && pp > 0.f) ? sp * rsqrtf(ss) * rsqrtf(pp) : 0.f;
        }
        // squared Frobenius norm of the deleted values (the denominator of RCR).  As a difference of two fp32 traces
        // it is resolved down to about 1e-6 of the squared norm of all values: below 1e-5 of it the deleted values
        // count as negligible beside the retained ones and nothing is injected.
        const float trAll = block_sum<ALG_NT>(tid < D ? B2[tid * LD + tid] : 0.f, red);
        const float trG = trAll - (p.gram_all ? sq_keep : 0.f);
        const bool del_negligible = p.gram_all && !(trG > 1e-5f * trAll);
        // M = (I - Q^T Q) G (I - Q^T Q) as two rank-m updates: B = Q X (m x d), X -= Q^T B, first on X = G from the
        // left, then on the transposed problem from the right (X is symmetric up to rounding, so "B = Q X^T")
        for (int side = 0; side < 2; ++side) {
            // B[j][c] = sum_a Q[j][a] X[a][c] (left) or sum_a Q[j][a] X[c][a] (right): a 1 x 4 register tile per thread,
            // its four columns d / 4 apart so that the lanes of a warp read neighbouring banks
            for (int t = tid; t < m * (D / 4); t += ALG_NT) {
                const int j = t / (D / 4), c0 = t % (D / 4);
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                const float *qj = Qb + j * LD;
                if (side == 0) {
#pragma unroll 4
                    for (int a = 0; a < D; ++a) {
                        const float qv = qj[a];
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[e] = fmaf(qv, B2[a * LD + c0 + e * (D / 4)], acc[e]);
                    }
                } else {
#pragma unroll 4
                    for (int a = 0; a < D; ++a) {
                        const float qv = qj[a];
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[e] = fmaf(qv, B2[(c0 + e * (D / 4)) * LD + a], acc[e]);
                    }
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) Bm[j * LD + c0 + e * (D / 4)] = acc[e];
            }
            __syncthreads();
            // left: X[a][c] -= sum_j Q[j][a] B[j][c];  right: X[a][c] -= sum_j B[j][a] Q[j][c].  4 x 4 tile per thread
            const float *Lf = side == 0 ? Qb : Bm, *Rf = side == 0 ? Bm : Qb;
            for (int t = tid; t < (D / 4) * (D / 4); t += ALG_NT) {
                const int a0 = (t / (D / 4)) * 4, c0 = t % (D / 4);       // rows a0 .. a0 + 3, columns c0 + e d / 4
                float acc[4][4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
                for (int j = 0; j < m; ++j) {
                    float l[4], r[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) { l[i] = Lf[j * LD + a0 + i]; r[i] = Rf[j * LD + c0 + i * (D / 4)]; }
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[i][e] = fmaf(l[i], r[e], acc[i][e]);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int e = 0; e < 4; ++e) B2[(a0 + i) * LD + c0 + e * (D / 4)] -= acc[i][e];
            }
            __syncthreads();
        }
        for (int e = tid; e < D * D; e += ALG_NT) {            // symmetrise
            const int a = e / D, bb = e % D;
            if (a < bb) {
                const float sy = 0.5f * (B2[a * LD + bb] + B2[bb * LD + a]);
                B2[a * LD + bb] = sy;
                B2[bb * LD + a] = sy;
            }
        }
        // r_bar = P u / (A_del + eps)
        project(vu);
        if (tid < D) vu[tid] = vu[tid] / (a_del + p.eps);
        __syncthreads();
        const float trM = block_sum<ALG_NT>(tid < D ? B2[tid * LD + tid] : 0.f, red);
        rcr = del_negligible ? 0.f : trM / (trG + p.eps);
        if (!(rcr >= RCR_SKIP_TOL)) { done = true; status |= OBF_DEV_SKIPPED; }

        // delta, projected once more off the basis rows, published and injected (Eq. 5-7): dl = this thread's channel
        auto finish_delta = [&](float dl) {
            if (tid < D) vw[tid] = dl;
            __syncthreads();
            project(vw);
            dl = tid < D ? vw[tid] : 0.f;
            const float dn2 = block_sum<ALG_NT>(dl * dl, red);
            dnorm = sqrtf(dn2);
            if (!isfinite(dn2)) { status |= OBF_DEV_NONFINITE | OBF_DEV_SKIPPED; dnorm = 0.f; }
            else if (rho == 0 || dn2 == 0.f) status |= OBF_DEV_SKIPPED;
            else {
                if (tid < D) {
                    p.delta[(size_t)g * D + tid] = dl;
                    if (c.delta_out) c.delta_out[(size_t)lh * D + tid] = dl;
                }
                if (tid == 0) p.hflag[g] = HFLAG_INJECT;
                // Eq. 7: V_out = V_keep + delta on every retained row; the fp32 sum is rounded once.  Attn-inject
                // (App. D.2): row t takes k * A_t / (A_keep + eps) times delta instead
                TIN *rows = reinterpret_cast<TIN *>(c.v_out) + (size_t)lh * k * D;
                const float *Am = p.scores + c.tok_off + (size_t)lh * T;
                const int32_t *ix = c.idx_out + (size_t)lh * k;
                const float share = (float)k / (a_keep + p.eps);
                for (int e = tid; e < k * D; e += ALG_NT) {
                    const float wgt = p.attn_inject ? share * Am[ix[e / D]] : 1.f;
                    const float sum = fmaf(wgt, vw[e % D], to_f32(rows[e]));
                    if constexpr (sizeof(TIN) == 4) rows[e] = sum;
                    else rows[e] = __float2bfloat16_rn(sum);
                }
            }
        };

        // ---- 4f. fast path of App. H: C <- orth(C M), a fixed number of times, from the first rows of the identity ----
        if (!done && p.fast_iters > 0) {
            const int lane = tid & 31, warp = tid >> 5;
            int rho_f = min(min(p.rank, D), D - m);               // rank(R) <= d - m
            float *C = WS, *Y = WS + min(p.rank, D) * LD;         // row blocks of length D (stride LD)
            for (int e = tid; e < rho_f * D; e += ALG_NT) C[(e / D) * LD + (e % D)] = (e / D == e % D) ? 1.f : 0.f;
            __syncthreads();
#pragma unroll 1
            for (int itn = 0; itn < p.fast_iters; ++itn) {
                for (int e = tid; e < rho_f * D; e += ALG_NT) {    // Y = C M
                    const int i = e / D, b = e % D;
                    float sacc = 0.f;
#pragma unroll 8
                    for (int a = 0; a < D; ++a) sacc = fmaf(C[i * LD + a], B2[a * LD + b], sacc);
                    Y[i * LD + b] = sacc;
                }
                __syncthreads();
                // orth: Gram-Schmidt over the rows in order, twice; a row with nothing left is dropped (warp 0)
                if (warp == 0) {
                    int kept = 0;
                    for (int i = 0; i < rho_f; ++i) {
                        float *y = Y + i * LD;
                        float n0 = 0.f;
                        for (int cc = lane; cc < D; cc += 32) n0 = fmaf(y[cc], y[cc], n0);
                        n0 = warp_sum(n0);
                        for (int pass = 0; pass < 2; ++pass)
                            for (int j = 0; j < kept; ++j) {
                                const float *qv = C + j * LD;
                                float dsum = 0.f;
                                for (int cc = lane; cc < D; cc += 32) dsum = fmaf(y[cc], qv[cc], dsum);
                                dsum = warp_sum(dsum);
                                for (int cc = lane; cc < D; cc += 32) y[cc] -= dsum * qv[cc];
                                __syncwarp();
                            }
                        float n1 = 0.f;
                        for (int cc = lane; cc < D; cc += 32) n1 = fmaf(y[cc], y[cc], n1);
                        n1 = warp_sum(n1);
                        if (n1 > 1e-10f * n0 && n1 > 0.f) {
                            const float inv = rsqrtf(n1);
                            for (int cc = lane; cc < D; cc += 32) C[kept * LD + cc] = y[cc] * inv;
                            ++kept;
                        }
                        __syncwarp();
                    }
                    if (lane == 0) misc[6] = (float)kept;
                }
                __syncthreads();
                rho_f = (int)misc[6];
            }
            rho = rho_f;
            // Rayleigh quotients of the rows (for the diagnostics), then Delta and delta
            if (warp < 16) {
                for (int i = warp; i < rho; i += 16) {
                    float rq = 0.f;
                    for (int a = lane; a < D; a += 32) {
                        float sacc = 0.f;
                        for (int b = 0; b < D; ++b) sacc = fmaf(B2[a * LD + b], C[i * LD + b], sacc);
                        rq = fmaf(C[i * LD + a], sacc, rq);
                    }
                    rq = warp_sum(rq);
                    if (lane == 0) vl[i] = rq;
                }
            }
            if (tid < rho) {
                float sacc = 0.f;
                for (int cc = 0; cc < D; ++cc) sacc = fmaf(C[tid * LD + cc], vu[cc], sacc);
                vc[tid] = sacc;
            }
            __syncthreads();
            for (int t = 0; t < rho; ++t) revr += vl[t];
            revr /= trM + p.eps;
            lam1 = rho > 0 ? vl[0] : 0.f; lam_rho = rho > 0 ? vl[rho - 1] : 0.f; lam_next = 0.f;
            float dl = 0.f;
            if (tid < D) {
                float sacc = 0.f;
                for (int t = 0; t < rho; ++t) sacc = fmaf(vc[t], C[t * LD + tid], sacc);
                dl = alpha * sacc;
            }
            __syncthreads();                                        // vc is scratch of the projection that follows
            finish_delta(dl);
            done = true;
        }

        // ---- 4a. few eigenpairs wanted: tridiagonal form, bisection, inverse iteration ----
        if (!done && p.rank <= ALG_TRI_MAX_RANK) {
            const int lane = tid & 31, warp = tid >> 5;
            const int ne = min(min(p.rank, D) + 1, D);             // eigenpairs computed: the wanted ones and the next
            float *ta = WS, *tb = WS + D;                          // diagonal, off-diagonal (tb[i] couples i and i + 1)
            float *tlam = tb + D;                                  // ne <= ALG_TRI_NE eigenvalues, largest first (16 floats)
            float *tz = tlam + 16;                                 // [ne][D] eigenvectors
            float *twk = tz + ne * D;                              // [ne][5][D] factors of T - lambda I
            // Householder reduction: reflector k (a unit vector) zeroes column k below the sub-diagonal.  During its step it
            // sits in one of two vectors (vl, vcs); afterwards in the part of column k of M that the step has emptied
            // (rows k + 1 .. d - 1).
            //
            // Two block barriers per column.  Step k:
            //   B  p = 2 M v_k on the trailing block (rows and columns > k), four threads per row;
            //   C  kk = v_k . p and w = p - kk v_k (every warp for itself), then
            //      - row k + 1 as the update M - v w^T - w v^T leaves it, formed by every warp for itself from the old row:
            //        its first entry is the next diagonal entry, the rest gives reflector k + 1 (norm, sign) at once, so
            //        no barrier stands between the update and the next reflector;
            //      - the update itself on rows and columns > k + 1 (row and column k + 1 are dead from here on; column
            //        k + 1 takes its reflector a step later);
            //      - reflector k into column k.
            // The loop starts at k = -1 with v = 0: that step only forms reflector 0 from row 0.
            const float tiny2 = 1e-20f * trM * trM;
            constexpr int RPW = (D + ALG_NT / 32 - 2) / (ALG_NT / 32 - 1);   // rows a warp of the update handles
            constexpr int CPL = (D + 31) / 32;                           // columns per lane
            if (tid < D) { vl[tid] = 0.f; vcs[tid] = 0.f; vc[tid] = 0.f; }
            __syncthreads();
#pragma unroll 1
            for (int k = -1; k < D - 2; ++k) {
                const float *v = (k & 1) ? vl : vcs;                // v_k; v_{k+1} goes to the other vector
                float *vnext = (k & 1) ? vcs : vl;
                if (k >= 0) {                                       // B: p = 2 M v on the trailing block -> vc
                    const int j = tid >> 2, part = tid & 3;
                    const bool on = j > k && j < D;
                    float s0 = 0.f, s1 = 0.f;
                    if (on) {
                        const float *row = B2 + j * LD;
                        // columns from the 32-column group of k + 1 on (v is zero up to k); the four threads of a row
                        // take eight columns of a group each, which keeps the lanes of a warp on different banks
#pragma unroll 1
                        for (int g32 = (k + 1) >> 5; g32 < D / 32; ++g32) {
                            const float *rw = row + (g32 << 5) + part * 8, *vv = v + (g32 << 5) + part * 8;
#pragma unroll
                            for (int i = 0; i < 8; i += 2) {
                                s0 = fmaf(rw[i], vv[i], s0);
                                s1 = fmaf(rw[i + 1], vv[i + 1], s1);
                            }
                        }
                    }
                    float sacc = s0 + s1;
                    sacc += __shfl_xor_sync(0xffffffffu, sacc, 1);
                    sacc += __shfl_xor_sync(0xffffffffu, sacc, 2);
                    if (on && part == 0) vc[j] = 2.f * sacc;
                    __syncthreads();
                }
                // C
                float kpart = 0.f;
                for (int cc = k + 1 + lane; cc < D; cc += 32) kpart = fmaf(v[cc], vc[cc], kpart);
                const float kk = warp_sum(kpart);                   // v . p, the same sum in every warp
                // groups of 32 columns the trailing block has (the same in every thread: whole groups are skipped)
                const int nc = (D - (k + 1) + 31) >> 5;
                float vj[CPL], wj[CPL];
#pragma unroll
                for (int cI = 0; cI < CPL; ++cI) {
                    vj[cI] = 0.f;
                    wj[cI] = 0.f;
                    if (cI < nc) {
                        const int j = k + 1 + lane + 32 * cI;
                        vj[cI] = j < D ? v[j] : 0.f;
                        wj[cI] = j < D ? vc[j] - kk * vj[cI] : 0.f;
                    }
                }
                if (warp == 0) {
                    // warp 0 forms reflector k + 1; the other warps share the update
                    float xj[CPL];
                    const float vr = v[k + 1], wr = vc[k + 1] - kk * vr;     // entries k + 1 of v and w
                    float part2 = 0.f;
#pragma unroll
                    for (int cI = 0; cI < CPL; ++cI) {
                        xj[cI] = 0.f;
                        if (cI < nc) {
                            const int j = k + 1 + lane + 32 * cI;
                            // row k + 1 after the update (the same expression as the update below)
                            xj[cI] = j < D ? B2[(k + 1) * LD + j] - (vr * wj[cI] + wr * vj[cI]) : 0.f;
                            if (j >= k + 3) part2 = fmaf(xj[cI], xj[cI], part2);
                        }
                    }
                    const float below2 = warp_sum(part2);              // squares right of the super-diagonal entry
                    const float dg = __shfl_sync(0xffffffffu, xj[0], 0);    // entry (k + 1, k + 1)
                    const float x0 = __shfl_sync(0xffffffffu, xj[0], 1);    // entry (k + 1, k + 2)
                    const float nrm2 = below2 + x0 * x0;
                    const float nrm = sqrtf(nrm2);
                    const float al = x0 >= 0.f ? -nrm : nrm;
                    const float vn2 = 2.f * nrm * (nrm + fabsf(x0));   // |x - al e_0|^2
                    const bool skip = !(below2 > tiny2) || !(vn2 > 0.f);   // nothing beyond the super-diagonal
                    const float rs = skip ? 0.f : rsqrtf(vn2);
#pragma unroll
                    for (int cI = 0; cI < CPL; ++cI) {
                        const int j = k + 1 + lane + 32 * cI;
                        if (cI < nc && j < D) vnext[j] = j == k + 1 ? 0.f : (j == k + 2 ? x0 - al : xj[cI]) * rs;
                    }
                    if (lane == 0) {
                        if (k >= 0) vnext[k] = 0.f;
                        ta[k + 1] = dg;
                        tb[k + 1] = skip ? x0 : al;
                    }
                }
                if (k >= 0 && warp > 0) {
                    // M <- H M H = M - v w^T - w v^T on rows and columns > k + 1; a warp's rows are read before the first
                    // is written back (the compiler cannot tell that they do not overlap), RB at a time
                    // RB = 1 measured fastest (0.60 ms on the paper's regime; 2: 0.63, 3: 0.66, 4: 0.68): registers, not
                    // the stores, are what the loop is short of
                    constexpr int RB = 1;
#pragma unroll
                    for (int r0 = 0; r0 < RPW; r0 += RB) {
                        // (the same in every lane of the warp: rows and column groups outside the block cost nothing)
                        if (k + 2 + (warp - 1) + r0 * (ALG_NT / 32 - 1) < D) {
                            float m_[RB][CPL], vi[RB], wi[RB];
#pragma unroll
                            for (int r = 0; r < RB; ++r) {
                                const int i = k + 2 + (warp - 1) + (r0 + r) * (ALG_NT / 32 - 1);
                                const bool on = r0 + r < RPW && i < D;
                                vi[r] = on ? v[i] : 0.f;
                                wi[r] = on ? vc[i] - kk * vi[r] : 0.f;
#pragma unroll
                                for (int cI = 0; cI < CPL; ++cI) {
                                    m_[r][cI] = 0.f;
                                    if (cI < nc) {
                                        const int j = k + 1 + lane + 32 * cI;
                                        m_[r][cI] = (on && j < D) ? B2[i * LD + j] : 0.f;
                                    }
                                }
                            }
#pragma unroll
                            for (int r = 0; r < RB; ++r) {
                                const int i = k + 2 + (warp - 1) + (r0 + r) * (ALG_NT / 32 - 1);
                                const bool on = r0 + r < RPW && i < D;
#pragma unroll
                                for (int cI = 0; cI < CPL; ++cI) {
                                    if (cI < nc) {
                                        const int j = k + 1 + lane + 32 * cI;
                                        if (on && j > k + 1 && j < D) B2[i * LD + j] = m_[r][cI] - (vi[r] * wj[cI] + wi[r] * vj[cI]);
                                    }
                                }
                            }
                        }
                    }
                }
                // reflector k into the column it has emptied
                if (k >= 0 && tid > k && tid < D) B2[tid * LD + k] = v[tid];
                __syncthreads();
            }
            if (tid == 0) { ta[D - 1] = B2[(D - 1) * LD + D - 1]; tb[D - 1] = 0.f; }
            __syncthreads();
            // bounds of the spectrum (Gershgorin) and the pivot floor of the Sturm counts
            float gl = INFINITY, gh = -INFINITY, b2 = 0.f;
            if (tid < D) {
                const float r = (tid > 0 ? fabsf(tb[tid - 1]) : 0.f) + fabsf(tb[tid]);
                gl = ta[tid] - r; gh = ta[tid] + r; b2 = tb[tid] * tb[tid];
            }
            const float g_hi = block_max<ALG_NT>(gh, red), g_lo = -block_max<ALG_NT>(-gl, red);
            const float pivmin = 1e-30f * fmaxf(1.f, block_max<ALG_NT>(b2, red));
            const float span = fmaxf(g_hi - g_lo, 1e-30f);
            // eigenvalue j (largest first) by 32-way multisection, one warp per eigenvalue
            if (warp < ne) {
                const int want = D - 1 - warp;                      // it has exactly `want` eigenvalues below it
                float lo = g_lo - 1e-3f * span, hi = g_hi + 1e-3f * span;
#pragma unroll 1
                for (int round = 0; round < 6; ++round) {                // 33^-6 of the spectrum's width: below fp32 resolution
                    const float x = lo + (hi - lo) * (float)(lane + 1) * (1.f / 33.f);
                    const bool below = sturm_count<D>(ta, tb, x, pivmin) <= want;     // x is not above the eigenvalue
                    const int nl = __popc(__ballot_sync(0xffffffffu, below));        // counts are monotone in x
                    const float x_lo = __shfl_sync(0xffffffffu, x, max(nl - 1, 0));
                    const float x_hi = __shfl_sync(0xffffffffu, x, min(nl, 31));
                    if (nl > 0) lo = x_lo;
                    if (nl < 32) hi = x_hi;
                }
                if (lane == 0) tlam[warp] = 0.5f * (lo + hi);
            }
            __syncthreads();
            const float l1 = tlam[0];
            // inverse iteration on T: factor T - lambda_j I once (LU with row interchanges), three solves
            if (warp < ne) {
                const float lam = tlam[warp];
                float *dd = twk + (warp * 5) * D, *dl = dd + D, *du = dl + D, *du2 = du + D, *pv = du2 + D;
                const float pert = 4e-7f * fmaxf(fabsf(g_hi), fabsf(g_lo)) + 1e-30f;
                for (int i = lane; i < D; i += 32) { dd[i] = ta[i] - lam; dl[i] = tb[i]; du[i] = tb[i]; du2[i] = 0.f; }
                __syncwarp();
                if (lane == 0) {
                    // the running pivot and the entry above the next one travel in registers: a step of the chain is a
                    // reciprocal and two multiply-adds, not a round trip through shared memory
                    float di = dd[0], ui = du[0];
                    for (int i = 0; i < D - 1; ++i) {
                        const float li = dl[i];
                        float dn = dd[i + 1], un = i < D - 2 ? du[i + 1] : 0.f;
                        if (fabsf(di) >= fabsf(li)) {
                            if (di == 0.f) di = pert;
                            const float f = __fdividef(li, di);
                            dd[i] = di; dl[i] = f; pv[i] = 0.f;
                            dn -= f * ui;
                        } else {
                            const float f = __fdividef(di, li);
                            dd[i] = li; dl[i] = f; du[i] = dn;
                            dn = ui - f * dn;
                            if (i < D - 2) { du2[i] = un; un = -f * un; }
                            pv[i] = 1.f;
                        }
                        di = dn; ui = un;
                        if (i < D - 2) du[i + 1] = un;
                    }
                    dd[D - 1] = di == 0.f ? pert : di;
                }
                __syncwarp();
                // the solves multiply by the pivots' reciprocals
                for (int i = lane; i < D; i += 32) {
                    float dv = dd[i];
                    if (fabsf(dv) < pert) dv = dv < 0.f ? -pert : pert;
                    dd[i] = 1.f / dv;
                }
            }
            if (warp < ne) {
                float *y = tz + warp * D;
                for (int i = lane; i < D; i += 32) {                // a start vector without structure
                    const uint32_t hsh = ((uint32_t)i * 2654435761u + (uint32_t)warp * 40503u + 12345u) >> 8;
                    y[i] = (float)(hsh & 0xFFFFu) * (1.f / 65536.f) - 0.5f;
                }
            }
            __syncthreads();
#pragma unroll 1
            for (int itn = 0; itn < 3; ++itn) {
                if (warp < ne) {
                    float *y = tz + warp * D;
                    if (lane == 0) {
                        // dd holds the reciprocals of the pivots; the value a step hands to the next stays in a register
                        const float *dd = twk + (warp * 5) * D, *dl = dd + D, *du = dl + D, *du2 = du + D, *pv = du2 + D;
                        float yi = y[0];
                        for (int i = 0; i < D - 1; ++i) {
                            const float yn = y[i + 1];
                            if (pv[i] == 0.f) { y[i] = yi; yi = yn - dl[i] * yi; }
                            else { y[i] = yn; yi = yi - dl[i] * yn; }
                        }
                        float y1 = yi * dd[D - 1];                               // y[i + 1]
                        y[D - 1] = y1;
                        float y0 = (y[D - 2] - du[D - 2] * y1) * dd[D - 2];      // y[i]
                        y[D - 2] = y0;
                        for (int i = D - 3; i >= 0; --i) {
                            const float t = (y[i] - du[i] * y0 - du2[i] * y1) * dd[i];
                            y[i] = t;
                            y1 = y0;
                            y0 = t;
                        }
                    }
                    __syncwarp();
                    // scaled to largest entry 1 by the whole warp
                    float mx = 0.f;
                    for (int i = lane; i < D; i += 32) mx = fmaxf(mx, fabsf(y[i]));
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                    const float sc1 = mx > 0.f ? 1.f / mx : 1.f;
                    for (int i = lane; i < D; i += 32) y[i] *= sc1;
                }
                __syncthreads();
                if (warp == 0) {
                    // in order of the eigenvalues: orthogonal to the close neighbours before it, unit length
                    for (int j = 0; j < ne; ++j) {
                        float *y = tz + j * D;
                        for (int i2 = 0; i2 < j; ++i2) {
                            if (fabsf(tlam[i2] - tlam[j]) > EIG_CLUSTER_TOL * fabsf(l1)) continue;
                            const float *z = tz + i2 * D;
                            float dsum = 0.f;
                            for (int cc = lane; cc < D; cc += 32) dsum = fmaf(y[cc], z[cc], dsum);
                            dsum = warp_sum(dsum);
                            for (int cc = lane; cc < D; cc += 32) y[cc] -= dsum * z[cc];
                            __syncwarp();
                        }
                        float n2 = 0.f;
                        for (int cc = lane; cc < D; cc += 32) n2 = fmaf(y[cc], y[cc], n2);
                        n2 = warp_sum(n2);
                        const float inv = n2 > 0.f ? rsqrtf(n2) : 0.f;
                        for (int cc = lane; cc < D; cc += 32) y[cc] *= inv;
                        __syncwarp();
                    }
                }
                __syncthreads();
            }
            // back through the reflectors: z = H_0 H_1 ... H_{D-3} y, one warp per vector, two reflectors per step:
            // H_{k-1} H_k z = z - 2 a v_k - 2 (b - 2 c a) v_{k-1} with a = v_k . z, b = v_{k-1} . z, c = v_{k-1} . v_k,
            // so that the three sums of a pair go through the warp together (half as many dependent reductions)
            static_assert(D % 2 == 0, "the reflectors are taken in pairs");
            if (warp < ne) {
                float *y = tz + warp * D;
                constexpr int CPLB = (D + 31) / 32;
#pragma unroll 1
                for (int k = D - 3; k >= 1; k -= 2) {
                    // reflector k: column k of B2 below the diagonal; reflector k - 1: column k - 1 from row k on
                    float vk[CPLB], vm[CPLB], zz[CPLB];
                    float a = 0.f, b = 0.f, cdot = 0.f;
#pragma unroll
                    for (int cI = 0; cI < CPLB; ++cI) {
                        const int cc = k + lane + 32 * cI;
                        vk[cI] = (cc > k && cc < D) ? B2[cc * LD + k] : 0.f;
                        vm[cI] = cc < D ? B2[cc * LD + k - 1] : 0.f;
                        zz[cI] = cc < D ? y[cc] : 0.f;
                        a = fmaf(vk[cI], zz[cI], a);
                        b = fmaf(vm[cI], zz[cI], b);
                        cdot = fmaf(vm[cI], vk[cI], cdot);
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        a += __shfl_xor_sync(0xffffffffu, a, o);
                        b += __shfl_xor_sync(0xffffffffu, b, o);
                        cdot += __shfl_xor_sync(0xffffffffu, cdot, o);
                    }
                    const float fa = 2.f * a, fb = 2.f * (b - 2.f * cdot * a);
#pragma unroll
                    for (int cI = 0; cI < CPLB; ++cI) {
                        const int cc = k + lane + 32 * cI;
                        if (cc < D) y[cc] = zz[cI] - fa * vk[cI] - fb * vm[cI];
                    }
                    __syncwarp();
                }
            }
            __syncthreads();
            // ---- 5a. Delta, delta from the wanted eigenvectors ----------------------------------
            const int rmax = min(p.rank, D);
            rho = 0;
            while (rho < rmax && rho < ne && tlam[rho] > EIG_RANK_TOL * l1 && tlam[rho] > 0.f) ++rho;
            lam1 = l1; lam_rho = rho > 0 ? tlam[rho - 1] : 0.f; lam_next = rho < ne ? fmaxf(tlam[rho], 0.f) : 0.f;
            for (int t = 0; t < rho; ++t) revr += tlam[t];
            revr /= trM + p.eps;                                    // trace of M = sum of all its eigenvalues
            if (tid < rho) {
                float sacc = 0.f;
                for (int cc = 0; cc < D; ++cc) sacc = fmaf(tz[tid * D + cc], vu[cc], sacc);
                vc[tid] = sacc;
            }
            __syncthreads();
            float dl = 0.f;
            if (tid < D) {
                float sacc = 0.f;
                for (int t = 0; t < rho; ++t) sacc = fmaf(vc[t], tz[t * D + tid], sacc);
                dl = alpha * sacc;
            }
            __syncthreads();                                        // vc is scratch of the projection that follows
            finish_delta(dl);
            done = true;
        }

        // ---- 4b. Jacobi eigen-decomposition of M (B2), eigenvectors in U (workspace) -----
        if (!done) {
            float *U = WS;                                          // d x d, starts as the identity
            for (int e = tid; e < D * D; e += ALG_NT) U[(e / D) * LD + (e % D)] = (e / D == e % D) ? 1.f : 0.f;
            __syncthreads();
            // rotations below the fp32 noise level of the largest eigenvalue never settle: stop there
            const float floor_abs = 2e-7f * block_max<ALG_NT>(tid < D ? B2[tid * LD + tid] : 0.f, red);
            bool converged = false;
#pragma unroll 1
            for (int sweep = 0; sweep < JACOBI_MAX_SWEEPS && !converged; ++sweep) {
                if (tid == 0) misc[0] = 0.f;
                __syncthreads();
#pragma unroll 1
                for (int r = 0; r < D - 1; ++r) {
                    if (tid < D / 2) {
                        int pp, qq;
                        if (tid == 0) { pp = D - 1; qq = r; }
                        else { pp = (r + tid) % (D - 1); qq = (r - tid + (D - 1)) % (D - 1); }
                        if (pp > qq) { const int t = pp; pp = qq; qq = t; }
                        const float app = B2[pp * LD + pp], aqq = B2[qq * LD + qq], apq = B2[pp * LD + qq];
                        float cs = 1.f, sn = 0.f;
                        if (fabsf(apq) > 1e-7f * sqrtf(fabsf(app * aqq)) + floor_abs) {
                            const float theta = (aqq - app) / (2.f * apq);
                            const float t = (theta >= 0.f ? 1.f : -1.f) / (fabsf(theta) + sqrtf(theta * theta + 1.f));
                            cs = rsqrtf(t * t + 1.f);
                            sn = t * cs;
                            misc[0] = 1.f;
                        }
                        vcs[2 * tid] = cs; vcs[2 * tid + 1] = sn;
                        ipq[2 * tid] = pp; ipq[2 * tid + 1] = qq;
                    }
                    __syncthreads();
                    for (int e = tid; e < D * (D / 2); e += ALG_NT) {      // columns of M and U
                        const int i = e / (D / 2), t = e % (D / 2);
                        const float cs = vcs[2 * t], sn = vcs[2 * t + 1];
                        if (sn != 0.f) {
                            const int pp = ipq[2 * t], qq = ipq[2 * t + 1];
                            const float mp = B2[i * LD + pp], mq = B2[i * LD + qq];
                            B2[i * LD + pp] = cs * mp - sn * mq;
                            B2[i * LD + qq] = sn * mp + cs * mq;
                            const float up = U[i * LD + pp], uq = U[i * LD + qq];
                            U[i * LD + pp] = cs * up - sn * uq;
                            U[i * LD + qq] = sn * up + cs * uq;
                        }
                    }
                    __syncthreads();
                    for (int e = tid; e < D * (D / 2); e += ALG_NT) {      // rows of M
                        const int t = e / D, j = e % D;
                        const float cs = vcs[2 * t], sn = vcs[2 * t + 1];
                        if (sn != 0.f) {
                            const int pp = ipq[2 * t], qq = ipq[2 * t + 1];
                            const float mp = B2[pp * LD + j], mq = B2[qq * LD + j];
                            B2[pp * LD + j] = cs * mp - sn * mq;
                            B2[qq * LD + j] = sn * mp + cs * mq;
                        }
                    }
                    __syncthreads();
                }
                converged = (misc[0] == 0.f);
                __syncthreads();
            }
            if (!converged) status |= OBF_DEV_NO_CONVERGE;

            // ---- 5. top-rank eigenvectors, Delta, delta ----------------------
            if (tid < D) vl[tid] = B2[tid * LD + tid];
            __syncthreads();
            if (tid == 0) {
                float l1 = 0.f;
                for (int i = 0; i < D; ++i) l1 = fmaxf(l1, vl[i]);
                int n = 0;
                float last = 0.f, kept = 0.f;
                const int rmax = min(p.rank, D);
                while (n < rmax) {
                    int b = -1; float best = EIG_RANK_TOL * l1;
                    for (int i = 0; i < D; ++i) if (vl[i] > best) { best = vl[i]; b = i; }
                    if (b < 0) break;
                    isel[n++] = b; last = vl[b]; kept += vl[b]; vl[b] = -1.f;
                }
                float nxt = 0.f;
                for (int i = 0; i < D; ++i) nxt = fmaxf(nxt, vl[i]);
                misc[1] = l1; misc[2] = last; misc[3] = nxt; misc[4] = (float)n; misc[5] = kept;
            }
            __syncthreads();
            lam1 = misc[1]; lam_rho = misc[2]; lam_next = misc[3]; rho = (int)misc[4];
            revr = misc[5] / (trM + p.eps);
            if (tid < rho) {
                const int col = isel[tid];
                float s = 0.f;
                for (int cc = 0; cc < D; ++cc) s = fmaf(U[cc * LD + col], vu[cc], s);
                vc[tid] = s;
            }
            __syncthreads();
            float dl = 0.f;
            if (tid < D) {
                float s = 0.f;
                for (int t = 0; t < rho; ++t) s = fmaf(vc[t], U[tid * LD + isel[t]], s);
                dl = alpha * s;
            }
            __syncthreads();                                        // vc is scratch of the projection that follows
            finish_delta(dl);
        }
    }

    if (tid == 0) {
        if (status & (OBF_DEV_NONFINITE | OBF_DEV_NO_CONVERGE)) atomicOr(p.status, status & 0xFFu);
        if (c.diag) {
            obf_diag_t *dg = c.diag + lh;
            dg->rcr = rcr; dg->delta_norm = dnorm;
            dg->lam_1 = lam1; dg->lam_rho = lam_rho; dg->lam_next = lam_next;
            dg->span_rank = m; dg->rho_eff = rho; dg->status = status;
            dg->revr = revr; dg->pc = pc;
        }
    }
}

}  // namespace obf
