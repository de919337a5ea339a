// Per-head dense algebra of Orthogonal BackFill (Eq. 2-6), one thread block per
// (cache, layer, KV head), everything in fp32 in shared memory.
//
// Inputs (from the streaming pass): Gram of the deleted values G_del, Gram of the
// retained values G_keep (only when k_eff >= d), u = sum_del A_j v_j, the demand
// sums, and the retained rows themselves (read back from v_out).
//
//   1. k_eff >= d: k_span_test has factorised G_keep (Cholesky).  If every pivot
//      stayed above 1e-3 of its diagonal entry the retained values span R^d, the
//      residual of Eq. 3 is identically zero and delta = 0.
//   2. Otherwise: orthonormal basis Q of span(V_keep) (Eq. 2) by twice-iterated
//      Gram-Schmidt over the retained rows; a row adds a direction when what is
//      left of it exceeds 1e-4 of its own norm.
//   3. P = I - Q^T Q,  M = P G_del P = R^T R  (Eq. 3 in Gram form, App. H),
//      r_bar = P u / (A_del + eps)  (Eq. 4).
//   4. Symmetric eigen-decomposition of M by parallel-order Jacobi rotations run
//      to convergence; C = eigenvectors of the `rank` largest eigenvalues above
//      1e-5 of the largest.
//   5. Delta = C^T C r_bar (Eq. 5), delta = A_del / (A_keep + eps) * Delta (Eq. 6),
//      V_out = V_keep + delta on the head's retained rows (Eq. 7).
#pragma once

#include "common.cuh"
#include "span_test.cuh"

namespace obf {

constexpr int ALG_NT = 512;
constexpr float SPAN_ROW_TOL = 1e-4f;
constexpr float RCR_SKIP_TOL = 1e-6f;
constexpr float EIG_RANK_TOL = 1e-5f;
constexpr int JACOBI_MAX_SWEEPS = 30;

template <int D>
constexpr size_t algebra_smem_bytes() { return (size_t)(3 * D * (D + 1) + 6 * D + 64) * sizeof(float) + 2 * D * sizeof(int); }

template <typename TIN, int D>
__global__ void __launch_bounds__(ALG_NT) k_obf_algebra(const __grid_constant__ CallDev p)
{
    constexpr int LD = D + 1;
    extern __shared__ float sm[];
    float *B0 = sm, *B1 = B0 + D * LD, *B2 = B1 + D * LD;
    float *vw = B2 + D * LD, *vc = vw + D, *vu = vc + D, *vl = vu + D, *vcs = vl + D;  // vcs: 2*D/2 floats (c,s)
    float *red = vcs + D;                          // 32 floats
    float *misc = red + 32;                        // 32 floats
    int *ipq = reinterpret_cast<int *>(misc + 32); // D ints: pairs (p,q); then D ints: selected eigen-columns
    int *isel = ipq + D;

    const int g = blockIdx.x, tid = threadIdx.x;
    int ci, lh;
    locate(p, g, ci, lh);
    const CacheDev &c = p.c[ci];
    const int T = c.T, k = c.k_eff, S = p.gram_slots;
    const int n_del = gram_partial_count(p, c, lh, 0), n_keep = gram_partial_count(p, c, lh, 1);
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
    float rcr = 0.f, lam1 = 0.f, lam_rho = 0.f, lam_next = 0.f, dnorm = 0.f;
    int rho = 0;
    bool done = false;

    // ---- 1. k_eff >= d: the span test kernel has already factorised G_keep --
    if (k >= D && (hflag_in & HFLAG_SPAN_FULL)) { m = D; done = true; status |= OBF_DEV_SKIPPED | OBF_DEV_SPAN_FULL; }

    // ---- 2. orthonormal basis of span(V_keep), Eq. 2 ------------------------
    if (!done) {
        const TIN *vk = reinterpret_cast<const TIN *>(c.v_out) + (size_t)lh * k * D;
#pragma unroll 1
        for (int i = 0; i < k && m < D; ++i) {
            if (tid < D) vw[tid] = to_f32(vk[(size_t)i * D + tid]);
            __syncthreads();
            const float w0 = tid < D ? vw[tid] : 0.f;
            const float n0 = sqrtf(block_sum<ALG_NT>(w0 * w0, red));
            for (int pass = 0; pass < 2; ++pass) {
                {
                    const int j = tid >> 2, part = tid & 3;
                    float s = 0.f;
                    if (j < m) {
                        const float *qj = B0 + j * LD + part * (D / 4);
                        const float *ww = vw + part * (D / 4);
#pragma unroll 8
                        for (int e = 0; e < D / 4; ++e) s = fmaf(qj[e], ww[e], s);
                    }
                    s += __shfl_xor_sync(0xffffffffu, s, 1);
                    s += __shfl_xor_sync(0xffffffffu, s, 2);
                    if (part == 0 && j < m) vc[j] = s;
                }
                __syncthreads();
                {
                    const int cc = tid >> 2, part = tid & 3;
                    float s = 0.f;
                    if (cc < D)
                        for (int j = part; j < m; j += 4) s = fmaf(vc[j], B0[j * LD + cc], s);
                    s += __shfl_xor_sync(0xffffffffu, s, 1);
                    s += __shfl_xor_sync(0xffffffffu, s, 2);
                    if (part == 0 && cc < D) vw[cc] -= s;
                }
                __syncthreads();
            }
            const float w1 = tid < D ? vw[tid] : 0.f;
            const float n1 = sqrtf(block_sum<ALG_NT>(w1 * w1, red));
            if (n1 > SPAN_ROW_TOL * n0 && n1 > 0.f) {
                if (tid < D) B0[m * LD + tid] = w1 / n1;
                ++m;
            }
            __syncthreads();
        }
        if (m >= D) { done = true; status |= OBF_DEV_SKIPPED | OBF_DEV_SPAN_FULL; }
    }

    if (!done) {
        // ---- 3. P = I - Q^T Q; M = P G_del P; r_bar --------------------------
        for (int e = tid; e < D * D; e += ALG_NT) {
            const int a = e / D, b = e % D;
            float s = 0.f;
            for (int j = 0; j < m; ++j) s = fmaf(B0[j * LD + a], B0[j * LD + b], s);
            B1[a * LD + b] = (a == b ? 1.f : 0.f) - s;
        }
        for (int e = tid; e < D * D; e += ALG_NT) {
            float s = 0.f;
            for (int sp = 0; sp < n_del; ++sp) s += p.gram_d[((size_t)g * S + sp) * D * D + e];
            B2[(e / D) * LD + (e % D)] = s;
        }
        if (tid < D) {
            float s = 0.f;
            for (int sp = 0; sp < n_del * p.u_groups; ++sp) s += p.uvec[((size_t)g * S * p.u_groups + sp) * D + tid];
            vu[tid] = s;
        }
        __syncthreads();
        const float trG = block_sum<ALG_NT>(tid < D ? B2[tid * LD + tid] : 0.f, red);
        for (int e = tid; e < D * D; e += ALG_NT) {            // W = G_del P  -> B0
            const int a = e / D, b = e % D;
            float s = 0.f;
#pragma unroll 8
            for (int cc = 0; cc < D; ++cc) s = fmaf(B2[a * LD + cc], B1[cc * LD + b], s);
            B0[a * LD + b] = s;
        }
        __syncthreads();
        for (int e = tid; e < D * D; e += ALG_NT) {            // M = P W -> B2
            const int a = e / D, b = e % D;
            float s = 0.f;
#pragma unroll 8
            for (int cc = 0; cc < D; ++cc) s = fmaf(B1[a * LD + cc], B0[cc * LD + b], s);
            B2[a * LD + b] = s;
        }
        if (tid < D) {                                          // r_bar = P u / (A_del + eps)
            float s = 0.f;
            for (int cc = 0; cc < D; ++cc) s = fmaf(B1[tid * LD + cc], vu[cc], s);
            vc[tid] = s / (a_del + p.eps);
        }
        __syncthreads();
        if (tid < D) vu[tid] = vc[tid];
        for (int e = tid; e < D * D; e += ALG_NT) {            // symmetrise
            const int a = e / D, b = e % D;
            if (a < b) {
                const float s = 0.5f * (B2[a * LD + b] + B2[b * LD + a]);
                B2[a * LD + b] = s;
                B2[b * LD + a] = s;
            }
        }
        for (int e = tid; e < D * D; e += ALG_NT) B1[(e / D) * LD + (e % D)] = (e / D == e % D) ? 1.f : 0.f;
        __syncthreads();
        const float trM = block_sum<ALG_NT>(tid < D ? B2[tid * LD + tid] : 0.f, red);
        rcr = trM / (trG + p.eps);
        if (!(rcr >= RCR_SKIP_TOL)) { done = true; status |= OBF_DEV_SKIPPED; }

        // ---- 4. Jacobi eigen-decomposition of M (B2), eigenvectors in B1 -----
        if (!done) {
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
                            const float up = B1[i * LD + pp], uq = B1[i * LD + qq];
                            B1[i * LD + pp] = cs * up - sn * uq;
                            B1[i * LD + qq] = sn * up + cs * uq;
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
                float last = 0.f;
                const int rmax = min(p.rank, D);
                while (n < rmax) {
                    int b = -1; float best = EIG_RANK_TOL * l1;
                    for (int i = 0; i < D; ++i) if (vl[i] > best) { best = vl[i]; b = i; }
                    if (b < 0) break;
                    isel[n++] = b; last = vl[b]; vl[b] = -1.f;
                }
                float nxt = 0.f;
                for (int i = 0; i < D; ++i) nxt = fmaxf(nxt, vl[i]);
                misc[1] = l1; misc[2] = last; misc[3] = nxt; misc[4] = (float)n;
            }
            __syncthreads();
            lam1 = misc[1]; lam_rho = misc[2]; lam_next = misc[3]; rho = (int)misc[4];
            if (tid < rho) {
                const int col = isel[tid];
                float s = 0.f;
                for (int cc = 0; cc < D; ++cc) s = fmaf(B1[cc * LD + col], vu[cc], s);
                vc[tid] = s;
            }
            __syncthreads();
            float dl = 0.f;
            if (tid < D) {
                float s = 0.f;
                for (int t = 0; t < rho; ++t) s = fmaf(vc[t], B1[tid * LD + isel[t]], s);
                dl = alpha * s;
            }
            const float dn2 = block_sum<ALG_NT>(dl * dl, red);
            dnorm = sqrtf(dn2);
            if (!isfinite(dn2)) { status |= OBF_DEV_NONFINITE | OBF_DEV_SKIPPED; dnorm = 0.f; }
            else if (rho == 0 || dn2 == 0.f) status |= OBF_DEV_SKIPPED;
            else {
                if (tid < D) {
                    p.delta[(size_t)g * D + tid] = dl;
                    if (c.delta_out) c.delta_out[(size_t)lh * D + tid] = dl;
                    vw[tid] = dl;
                }
                if (tid == 0) p.hflag[g] = HFLAG_INJECT;
                __syncthreads();
                // Eq. 7: V_out = V_keep + delta on every retained row; the fp32 sum is rounded once
                TIN *rows = reinterpret_cast<TIN *>(c.v_out) + (size_t)lh * k * D;
                for (int e = tid; e < k * D; e += ALG_NT) {
                    const float sum = to_f32(rows[e]) + vw[e % D];
                    if constexpr (sizeof(TIN) == 4) rows[e] = sum;
                    else rows[e] = __float2bfloat16_rn(sum);
                }
            }
        }
    }

    if (tid == 0) {
        if (status & (OBF_DEV_NONFINITE | OBF_DEV_NO_CONVERGE)) atomicOr(p.status, status & 0xFFu);
        if (c.diag) {
            obf_diag_t *dg = c.diag + lh;
            dg->rcr = rcr; dg->delta_norm = dnorm;
            dg->lam_1 = lam1; dg->lam_rho = lam_rho; dg->lam_next = lam_next;
            dg->span_rank = m; dg->rho_eff = rho; dg->status = status;
        }
    }
}

}  // namespace obf
