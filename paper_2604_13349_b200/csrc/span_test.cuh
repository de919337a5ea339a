// Span test of Orthogonal BackFill for budgets k_eff >= head_dim: does span(V_keep)
// (Eq. 2) fill all of R^d?  If it does, the residual of Eq. 3 is identically zero
// and delta = 0, whatever the deleted values are.
//
// The test is a Cholesky factorisation of G_keep = V_keep^T V_keep without
// pivoting: pivot j is the squared distance of value channel j from the span of
// channels 0..j-1 (over the retained rows); the span is declared full when every
// pivot stays above CHOL_PIVOT_TOL of the channel's own squared norm.  One block
// per (cache, layer, KV head); right-looking blocked algorithm with 32-wide
// panels: the diagonal block is factorised by one warp in registers, the panel
// below it by one thread per row, the trailing matrix by 4x4 register tiles.
// Result: bit 1 of hflag[head].
#pragma once

#include "common.cuh"

namespace obf {

constexpr int ST_NT = 256;
constexpr float CHOL_PIVOT_TOL = 1e-3f;
constexpr uint32_t HFLAG_INJECT = 1u;      // delta != 0: the injection kernel has work for this head
constexpr uint32_t HFLAG_SPAN_FULL = 2u;   // span(V_keep) = R^d

template <int D>
constexpr size_t span_smem_bytes() { return (size_t)(D * (D + 1) + 32 * 32 + 32 + D) * sizeof(float); }

template <int D>
__global__ void __launch_bounds__(ST_NT) k_span_test(const __grid_constant__ CallDev p)
{
    constexpr int LD = D + 1, NB = 32;
    extern __shared__ float st_sm[];
    float *A = st_sm;                  // D x LD, lower triangle is what counts
    float *L11 = A + D * LD;           // 32 x 32 factor of the current diagonal block (16-byte aligned)
    float *rinv = L11 + NB * NB;       // 32 reciprocals of its diagonal
    float *d0 = rinv + NB;             // D original diagonal entries
    __shared__ int s_ok;

    const int g = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int ci, lh;
    locate(p, g, ci, lh);
    const CacheDev &c = p.c[ci];
    const bool need = p.rank > 0 && c.T > c.k_eff && c.k_eff >= D;
    if (!need) {
        if (tid == 0) p.hflag[g] = 0u;
        return;
    }
    const int n_part = gram_partial_count(p, c, lh, 1);
    const float *parts = p.gram_k + (size_t)g * p.gram_slots * D * D;
    for (int e4 = tid; e4 < D * D / 4; e4 += ST_NT) {
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sp = 0; sp < n_part; ++sp) {
            const float4 v = *reinterpret_cast<const float4 *>(parts + (size_t)sp * D * D + e4 * 4);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        const int r = (e4 * 4) / D, cc = (e4 * 4) % D;
        float *o = A + r * LD + cc;
        o[0] = s.x; o[1] = s.y; o[2] = s.z; o[3] = s.w;
    }
    if (tid == 0) s_ok = 1;
    __syncthreads();
    if (tid < D) d0[tid] = A[tid * LD + tid];
    __syncthreads();

#pragma unroll 1
    for (int j0 = 0; j0 < D; j0 += NB) {
        const int nrem = D - j0 - NB;                      // rows below the diagonal block
        if (warp == 0) {
            // lane i owns row i of the diagonal block
            float a[NB];
#pragma unroll
            for (int cc = 0; cc < NB; ++cc) a[cc] = cc <= lane ? A[(j0 + lane) * LD + j0 + cc] : 0.f;
            bool ok = true;
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                const float piv = __shfl_sync(0xffffffffu, a[j], j);
                ok = ok && (piv > CHOL_PIVOT_TOL * d0[j0 + j]) && (piv > 0.f);
                const float inv = rsqrtf(piv);
                const float l = a[j] * inv;                  // lanes >= j: L[lane][j]
                a[j] = l;
#pragma unroll
                for (int cc = j + 1; cc < NB; ++cc) {
                    const float lc = __shfl_sync(0xffffffffu, l, cc);   // L[cc][j]
                    a[cc] = fmaf(-l, lc, a[cc]);
                }
            }
#pragma unroll
            for (int cc = 0; cc < NB; ++cc) L11[lane * NB + cc] = cc <= lane ? a[cc] : 0.f;
#pragma unroll
            for (int cc = 0; cc < NB; ++cc)
                if (cc == lane) rinv[lane] = 1.0f / a[cc];
            if (!ok && lane == 0) s_ok = 0;
        }
        __syncthreads();
        if (!s_ok) break;
        if (nrem > 0) {
            // panel: L21 = A21 L11^-T, one thread per row
            if (tid < nrem) {
                float *row = A + (j0 + NB + tid) * LD + j0;
                float x[NB];
#pragma unroll
                for (int cc = 0; cc < NB; ++cc) {
                    float s = row[cc];
#pragma unroll
                    for (int k = 0; k < cc; ++k) s = fmaf(-x[k], L11[cc * NB + k], s);
                    x[cc] = s * rinv[cc];
                }
#pragma unroll
                for (int cc = 0; cc < NB; ++cc) row[cc] = x[cc];
            }
            __syncthreads();
            // trailing matrix -= L21 L21^T, 4x4 tiles on interleaved rows (bank-conflict free)
            const int nt = nrem / 4;
            for (int t = tid; t < nt * nt; t += ST_NT) {
                const int ti = t / nt, tj = t - ti * nt;
                float acc[4][4];
#pragma unroll
                for (int a_ = 0; a_ < 4; ++a_)
#pragma unroll
                    for (int b_ = 0; b_ < 4; ++b_) acc[a_][b_] = 0.f;
                const float *Li = A + (j0 + NB + ti) * LD + j0;
                const float *Lj = A + (j0 + NB + tj) * LD + j0;
#pragma unroll 8
                for (int k = 0; k < NB; ++k) {
                    float li[4], lj[4];
#pragma unroll
                    for (int a_ = 0; a_ < 4; ++a_) { li[a_] = Li[a_ * nt * LD + k]; lj[a_] = Lj[a_ * nt * LD + k]; }
#pragma unroll
                    for (int a_ = 0; a_ < 4; ++a_)
#pragma unroll
                        for (int b_ = 0; b_ < 4; ++b_) acc[a_][b_] = fmaf(li[a_], lj[b_], acc[a_][b_]);
                }
#pragma unroll
                for (int a_ = 0; a_ < 4; ++a_)
#pragma unroll
                    for (int b_ = 0; b_ < 4; ++b_)
                        A[(j0 + NB + ti + a_ * nt) * LD + j0 + NB + tj + b_ * nt] -= acc[a_][b_];
            }
            __syncthreads();
        }
    }
    if (tid == 0) p.hflag[g] = s_ok ? HFLAG_SPAN_FULL : 0u;
}

}  // namespace obf
