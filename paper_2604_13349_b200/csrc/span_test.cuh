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
// below it by one thread per row, the lower triangle of the trailing matrix by
// 8x4 register tiles.
// Result: bit 1 of hflag[head].
//
// FROM_ROWS (tuned path: bf16, head_dim 128): G_keep is not read from the workspace but formed here from the
// first 256 gathered rows of the head (any subset of the retained rows that spans R^d certifies the test), with
// warp-level mma (bf16 products are exact, fp32 accumulation) while the rows sit in the memory the matrix then takes.
#pragma once

#include "common.cuh"

namespace obf {

constexpr int ST_NT = 256;
constexpr float CHOL_PIVOT_TOL = 1e-3f;

template <int D>
constexpr size_t span_smem_bytes() { return (size_t)(D * (D + 1) + 32 * 33 + 32 + D + 64 + 256 + 3) * sizeof(float); }

constexpr int SPAN_ROWS = 256;          // retained rows that enter G_keep with FROM_ROWS

template <int D, bool FROM_ROWS = false>
__global__ void __launch_bounds__(ST_NT, 3) k_span_test(const __grid_constant__ CallDev p)
{
    constexpr int LD = D + 1, NB = 32, L11_LD = NB + 1;
    extern __shared__ float st_sm[];
    float *A = st_sm;                  // D x LD, lower triangle is what counts
    float *L11 = A + D * LD;           // 32 x 32 factor of the current diagonal block (16-byte aligned)
    float *rinv = L11 + NB * L11_LD;   // 32 reciprocals of its diagonal
    float *d0 = rinv + NB;             // D original diagonal entries
    float *pvt = d0 + D;               // 8 x 8 pivot block of the diagonal block (16-byte aligned)
    float *lrow = pvt + 64;            // 32 x 8: the newest 8 columns of the factor, row by row
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
    if constexpr (FROM_ROWS) {
        static_assert(D == 128, "the row-based Gram matrix is written for head_dim 128");
        static_assert(SPAN_ROWS * D * 2 <= D * (D + 1) * 4, "the rows are staged in the matrix's memory");
        // X: the first rows of the head's compacted values, [SPAN_ROWS][128] bf16, rows past the end zero; the
        // 16-byte chunks of a row are permuted by the row number so that 8 x 8 matrix loads hit distinct banks
        uint8_t *X = reinterpret_cast<uint8_t *>(A);
        const int n_rows = c.k_eff < SPAN_ROWS ? c.k_eff : SPAN_ROWS;
        const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(c.v_out) + (size_t)lh * c.k_eff * D);
        // eight 16-byte loads in flight per thread
#pragma unroll 1
        for (int i0 = tid; i0 < SPAN_ROWS * 16; i0 += 8 * ST_NT) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = i0 + u * ST_NT, r = i >> 4, ch = i & 15;
                v[u] = r < n_rows ? __ldg(src + (size_t)r * 16 + ch) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = i0 + u * ST_NT, r = i >> 4, ch = i & 15;
                *reinterpret_cast<uint4 *>(X + r * 256 + (((ch & 8) | ((ch ^ r) & 7)) << 4)) = v[u];
            }
        }
        __syncthreads();
        // G = X^T X: warp w owns rows [16 w, 16 w + 16) of G, in two halves of 64 columns (m16n8k16, A = X^T and
        // B = X both read with transposing 8 x 8 loads from the row-major X)
        const uint32_t xbase = (uint32_t)__cvta_generic_to_shared(X);
        const int mi = lane >> 3, rr = lane & 7;
        float acc[2][8][4];
#pragma unroll
        for (int hf = 0; hf < 2; ++hf)
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[hf][nt][e] = 0.f;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
#pragma unroll 1
            for (int k0 = 0; k0 < SPAN_ROWS; k0 += 16) {
                uint32_t a[4];
                {
                    // matrices: (tokens k0.., dims i0..), (tokens k0.., dims i0 + 8..), (tokens k0 + 8.., dims i0..), (k0 + 8.., i0 + 8..)
                    const int tok = k0 + (mi >> 1) * 8 + rr, chn = (16 * warp + (mi & 1) * 8) >> 3;
                    const uint32_t addr = xbase + tok * 256 + (((chn & 8) | ((chn ^ tok) & 7)) << 4);
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]) : "r"(addr));
                }
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    // two 8-column tiles at once: (tokens k0.., dims n0..), (k0 + 8.., n0..), (k0.., n0 + 8..), (k0 + 8.., n0 + 8..)
                    const int n0 = hf * 64 + np * 16;
                    if (n0 > 16 * warp) continue;              // right of the diagonal: only the lower triangle is ever read
                    const int tok = k0 + (mi & 1) * 8 + rr, chn = (n0 + (mi >> 1) * 8) >> 3;
                    const uint32_t addr = xbase + tok * 256 + (((chn & 8) | ((chn ^ tok) & 7)) << 4);
                    uint32_t b[4];
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3]) : "r"(addr));
#pragma unroll
                    for (int t2 = 0; t2 < 2; ++t2) {
                        float *d4 = acc[hf][2 * np + t2];
                        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                     : "+f"(d4[0]), "+f"(d4[1]), "+f"(d4[2]), "+f"(d4[3])
                                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[2 * t2]), "r"(b[2 * t2 + 1]));
                    }
                }
            }
        }
        __syncthreads();                                   // every warp is done reading X: the matrix takes its place
#pragma unroll
        for (int hf = 0; hf < 2; ++hf)
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                const int row = 16 * warp + (lane >> 2), col = hf * 64 + nt * 8 + 2 * (lane & 3);
                if (hf * 64 + (nt >> 1) * 16 > 16 * warp) continue;
                A[row * LD + col] = acc[hf][nt][0];
                A[row * LD + col + 1] = acc[hf][nt][1];
                A[(row + 8) * LD + col] = acc[hf][nt][2];
                A[(row + 8) * LD + col + 1] = acc[hf][nt][3];
            }
    } else {
        const int n_part = gram_partial_count(p, c, lh);           // shape-generic path: one per token split
        const float *parts = p.gram_k + (size_t)g * p.gram_slots * D * D;
        for (int e0 = tid; e0 < D * D / 4; e0 += 4 * ST_NT) {
            float4 acc[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int sp = 0; sp < n_part; ++sp) {
                float4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int e4 = e0 + u * ST_NT;
                    // only the lower triangle is ever read: skip the 4-element groups right of the diagonal
                    const bool lower = e4 < D * D / 4 && (e4 * 4) % D <= (e4 * 4) / D;
                    v[u] = lower ? *reinterpret_cast<const float4 *>(parts + (size_t)sp * D * D + e4 * 4)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) { acc[u].x += v[u].x; acc[u].y += v[u].y; acc[u].z += v[u].z; acc[u].w += v[u].w; }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int e4 = e0 + u * ST_NT;
                if (e4 < D * D / 4) {
                    const int r = (e4 * 4) / D, cc = (e4 * 4) % D;
                    float *o = A + r * LD + cc;
                    o[0] = acc[u].x; o[1] = acc[u].y; o[2] = acc[u].z; o[3] = acc[u].w;
                }
            }
        }
    }
    if (tid == 0) s_ok = 1;
    __syncthreads();
    if (tid < D) d0[tid] = A[tid * LD + tid];
    __syncthreads();

#pragma unroll 1
    for (int j0 = 0; j0 < D; j0 += NB) {
        const int nrem = D - j0 - NB;                      // rows below the diagonal block
        if (warp == 0) {
            // Lane i owns row i of the diagonal block in registers.  The block is factorised 8 columns at a
            // time: the 8 x 8 pivot block is published through shared memory and factorised by EVERY lane
            // in registers (redundantly, so no lane waits for another inside those 8 columns); each lane
            // then solves its own 8 entries and the lanes exchange them once for the rank-8 update.
            float a[NB];
#pragma unroll
            for (int cc = 0; cc < NB; ++cc) a[cc] = cc <= lane ? A[(j0 + lane) * LD + j0 + cc] : 0.f;
            bool ok = true;
#pragma unroll
            for (int c0 = 0; c0 < NB; c0 += 8) {
                // rows c0..c0+7 publish their entries of the pivot block (lower triangle is what counts)
                if (lane >= c0 && lane < c0 + 8) {
                    float4 *dst = reinterpret_cast<float4 *>(pvt + (lane - c0) * 8);
                    dst[0] = make_float4(a[c0], a[c0 + 1], a[c0 + 2], a[c0 + 3]);
                    dst[1] = make_float4(a[c0 + 4], a[c0 + 5], a[c0 + 6], a[c0 + 7]);
                }
                __syncwarp();
                float l8[8][8];                                // factor of the pivot block, row-major, lower
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    const float4 v0 = *reinterpret_cast<const float4 *>(pvt + r * 8);
                    const float4 v1 = *reinterpret_cast<const float4 *>(pvt + r * 8 + 4);
                    l8[r][0] = v0.x; l8[r][1] = v0.y; l8[r][2] = v0.z; l8[r][3] = v0.w;
                    l8[r][4] = v1.x; l8[r][5] = v1.y; l8[r][6] = v1.z; l8[r][7] = v1.w;
                }
                float inv8[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float piv = l8[k][k];
                    ok = ok && (piv > CHOL_PIVOT_TOL * d0[j0 + c0 + k]) && (piv > 0.f);
                    asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(inv8[k]) : "f"(piv));
                    if (lane == 0) rinv[c0 + k] = inv8[k];
#pragma unroll
                    for (int r = k; r < 8; ++r) l8[r][k] *= inv8[k];
#pragma unroll
                    for (int c2 = k + 1; c2 < 8; ++c2)
#pragma unroll
                        for (int r = c2; r < 8; ++r) l8[r][c2] = fmaf(-l8[r][k], l8[c2][k], l8[r][c2]);
                }
                // this lane's 8 entries of L: forward substitution against the pivot block's factor
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    float v = a[c0 + k];
#pragma unroll
                    for (int mm = 0; mm < k; ++mm) v = fmaf(-a[c0 + mm], l8[k][mm], v);
                    a[c0 + k] = v * inv8[k];
                }
                if (c0 + 8 < NB) {
                    // exchange the 8 entries of every row, then the rank-8 update of the columns to the right
                    float4 *dst = reinterpret_cast<float4 *>(lrow + lane * 8);
                    dst[0] = make_float4(a[c0], a[c0 + 1], a[c0 + 2], a[c0 + 3]);
                    dst[1] = make_float4(a[c0 + 4], a[c0 + 5], a[c0 + 6], a[c0 + 7]);
                    __syncwarp();
#pragma unroll
                    for (int cc = c0 + 8; cc < NB; ++cc) {
                        const float4 w0 = *reinterpret_cast<const float4 *>(lrow + cc * 8);
                        const float4 w1 = *reinterpret_cast<const float4 *>(lrow + cc * 8 + 4);
                        float v = a[cc];
                        v = fmaf(-a[c0], w0.x, v); v = fmaf(-a[c0 + 1], w0.y, v);
                        v = fmaf(-a[c0 + 2], w0.z, v); v = fmaf(-a[c0 + 3], w0.w, v);
                        v = fmaf(-a[c0 + 4], w1.x, v); v = fmaf(-a[c0 + 5], w1.y, v);
                        v = fmaf(-a[c0 + 6], w1.z, v); v = fmaf(-a[c0 + 7], w1.w, v);
                        a[cc] = v;
                    }
                    __syncwarp();
                }
            }
#pragma unroll
            for (int cc = 0; cc < NB; ++cc) L11[lane * L11_LD + cc] = cc <= lane ? a[cc] : 0.f;
            if (!ok && lane == 0) s_ok = 0;
        }
        __syncthreads();
        if (!s_ok) break;
        if (nrem > 0) {
            // panel: L21 = A21 L11^-T, one thread per row; once x_c is known every later entry of the
            // row is updated independently, so the dependency chain is 32 steps long, not 496
            if (tid < nrem) {
                float *row = A + (j0 + NB + tid) * LD + j0;
                float x[NB];
#pragma unroll
                for (int cc = 0; cc < NB; ++cc) x[cc] = row[cc];
#pragma unroll
                for (int cc = 0; cc < NB; ++cc) {
                    x[cc] *= rinv[cc];
#pragma unroll
                    for (int c2 = cc + 1; c2 < NB; ++c2) x[c2] = fmaf(-x[cc], L11[c2 * L11_LD + cc], x[c2]);
                }
#pragma unroll
                for (int cc = 0; cc < NB; ++cc) row[cc] = x[cc];
            }
            __syncthreads();
            // trailing matrix -= L21 L21^T.  Only the lower triangle is ever read again: the trailing matrix is
            // cut into 32 x 32 blocks and a thread updates an 8 x 4 register tile of a block on or below the
            // diagonal (rows r0 + 4a.., columns c0 + 8b.. interleaved inside the block, bank-conflict free).
            const int nb = nrem / NB;                      // blocks per side
            const int n_blk = nb * (nb + 1) / 2;           // blocks on or below the diagonal
            for (int t = tid; t < n_blk * 32; t += ST_NT) {
                const int blk = t >> 5, sub = t & 31;      // 32 threads per block: 4 row groups x 8 column groups
                int bi = 0, rem = blk;
                while (rem > bi) { rem -= bi + 1; ++bi; }  // block row bi, block column rem (rem <= bi)
                const int bj = rem;
                const int ri = sub >> 3, cj = sub & 7;     // rows ri + 4a (a < 8), columns cj + 8b (b < 4)
                float acc[8][4];
#pragma unroll
                for (int a_ = 0; a_ < 8; ++a_)
#pragma unroll
                    for (int b_ = 0; b_ < 4; ++b_) acc[a_][b_] = 0.f;
                const float *Li = A + (j0 + NB + bi * NB + ri) * LD + j0;
                const float *Lj = A + (j0 + NB + bj * NB + cj) * LD + j0;
#pragma unroll 4
                for (int k = 0; k < NB; ++k) {
                    float li[8], lj[4];
#pragma unroll
                    for (int a_ = 0; a_ < 8; ++a_) li[a_] = Li[a_ * 4 * LD + k];
#pragma unroll
                    for (int b_ = 0; b_ < 4; ++b_) lj[b_] = Lj[b_ * 8 * LD + k];
#pragma unroll
                    for (int a_ = 0; a_ < 8; ++a_)
#pragma unroll
                        for (int b_ = 0; b_ < 4; ++b_) acc[a_][b_] = fmaf(li[a_], lj[b_], acc[a_][b_]);
                }
#pragma unroll
                for (int a_ = 0; a_ < 8; ++a_)
#pragma unroll
                    for (int b_ = 0; b_ < 4; ++b_)
                        A[(j0 + NB + bi * NB + ri + 4 * a_) * LD + j0 + NB + bj * NB + cj + 8 * b_] -= acc[a_][b_];
            }
            __syncthreads();
        }
    }
    if (tid == 0) p.hflag[g] = s_ok ? HFLAG_SPAN_FULL : 0u;
}

}  // namespace obf
