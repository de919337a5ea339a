// Cache-merging baseline (App. E of the paper, the comparison method "in the spirit of CaM"), per
// (cache, layer, KV head), after the usual selection and gather:
//   (ii)  every deleted position j is routed to the retained position whose key has the largest cosine
//         similarity with K_j (ties: the lowest position; a key of zero norm has similarity 0 with everything),
//   (iii) V*_t = V_t + sum over the j routed to t of A_j / (A_t + eps) * V_j;  keys unchanged.
// Shape-generic CUDA-core kernels (fp32 arithmetic): this is a second workload on the skeleton of the hot path,
// not part of it.
#pragma once

#include "common.cuh"

namespace obf {

constexpr int MG_TILE = 64;                 // deleted positions per block, retained positions per inner tile

template <int D>
constexpr size_t merge_smem_bytes() { return (size_t)(2 * MG_TILE * (D + 1) + 2 * MG_TILE) * sizeof(float); }

// Routing: assign[j] = slot (0 .. k_eff - 1) of the retained position most similar to position j, -1 for retained j.
// grid = (ceil(T_max / MG_TILE), heads_total), 256 threads as 16 x 16: a thread holds 4 positions x 4 slots.
template <typename TIN, int D>
__global__ void __launch_bounds__(256) k_merge_assign(const __grid_constant__ CallDev p)
{
    constexpr int LD = D + 1;
    extern __shared__ float mg_sm[];
    float *Kj = mg_sm, *Kt = Kj + MG_TILE * LD, *inv_j = Kt + MG_TILE * LD, *inv_t = inv_j + MG_TILE;
    int ci, lh;
    locate(p, blockIdx.y, ci, lh);
    const CacheDev &c = p.c[ci];
    const int T = c.T, k = c.k_eff, j0 = blockIdx.x * MG_TILE;
    if (j0 >= T) return;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const TIN *Kh = reinterpret_cast<const TIN *>(c.k) + (size_t)lh * T * D;
    const TIN *Kr = reinterpret_cast<const TIN *>(c.k_out) + (size_t)lh * k * D;      // retained keys, compacted
    const uint8_t *keep = p.keep + c.tok_off + (size_t)lh * T;

    // 1 / norm of the rows of a tile (0 for a zero row or a row past the end): 4 threads per row
    auto inv_norms = [&](const float *rows, float *inv, int n_valid) {
        const int r = tid >> 2, part = tid & 3;
        float s = 0.f;
        for (int e = part; e < D; e += 4) s = fmaf(rows[r * LD + e], rows[r * LD + e], s);
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        if (part == 0) inv[r] = (r < n_valid && s > 0.f) ? rsqrtf(s) : 0.f;
    };
    load_rows_f32<TIN, D, 256>(Kj, LD, Kh, j0, T, MG_TILE);
    __syncthreads();
    inv_norms(Kj, inv_j, T - j0);

    float best[4];
    int best_r[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { best[i] = -INFINITY; best_r[i] = 0; }
    for (int r0 = 0; r0 < k; r0 += MG_TILE) {
        __syncthreads();
        load_rows_f32<TIN, D, 256>(Kt, LD, Kr, r0, k, MG_TILE);
        __syncthreads();
        inv_norms(Kt, inv_t, k - r0);
        __syncthreads();
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) acc[i][jj] = 0.f;
#pragma unroll 4
        for (int e = 0; e < D; ++e) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = Kj[(ty + 16 * i) * LD + e]; b[i] = Kt[(tx + 16 * i) * LD + e]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) acc[i][jj] = fmaf(a[i], b[jj], acc[i][jj]);
        }
        // slots in ascending order within the thread: a later slot wins only with a strictly larger similarity
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int r = r0 + tx + 16 * jj;
                const float cs = acc[i][jj] * inv_j[ty + 16 * i] * inv_t[tx + 16 * jj];
                if (r < k && (cs > best[i] || (cs == best[i] && r < best_r[i]))) { best[i] = cs; best_r[i] = r; }
            }
    }
    // the 16 threads of a position (consecutive lanes) agree on the best slot: larger similarity, then lower slot
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, best[i], o);
            const int orr = __shfl_xor_sync(0xffffffffu, best_r[i], o);
            if (ob > best[i] || (ob == best[i] && orr < best_r[i])) { best[i] = ob; best_r[i] = orr; }
        }
        const int j = j0 + ty + 16 * i;
        if (tx == 0 && j < T) {
            const int a = keep[j] ? -1 : best_r[i];
            p.assign[c.tok_off + (size_t)lh * T + j] = a;
            if (c.assign_out) c.assign_out[(size_t)lh * T + j] = a;
        }
    }
}

// Merge: a warp per retained slot walks the head's routing in ascending position order (a fixed order: the result
// does not depend on scheduling) and adds the routed values in; the fp32 sum is rounded once to the output type.
// grid = (ceil(k_eff_max / 8), heads_total), 256 threads.
template <typename TIN, int D>
__global__ void __launch_bounds__(256) k_merge_apply(const __grid_constant__ CallDev p)
{
    int ci, lh;
    locate(p, blockIdx.y, ci, lh);
    const CacheDev &c = p.c[ci];
    const int T = c.T, k = c.k_eff, lane = threadIdx.x & 31;
    const int r = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (r >= k) return;
    constexpr int PER = D / 32;
    const TIN *Vh = reinterpret_cast<const TIN *>(c.v) + (size_t)lh * T * D;
    const float *A = p.scores + c.tok_off + (size_t)lh * T;
    const int32_t *assign = p.assign + c.tok_off + (size_t)lh * T;
    const float inv_at = 1.f / (A[c.idx_out[(size_t)lh * k + r]] + p.eps);
    float acc[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e) acc[e] = 0.f;
    for (int jb = 0; jb < T; jb += 32) {
        const int j = jb + lane;
        uint32_t hit = __ballot_sync(0xffffffffu, j < T && assign[j] == r);
        while (hit) {
            const int jj = jb + __ffs(hit) - 1;
            hit &= hit - 1;
            const float w = A[jj] * inv_at;
#pragma unroll
            for (int e = 0; e < PER; ++e) acc[e] = fmaf(w, to_f32(Vh[(size_t)jj * D + lane * PER + e]), acc[e]);
        }
    }
    TIN *row = reinterpret_cast<TIN *>(c.v_out) + ((size_t)lh * k + r) * D + lane * PER;
#pragma unroll
    for (int e = 0; e < PER; ++e) {
        const float sum = to_f32(row[e]) + acc[e];
        if constexpr (sizeof(TIN) == 4) row[e] = sum;
        else row[e] = __float2bfloat16_rn(sum);
    }
}

}  // namespace obf
