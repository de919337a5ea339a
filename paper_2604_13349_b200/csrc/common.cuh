// Shared device-side definitions for the relay-compression kernels.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "obf.h"

namespace obf {

// One cache as the kernels see it (device pointers, resolved sizes).
// Per-head flags in the workspace (hflag).
constexpr uint32_t HFLAG_INJECT = 1u;      // delta != 0: the injection kernel has work for this head
constexpr uint32_t HFLAG_SPAN_FULL = 2u;   // span(V_keep) = R^d

struct CacheDev {
    const void *k, *v, *q;
    void *k_out, *v_out;
    int32_t *idx_out;
    obf_diag_t *diag;
    float *scores_out;
    float *delta_out;
    const float *lse_extra;   // out-of-prompt softmax mass per query row (natural log), or null
    int8_t *k_q8, *v_q8;      // optional int8 copy of the compacted relay, with one scale per row
    float *k_scale, *v_scale;
    int32_t *assign_out;      // optional: routing of the cache-merging baseline
    int32_t T, k_eff;
    int32_t head_base;        // global id of this cache's first (layer, kv head)
    int32_t nsub_del;         // tuned path: 128-token tiles of V per head (ceil(T / 128))
    int32_t pad0_;
    int32_t pad_;
    size_t tok_off;           // offset of this cache in the per-token workspace arrays (elements)
    long long sub_base;       // tuned path: index of this cache's first tile in the tile sequence of the pass over V
    // tuned score kernel: a head's chunks are worked on by a team of slots, heads are dealt in rounds
    int32_t sc_team;          // chunks (= blocks) per head
    int32_t sc_hpr;           // heads per round
    int32_t sc_round_base;    // first round of this cache
    int32_t pad2_;
    size_t sc_part_off;       // offset of this cache in sc_part, in (max, sum) pairs
};

// Tensor maps of a tuned-path kernel, two per cache, passed as a kernel parameter
// (score kernel: a = K, b = Q; Gram kernel: a = V).
struct TcMaps {
    CUtensorMap a[OBF_MAX_CACHES];
    CUtensorMap b[OBF_MAX_CACHES];
};

// Everything one call needs, passed by value as a __grid_constant__ kernel parameter.
struct CallDev {
    CacheDev c[OBF_MAX_CACHES];
    int32_t n_caches;
    int32_t heads_per_cache;  // layers * kv_heads
    int32_t heads_total;
    int32_t n_q;              // G * n_obs query rows pooled into one KV head
    int32_t d;
    int32_t rank;
    int32_t splits;           // token splits of the Gram pass (shape-generic path)
    int32_t gram_slots;       // partial Gram matrices stored per head (stride of gram_d / gram_k / uvec)
    int32_t tc_per;           // tuned path: tiles per block of the pass over V (0: shape-generic path)
    int32_t pad1_;
    long long tc_total_sub;   // tuned path: tiles in the tile sequence of the pass over V
    int32_t gram_all;         // 1: gram_d and uvec run over all rows of V (tuned path), 0: over the deleted rows only
    int32_t u_levels;         // partial u vectors per partial Gram matrix: U_LEVELS with gram_all, else 1
    int32_t alg_rows;         // dense algebra: basis rows any head of the call can have, min(largest k_eff, d)
    int32_t sc_nq;            // tuned score kernel: query rows of its tiles (0: shape-generic score kernels)
    int32_t sc_subs;          // 128-key tiles per chunk
    int32_t sc_rounds;        // rounds of the persistent score kernel
    int32_t sc_qt;            // tuned score kernel: 128-row query tiles per head (1 or 2)
    float *sc_part;           // per (head, chunk, query of 128): chunk maximum and normaliser
    float *sc_head;           // per (head, query of 128): one 64-bit word, low = M + log2(Z) over all keys, high = 1 when valid
    uint32_t *sc_cnt;         // per head: chunks that have published
    float eps;
    int32_t kv_heads;         // KV heads per layer
    int32_t layerwise;        // 1: one retained set per layer (masses summed over its KV heads)
    int32_t n_sink;           // protected prefix: the first n_sink positions are retained besides the budget
    int32_t fast_iters;       // > 0: that many Gram subspace iterations instead of the exact eigenvectors
    int32_t merge;            // 1: cache-merging baseline after the gather (App. E)
    int32_t attn_inject;      // 1: delta is added in proportion to the retained positions' masses (App. D.2)
    int32_t skip_full;        // 1: the span test has run before the pass over V, which skips the heads it found full
    int32_t debug_drop_publish;   // test hook: the score kernel never publishes a head's normalisers, so the wait for them runs out
    unsigned long long wait_limit_ns;   // after this long a device-side wait gives up and reports OBF_DEV_TIMEOUT
    // workspace
    uint32_t *status;
    float *scores;            // [sum heads*T] attention mass (Eq. 1)
    float *scores2;           // tuned score kernel with two query tiles: masses of the second tile, added into `scores` afterwards
    float *lscores;           // layerwise selector: [sum layers*T] masses summed over a layer's KV heads (cache offset tok_off / kv_heads)
    uint8_t *keep;            // [sum heads*T] 1 = retained
    int32_t *assign;          // [sum heads*T] cache-merging baseline: slot a deleted position is routed to, -1 = retained
    float *stats;             // [heads_total, n_q, 2] softmax row max (log2 domain) and normaliser
    float *sums;              // [heads_total, 4] a_keep, a_del, kth, next
    float *gram_d;            // [heads_total, gram_slots, d, d] partial Gram of the deleted (gram_all: of all) values
    float *gram_k;            // [heads_total, gram_slots, d, d] partial Gram of retained values (shape-generic path only)
    float *uvec;              // [heads_total, gram_slots, u_levels, d] partial sum_j A_j v_j over the same rows as gram_d, per mass level
    float *delta;             // [heads_total, d]
    float *svec;              // [heads_total, d] sum of the deleted value rows (only filled when diagnostics are asked for)
    uint32_t *hflag;          // [heads_total] bit0: delta != 0 -> inject
};

__device__ __forceinline__ void locate(const CallDev &p, int g, int &ci, int &lh)
{
    ci = 0;
#pragma unroll 1
    for (int i = 1; i < p.n_caches; ++i)
        if (g >= p.c[i].head_base) ci = i;
    lh = g - p.c[ci].head_base;
}

// How many partial Gram matrices (and u vectors) the streaming pass left for one head.
// Shape-generic path: one per token split (for the deleted and for the retained rows alike).  Tuned path: the
// tile sequence of the pass over V is cut into runs of tc_per tiles, one run per block; a head's tiles land in
// consecutive blocks, each of which stores one partial.
__device__ __forceinline__ int gram_partial_count(const CallDev &p, const CacheDev &c, int lh)
{
    if (p.tc_per == 0) return p.splits;
    const long long len = c.nsub_del;
    const long long start = c.sub_base + (long long)lh * len;
    return (int)((start + len - 1) / p.tc_per - start / p.tc_per) + 1;
}

// The sum u = sum_j A_j v_j over ALL rows is kept apart by the magnitude of the mass, one partial sum per level
// (factors of 64 between the levels): the retained rows, whose masses are the largest, are subtracted from it
// afterwards, and a few large terms must not cost the many small ones their low bits.
constexpr int U_LEVELS = 5;
__device__ __forceinline__ int u_level(float a)
{
    const int e = (int)((__float_as_uint(a) >> 23) & 0xFFu);       // biased exponent; masses are not negative
    return e >= 127 ? 4 : e >= 121 ? 3 : e >= 115 ? 2 : e >= 109 ? 1 : 0;
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

// Loads `rows_tile` rows of D elements starting at row0 of a [n_rows, D] matrix
// into shared memory as float with row stride `ld`; rows >= n_rows become zero.
template <typename TIN, int D, int NT>
__device__ __forceinline__ void load_rows_f32(float *dst, int ld, const TIN *src, int row0, int n_rows,
                                              int rows_tile)
{
    constexpr int VEC = 16 / sizeof(TIN);        // elements per 16-byte vector
    constexpr int CH = D / VEC;                  // vectors per row
    for (int i = threadIdx.x; i < rows_tile * CH; i += NT) {
        int r = i / CH, ch = i - r * CH;
        float *o = dst + r * ld + ch * VEC;
        if (row0 + r < n_rows) {
            const uint4 raw = *reinterpret_cast<const uint4 *>(src + (size_t)(row0 + r) * D + ch * VEC);
            if constexpr (sizeof(TIN) == 4) {
                o[0] = __uint_as_float(raw.x); o[1] = __uint_as_float(raw.y);
                o[2] = __uint_as_float(raw.z); o[3] = __uint_as_float(raw.w);
            } else {
                const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    o[2 * e] = __uint_as_float(w[e] << 16);
                    o[2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
                }
            }
        } else {
#pragma unroll
            for (int e = 0; e < VEC; ++e) o[e] = 0.f;
        }
    }
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Block-wide sum in a fixed order (deterministic).  `red` holds >= 32 floats.
template <int NT>
__device__ __forceinline__ float block_sum(float v, float *red)
{
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
    if (threadIdx.x < 32) {
        t = threadIdx.x < NT / 32 ? red[threadIdx.x] : 0.f;
        t = warp_sum(t);
        if (threadIdx.x == 0) red[0] = t;
    }
    __syncthreads();
    t = red[0];
    __syncthreads();
    return t;
}

template <int NT>
__device__ __forceinline__ float block_max(float v, float *red)
{
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t;
    if (threadIdx.x < 32) {
        t = threadIdx.x < NT / 32 ? red[threadIdx.x] : -INFINITY;
        t = warp_max(t);
        if (threadIdx.x == 0) red[0] = t;
    }
    __syncthreads();
    t = red[0];
    __syncthreads();
    return t;
}

// Folds the out-of-prompt softmax mass of a query row (natural log of the sum of exp(logit) over the keys outside
// the prompt) into the row's running maximum m (log2 domain) and normaliser z = sum_j 2^(x_j - m).
__device__ __forceinline__ void fold_lse_extra(float lse_natural, float &m, float &z)
{
    const float L = lse_natural * 1.4426950408889634f;
    if (L > -INFINITY) {
        const float mn = fmaxf(m, L);
        z = (m > -INFINITY ? z * exp2f(m - mn) : 0.f) + exp2f(L - mn);
        m = mn;
    }
}

// Order-preserving map from a float's bits to an unsigned key (larger float -> larger key).
__device__ __forceinline__ uint32_t score_key_bits(uint32_t u)
{
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Selection key of position j: protected positions sort above every mass.
__device__ __forceinline__ uint32_t select_key(const CallDev &p, int j, uint32_t mass_bits)
{
    return j < p.n_sink ? 0xFFFFFFFFu : score_key_bits(mass_bits);
}

__device__ __forceinline__ float key_score(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

}  // namespace obf
