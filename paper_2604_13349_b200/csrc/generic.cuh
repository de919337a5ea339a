// Shape-generic kernels (any n_q, T; head_dim 64 or 128; fp32 or bf16 inputs).
// All arithmetic is fp32 on the CUDA cores.  These kernels are the only path for
// fp32 caches and for shapes the tuned bf16 path does not cover.
#pragma once

#include "common.cuh"
#include "span_test.cuh"

namespace obf {

constexpr int SC_TILE = 64;           // queries x keys per score tile
constexpr int SC_NT = 256;
constexpr float LOG2E = 1.4426950408889634f;

template <int D>
constexpr size_t score_smem_bytes() { return 2 * SC_TILE * (D + 1) * sizeof(float) + 2 * SC_TILE * sizeof(float)
                                             + 16 * SC_TILE * sizeof(float); }

// 64x64 tile of Q K^T on a 16x16 thread grid: thread (ty,tx) owns rows ty+16i, cols tx+16j.
template <int D>
__device__ __forceinline__ void score_tile(const float *Qs, const float *Ks, int ty, int tx, float (&acc)[4][4])
{
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 4
    for (int c = 0; c < D; ++c) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = Qs[(ty + 16 * i) * (D + 1) + c];
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = Ks[(tx + 16 * j) * (D + 1) + c];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
}

// Step a1, first pass (Eq. 1): for every query row the running maximum of the
// scaled logits (log2 domain) and the softmax normaliser over all T keys.
// grid = (ceil(n_q/64), heads_total).
template <typename TIN, int D>
__global__ void __launch_bounds__(SC_NT) k_score_stats(const __grid_constant__ CallDev p)
{
    extern __shared__ float sm[];
    float *Qs = sm, *Ks = sm + SC_TILE * (D + 1);
    int ci, lh;
    locate(p, blockIdx.y, ci, lh);
    const CacheDev &c = p.c[ci];
    const int T = c.T, n_q = p.n_q;
    const int q0 = blockIdx.x * SC_TILE;
    const TIN *Kh = reinterpret_cast<const TIN *>(c.k) + (size_t)lh * T * D;
    const TIN *Qh = reinterpret_cast<const TIN *>(c.q) + (size_t)lh * n_q * D;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const float sc = LOG2E * rsqrtf((float)D);

    load_rows_f32<TIN, D, SC_NT>(Qs, D + 1, Qh, q0, n_q, SC_TILE);
    float m[4], Z[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { m[i] = -INFINITY; Z[i] = 0.f; }

    for (int j0 = 0; j0 < T; j0 += SC_TILE) {
        __syncthreads();
        load_rows_f32<TIN, D, SC_NT>(Ks, D + 1, Kh, j0, T, SC_TILE);
        __syncthreads();
        float acc[4][4];
        score_tile<D>(Qs, Ks, ty, tx, acc);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float tm = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[i][j] = (j0 + tx + 16 * j < T) ? acc[i][j] * sc : -INFINITY;
                tm = fmaxf(tm, acc[i][j]);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, o));
            const float nm = fmaxf(m[i], tm);
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) s += exp2f(acc[i][j] - nm);
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            Z[i] = Z[i] * exp2f(m[i] - nm) + s;
            m[i] = nm;
        }
    }
    if (tx == 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = q0 + ty + 16 * i;
            if (row < n_q) {
                if (c.lse_extra) fold_lse_extra(c.lse_extra[(size_t)lh * n_q + row], m[i], Z[i]);
                float *st = p.stats + ((size_t)blockIdx.y * n_q + row) * 2;
                st[0] = m[i];
                st[1] = Z[i];
            }
        }
    }
}

// Step a1, second pass (Eq. 1): A_j = sum_t exp(s_tj - m_t) / Z_t for a tile of 64 keys.
// grid = (ceil(T_max/64), heads_total); blocks beyond a cache's T exit.
template <typename TIN, int D>
__global__ void __launch_bounds__(SC_NT) k_score_pool(const __grid_constant__ CallDev p)
{
    extern __shared__ float sm[];
    float *Qs = sm, *Ks = sm + SC_TILE * (D + 1);
    float *rm = Ks + SC_TILE * (D + 1), *rz = rm + SC_TILE, *red = rz + SC_TILE;
    int ci, lh;
    locate(p, blockIdx.y, ci, lh);
    const CacheDev &c = p.c[ci];
    const int T = c.T, n_q = p.n_q;
    const int j0 = blockIdx.x * SC_TILE;
    if (j0 >= T) return;
    const TIN *Kh = reinterpret_cast<const TIN *>(c.k) + (size_t)lh * T * D;
    const TIN *Qh = reinterpret_cast<const TIN *>(c.q) + (size_t)lh * n_q * D;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const float sc = LOG2E * rsqrtf((float)D);

    load_rows_f32<TIN, D, SC_NT>(Ks, D + 1, Kh, j0, T, SC_TILE);
    float colsum[4] = {0.f, 0.f, 0.f, 0.f};
    for (int q0 = 0; q0 < n_q; q0 += SC_TILE) {
        __syncthreads();
        load_rows_f32<TIN, D, SC_NT>(Qs, D + 1, Qh, q0, n_q, SC_TILE);
        if (threadIdx.x < SC_TILE) {
            const int row = q0 + threadIdx.x;
            const float *st = p.stats + ((size_t)blockIdx.y * n_q + min(row, n_q - 1)) * 2;
            rm[threadIdx.x] = row < n_q ? st[0] : 0.f;
            rz[threadIdx.x] = row < n_q ? 1.0f / st[1] : 0.f;
        }
        __syncthreads();
        float acc[4][4];
        score_tile<D>(Qs, Ks, ty, tx, acc);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float mi = rm[ty + 16 * i], zi = rz[ty + 16 * i];
#pragma unroll
            for (int j = 0; j < 4; ++j) colsum[j] += exp2f(acc[i][j] * sc - mi) * zi;
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) red[ty * SC_TILE + tx + 16 * j] = colsum[j];
    __syncthreads();
    if (threadIdx.x < SC_TILE && j0 + threadIdx.x < T) {
        float a = 0.f;
#pragma unroll
        for (int r = 0; r < 16; ++r) a += red[r * SC_TILE + threadIdx.x];
        if (!isfinite(a)) atomicOr(p.status, OBF_DEV_NONFINITE);
        p.scores[c.tok_off + (size_t)lh * T + j0 + threadIdx.x] = a;
        if (c.scores_out) c.scores_out[(size_t)lh * T + j0 + threadIdx.x] = a;
    }
}

// Step a2: radix select of the k_eff largest masses on their order-preserving
// 32-bit keys (4 passes of 8 bits), then one ordered pass that emits the
// retained positions in ascending order; among masses equal to the k_eff-th
// largest, the lowest positions are taken.  One block per (cache, layer, head).
constexpr int SEL_NT = 1024;

__global__ void __launch_bounds__(SEL_NT) k_select(const __grid_constant__ CallDev p)
{
    __shared__ uint32_t hist[256];
    __shared__ uint32_t s_prefix, s_want;
    __shared__ uint32_t wsum[32];
    __shared__ float red[32];
    int ci, lh;
    locate(p, blockIdx.x, ci, lh);
    const CacheDev &c = p.c[ci];
    const int T = c.T, k = c.k_eff;
    // the masses are handled as raw bit patterns so that every pass sees identical keys
    const uint32_t *A = reinterpret_cast<const uint32_t *>(p.scores + c.tok_off + (size_t)lh * T);
    uint8_t *keep = p.keep + c.tok_off + (size_t)lh * T;
    int32_t *idx = c.idx_out + (size_t)lh * k;
    const int tid = threadIdx.x;

    if (tid == 0) { s_prefix = 0u; s_want = (uint32_t)k; }
    uint32_t mask = 0u;
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        for (int j = tid; j < T; j += SEL_NT) {
            const uint32_t u = select_key(p, j, A[j]);
            if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (tid == 0) {
            uint32_t want = s_want, cum = 0u;
            int b = 255;
            for (; b > 0; --b) {
                if (cum + hist[b] >= want) break;
                cum += hist[b];
            }
            s_want = want - cum;
            s_prefix = prefix | ((uint32_t)b << shift);
        }
        mask |= 255u << shift;
        __syncthreads();
    }
    const uint32_t tau = s_prefix;       // key of the k-th largest mass
    const uint32_t want = s_want;        // how many positions with key == tau are retained (>= 1)

    uint32_t run_gt = 0u, run_eq = 0u;
    float sk = 0.f, sd = 0.f, nx = -1.0f;
    for (int base = 0; base < T; base += SEL_NT) {
        const int j = base + tid;
        const bool valid = j < T;
        const uint32_t abits = valid ? A[j] : 0u;
        const float a = __uint_as_float(abits);
        const uint32_t u = valid ? select_key(p, j, abits) : 0u;
        const bool gt = valid && u > tau, eq = valid && u == tau;
        uint32_t v = (gt ? 1u : 0u) | (eq ? 0x10000u : 0u);
        uint32_t inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
            if ((tid & 31) >= o) inc += n;
        }
        if ((tid & 31) == 31) wsum[tid >> 5] = inc;
        __syncthreads();
        if (tid < 32) {
            uint32_t w = wsum[tid], winc = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t n = __shfl_up_sync(0xffffffffu, winc, o);
                if (tid >= o) winc += n;
            }
            wsum[tid] = winc - w;          // exclusive prefix of warp totals
            if (tid == 31) hist[0] = winc; // block total
        }
        __syncthreads();
        const uint32_t excl = inc - v + wsum[tid >> 5];
        const uint32_t gt_before = run_gt + (excl & 0xFFFFu), eq_before = run_eq + (excl >> 16);
        const bool kp = gt || (eq && eq_before < want);
        if (valid) {
            keep[j] = kp ? 1 : 0;
            if (kp) {
                const uint32_t pos = gt_before + min(eq_before, want);
                if (pos < (uint32_t)k) idx[pos] = j;
                else atomicOr(p.status, OBF_DEV_INTERNAL);
                sk += a;
            }
            else { sd += a; nx = fmaxf(nx, a); }
        }
        const uint32_t tot = hist[0];
        run_gt += tot & 0xFFFFu;
        run_eq += tot >> 16;
        __syncthreads();
    }
    const float a_keep = block_sum<SEL_NT>(sk, red);
    const float a_del = block_sum<SEL_NT>(sd, red);
    const float next = block_max<SEL_NT>(nx, red);
    if (tid == 0) {
        float *s = p.sums + (size_t)blockIdx.x * 4;
        s[0] = a_keep; s[1] = a_del; s[2] = tau == 0xFFFFFFFFu ? INFINITY : key_score(tau); s[3] = next;
        if (c.diag) {
            obf_diag_t dg;
            dg.a_keep = a_keep; dg.a_del = a_del; dg.alpha = a_del / (a_keep + p.eps);
            dg.rcr = 0.f; dg.delta_norm = 0.f; dg.kth_score = tau == 0xFFFFFFFFu ? INFINITY : key_score(tau); dg.next_score = next;
            dg.lam_1 = dg.lam_rho = dg.lam_next = 0.f;
            dg.span_rank = -1; dg.rho_eff = 0; dg.status = OBF_DEV_SKIPPED; dg.revr = 0.f; dg.pc = 0.f;
            c.diag[lh] = dg;
        }
    }
}

// Step a2 for heads whose T keys fit in shared memory (the usual case): same result as
// k_select, bit for bit, but the order-preserving keys are read from global memory
// once.  The radix histogram is built with one shared-memory atomic per distinct digit
// and warp; the ordered pass gives every warp a contiguous run of positions, so two
// block-wide barriers suffice.
constexpr int SEL_SMEM_MAX_T = 16384;

// Layerwise selector, first half (Section 3.2, retention rule, second form): the masses of a layer's KV heads
// added up per position, head 0 first.  grid = (ceil(T_max / 256), layers of all caches).
__global__ void __launch_bounds__(256) k_layer_sum(const __grid_constant__ CallDev p)
{
    int ci, lh;
    locate(p, blockIdx.y * p.kv_heads, ci, lh);
    const CacheDev &c = p.c[ci];
    const int j = blockIdx.x * 256 + threadIdx.x;
    if (j >= c.T) return;
    const float *A = p.scores + c.tok_off + (size_t)lh * c.T + j;
    float s = 0.f;
    for (int h = 0; h < p.kv_heads; ++h) s += A[(size_t)h * c.T];
    p.lscores[c.tok_off / p.kv_heads + (size_t)(lh / p.kv_heads) * c.T + j] = s;
}

// With LAYER every head's block selects on its layer's summed masses (the layer's heads repeat the same
// selection side by side rather than one block writing all of them in turn) and then writes the shared
// positions, the keep flags and the demand sums of the head's own masses.
template <int NT, bool LAYER = false>
__global__ void __launch_bounds__(NT) k_select_smem(const __grid_constant__ CallDev p)
{
    extern __shared__ uint32_t sel_keys[];
    __shared__ uint32_t hist[256];
    __shared__ uint32_t s_prefix, s_want;
    constexpr int NW = NT / 32;
    __shared__ uint32_t wtot[32];
    __shared__ float red[32];
    int ci, lh;
    locate(p, blockIdx.x, ci, lh);
    const CacheDev &c = p.c[ci];
    const int T = c.T, k = c.k_eff;
    float *Af = p.scores + c.tok_off + (size_t)lh * T;
    const uint32_t *A = LAYER ? reinterpret_cast<const uint32_t *>(p.lscores + c.tok_off / p.kv_heads + (size_t)(lh / p.kv_heads) * T)
                              : reinterpret_cast<const uint32_t *>(Af);
    uint8_t *keep = p.keep + c.tok_off + (size_t)lh * T;
    int32_t *idx = c.idx_out + (size_t)lh * k;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int j = tid; j < T; j += NT) sel_keys[j] = select_key(p, j, A[j]);
    if (tid == 0) { s_prefix = 0u; s_want = (uint32_t)k; }
    uint32_t mask = 0u;
    const int T_pad = (T + NT - 1) / NT * NT;
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        for (int j = tid; j < T_pad; j += NT) {
            const uint32_t u = j < T ? sel_keys[j] : 0u;
            const bool cand = j < T && (u & mask) == prefix;
            const uint32_t digit = (u >> shift) & 255u;
            // after the first passes few keys are still candidates: most warps have none and skip the counting
            const uint32_t cands = __ballot_sync(0xffffffffu, cand);
            if (cands == 0u) continue;
            if (shift == 24) {
                // top byte (sign and exponent): a handful of values per warp.  Lanes with the same digit add up among
                // themselves first; lanes that are no candidates form one group of their own, which adds nothing
                const uint32_t peers = __match_any_sync(0xffffffffu, cand ? digit : 256u);
                if (cand && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
            } else {
                // mantissa bytes: spread over the bins, so every candidate counts itself (matching 32 different digits
                // costs far more than 32 atomics on different banks); one digit for the whole warp is counted once
                const uint32_t d0 = __shfl_sync(0xffffffffu, digit, __ffs(cands) - 1);
                if (__all_sync(0xffffffffu, !cand || digit == d0)) {
                    if (lane == __ffs(cands) - 1) atomicAdd(&hist[d0], (uint32_t)__popc(cands));
                } else if (cand) {
                    atomicAdd(&hist[digit], 1u);
                }
            }
        }
        __syncthreads();
        if (warp == 0) {
            // lane l owns bins [8l, 8l+8); walk down from the top bin
            uint32_t own = 0u;
#pragma unroll
            for (int b = 0; b < 8; ++b) own += hist[lane * 8 + b];
            uint32_t above = own;                       // inclusive sum over lanes >= this one
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t n = __shfl_down_sync(0xffffffffu, above, o);
                if (lane + o < 32) above += n;
            }
            const uint32_t want = s_want;
            const uint32_t excl = above - own;          // keys in bins above this lane's
            const bool mine = excl < want && want <= above;
            const uint32_t who = __ballot_sync(0xffffffffu, mine);
            // total < want cannot happen (want <= candidates); guard anyway: lowest bin
            const int sel_lane = who ? 31 - __clz(who) : 0;
            if (lane == sel_lane) {
                uint32_t cum = who ? excl : 0u;
                int b = 7;
                for (; b > 0; --b) {
                    const uint32_t h = hist[lane * 8 + b];
                    if (cum + h >= want) break;
                    cum += h;
                }
                s_want = want - cum;
                s_prefix = prefix | ((uint32_t)(lane * 8 + b) << shift);
            }
        }
        mask |= 255u << shift;
        __syncthreads();
    }
    const uint32_t tau = s_prefix;       // key of the k-th largest mass
    const uint32_t want = s_want;        // how many positions with key == tau are retained (>= 1)

    // ordered pass: warp w owns positions [w * seg, (w + 1) * seg)
    const int seg = ((T + NW - 1) / NW + 31) / 32 * 32;
    const int j_begin = warp * seg, j_end = min(T, j_begin + seg);
    uint32_t n_gt = 0u, n_eq = 0u;
    for (int j0 = j_begin; j0 < j_end; j0 += 32) {
        const int j = j0 + lane;
        const uint32_t u = j < j_end ? sel_keys[j] : 0u;
        n_gt += __popc(__ballot_sync(0xffffffffu, j < j_end && u > tau));
        n_eq += __popc(__ballot_sync(0xffffffffu, j < j_end && u == tau));
    }
    if (lane == 0) wtot[warp] = n_gt | (n_eq << 16);
    __syncthreads();
    if (warp == 0) {
        const uint32_t w = lane < NW ? wtot[lane] : 0u;
        uint32_t inc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += n;
        }
        wtot[lane] = inc - w;              // positions before this warp's run: greater (low half), equal (high half)
    }
    __syncthreads();
    uint32_t run_gt = wtot[warp] & 0xFFFFu, run_eq = wtot[warp] >> 16;
    float sk = 0.f, sd = 0.f, nx = -1.0f;
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int j0 = j_begin; j0 < j_end; j0 += 32) {
        const int j = j0 + lane;
        const bool valid = j < j_end;
        const uint32_t u = valid ? sel_keys[j] : 0u;
        const bool gt = valid && u > tau, eq = valid && u == tau;
        const uint32_t m_gt = __ballot_sync(0xffffffffu, gt), m_eq = __ballot_sync(0xffffffffu, eq);
        const uint32_t gt_before = run_gt + __popc(m_gt & lt_mask), eq_before = run_eq + __popc(m_eq & lt_mask);
        const bool kp = gt || (eq && eq_before < want);
        if (LAYER) {
            // what was decided for a position, kept for the per-head sweep below: its output slot, or "deleted"
            if (valid) {
                const uint32_t pos = gt_before + min(eq_before, want);
                if (kp && pos >= (uint32_t)k) atomicOr(p.status, OBF_DEV_INTERNAL);
                sel_keys[j] = (kp && pos < (uint32_t)k) ? pos : 0xFFFFFFFFu;
            }
        } else if (valid) {
            const float a = j < p.n_sink ? __uint_as_float(A[j]) : key_score(u);     // a protected position's key is not its mass
            keep[j] = kp ? 1 : 0;
            if (kp) {
                const uint32_t pos = gt_before + min(eq_before, want);
                if (pos < (uint32_t)k) idx[pos] = j;
                else atomicOr(p.status, OBF_DEV_INTERNAL);
                sk += a;
            } else { sd += a; nx = fmaxf(nx, a); }
        }
        run_gt += __popc(m_gt);
        run_eq += __popc(m_eq);
    }
    if (LAYER) {
        __syncthreads();
        // the largest summed mass among the deleted positions, for the diagnostics
        for (int j = tid; j < T; j += NT)
            if (sel_keys[j] == 0xFFFFFFFFu) nx = fmaxf(nx, __uint_as_float(A[j]));
        const float next = block_max<NT>(nx, red);
        {
            float *Ah = Af;
            uint8_t *keep_h = keep;
            int32_t *idx_h = idx;
            sk = 0.f; sd = 0.f;
            for (int j = tid; j < T; j += NT) {
                const uint32_t pos = sel_keys[j];
                const float a = Ah[j];
                const bool kp = pos != 0xFFFFFFFFu;
                keep_h[j] = kp ? 1 : 0;
                if (kp) {
                    idx_h[pos] = j;
                    sk += a;
                } else {
                    sd += a;
                }
            }
            const float a_keep = block_sum<NT>(sk, red);
            const float a_del = block_sum<NT>(sd, red);
            if (tid == 0) {
                float *sm = p.sums + (size_t)blockIdx.x * 4;
                sm[0] = a_keep; sm[1] = a_del; sm[2] = tau == 0xFFFFFFFFu ? INFINITY : key_score(tau); sm[3] = next;
                if (c.diag) {
                    obf_diag_t dg;
                    dg.a_keep = a_keep; dg.a_del = a_del; dg.alpha = a_del / (a_keep + p.eps);
                    dg.rcr = 0.f; dg.delta_norm = 0.f; dg.kth_score = tau == 0xFFFFFFFFu ? INFINITY : key_score(tau); dg.next_score = next;
                    dg.lam_1 = dg.lam_rho = dg.lam_next = 0.f;
                    dg.span_rank = -1; dg.rho_eff = 0; dg.status = OBF_DEV_SKIPPED; dg.revr = 0.f; dg.pc = 0.f;
                    c.diag[lh] = dg;
                }
            }
        }
        return;
    }
    const float a_keep = block_sum<NT>(sk, red);
    const float a_del = block_sum<NT>(sd, red);
    const float next = block_max<NT>(nx, red);
    if (tid == 0) {
        float *sm = p.sums + (size_t)blockIdx.x * 4;
        sm[0] = a_keep; sm[1] = a_del; sm[2] = tau == 0xFFFFFFFFu ? INFINITY : key_score(tau); sm[3] = next;
        if (c.diag) {
            obf_diag_t dg;
            dg.a_keep = a_keep; dg.a_del = a_del; dg.alpha = a_del / (a_keep + p.eps);
            dg.rcr = 0.f; dg.delta_norm = 0.f; dg.kth_score = tau == 0xFFFFFFFFu ? INFINITY : key_score(tau); dg.next_score = next;
            dg.lam_1 = dg.lam_rho = dg.lam_next = 0.f;
            dg.span_rank = -1; dg.rho_eff = 0; dg.status = OBF_DEV_SKIPPED; dg.revr = 0.f; dg.pc = 0.f;
            c.diag[lh] = dg;
        }
    }
}

// Step a3: K_out = K[idx], V_out = V[idx] as 16-byte vectors.  A block copies GATHER_ROWS
// retained rows of one head; every thread moves one vector of four different rows of K
// and of V, with all eight loads in flight before the first store.
// grid = (ceil(k_eff_max / GATHER_ROWS), heads_total).
constexpr int GATHER_ROWS = 64;

// WHICH: 3 = keys and values, 1 = values only, 2 = keys only (the keys are needed by nothing that follows in
// the call, so their copy can run beside the later kernels).
template <int ROW_BYTES, int WHICH = 3>
__global__ void __launch_bounds__(256) k_gather(const __grid_constant__ CallDev p)
{
    constexpr int CH = ROW_BYTES / 16;             // vectors per row
    constexpr int RPP = 256 / CH;                  // rows per pass of the block
    constexpr int PASSES = GATHER_ROWS / RPP;
    int ci, lh;
    locate(p, blockIdx.y, ci, lh);
    const CacheDev &c = p.c[ci];
    const int r0 = blockIdx.x * GATHER_ROWS;
    if (r0 >= c.k_eff) return;
    const int ch = threadIdx.x % CH, rr = threadIdx.x / CH;
    const char *kb = reinterpret_cast<const char *>(c.k) + (size_t)lh * c.T * ROW_BYTES;
    const char *vb = reinterpret_cast<const char *>(c.v) + (size_t)lh * c.T * ROW_BYTES;
    char *ko = reinterpret_cast<char *>(c.k_out) + (size_t)lh * c.k_eff * ROW_BYTES;
    char *vo = reinterpret_cast<char *>(c.v_out) + (size_t)lh * c.k_eff * ROW_BYTES;
    const int32_t *idx = c.idx_out + (size_t)lh * c.k_eff;
#pragma unroll 1
    for (int p0 = 0; p0 < PASSES; p0 += 4) {
        int r[4], j[4];
        uint4 kv[4], vv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            r[u] = r0 + (p0 + u) * RPP + rr;
            j[u] = -1;
            if (p0 + u < PASSES && r[u] < c.k_eff) {
                j[u] = idx[r[u]];
                if ((unsigned)j[u] >= (unsigned)c.T) {     // never dereference a position outside the cache
                    atomicOr(p.status, OBF_DEV_INTERNAL);
                    j[u] = -1;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (j[u] >= 0) {
                if (WHICH & 2) kv[u] = *reinterpret_cast<const uint4 *>(kb + (size_t)j[u] * ROW_BYTES + ch * 16);
                if (WHICH & 1) vv[u] = *reinterpret_cast<const uint4 *>(vb + (size_t)j[u] * ROW_BYTES + ch * 16);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (j[u] >= 0) {
                if (WHICH & 2) *reinterpret_cast<uint4 *>(ko + (size_t)r[u] * ROW_BYTES + ch * 16) = kv[u];
                if (WHICH & 1) *reinterpret_cast<uint4 *>(vo + (size_t)r[u] * ROW_BYTES + ch * 16) = vv[u];
            }
        }
    }
}

// Post-hoc int8 quantisation of the compacted relay (App. E): symmetric, one fp32 scale per row of K_out and of
// V_out, scale = max|x| / 127, code = round-half-even(x / scale).
// A row is read as 16-byte vectors, one per thread, so a row of ROW_BYTES takes ROW_BYTES / 16 neighbouring lanes
// (they find the row's maximum with that many shuffle steps); a thread has QR_ROWS rows of both arrays in flight.
// grid = (ceil(k_eff_max / QR_BLOCK_ROWS), heads_total), 256 threads.
constexpr int QR_ROWS = 4;

// 16 bytes of a row as floats: 8 bf16 or 4 fp32 values.
template <typename TIN>
__device__ __forceinline__ void unpack16(const uint4 &v, float (&x)[16 / sizeof(TIN)])
{
    if constexpr (sizeof(TIN) == 4) {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    } else {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) { x[2 * e] = __uint_as_float(w[e] << 16); x[2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u); }
    }
}

template <typename TIN, int D>
constexpr int qr_block_rows() { return 256 / (D * (int)sizeof(TIN) / 16) * QR_ROWS; }

template <typename TIN, int D>
__global__ void __launch_bounds__(256) k_quantize_rows(const __grid_constant__ CallDev p)
{
    constexpr int CH = D * (int)sizeof(TIN) / 16;                      // threads per row
    constexpr int EPT = 16 / (int)sizeof(TIN);                         // elements per thread
    constexpr int RPP = 256 / CH;                                      // rows per pass of the block
    static_assert(CH >= 1 && CH <= 32 && (CH & (CH - 1)) == 0, "a row's threads are a power-of-two run of lanes");
    int ci, lh;
    locate(p, blockIdx.y, ci, lh);
    const CacheDev &c = p.c[ci];
    if (!c.k_q8) return;
    const int ch = threadIdx.x % CH, rr = threadIdx.x / CH;
    const int r0 = blockIdx.x * (RPP * QR_ROWS) + rr;                  // this thread's rows: r0 + i RPP
    if (blockIdx.x * (RPP * QR_ROWS) >= c.k_eff) return;
    const size_t row0 = (size_t)lh * c.k_eff;
    uint4 raw[2][QR_ROWS];
#pragma unroll
    for (int which = 0; which < 2; ++which)
#pragma unroll
        for (int i = 0; i < QR_ROWS; ++i) {
            const int r = r0 + i * RPP;
            const TIN *src = reinterpret_cast<const TIN *>(which ? c.v_out : c.k_out) + (row0 + r) * D + ch * EPT;
            raw[which][i] = r < c.k_eff ? *reinterpret_cast<const uint4 *>(src) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
    for (int which = 0; which < 2; ++which)
#pragma unroll
        for (int i = 0; i < QR_ROWS; ++i) {
            const int r = r0 + i * RPP;
            float x[EPT];
            unpack16<TIN>(raw[which][i], x);
            float amax = 0.f;
#pragma unroll
            for (int e = 0; e < EPT; ++e) amax = fmaxf(amax, fabsf(x[e]));
            // (every lane takes part: rows past the end hold zeros)
#pragma unroll
            for (int o = CH / 2; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            const float scale = amax / 127.0f;
            // code = rint(x / scale) with the quotient rounded to fp32 first.  x * (1 / scale) is within 2.3e-5 of that
            // quotient (|x / scale| <= 127), so both round to the same integer unless the product is that close to a
            // half-integer: only then (a few elements in ten thousand) the quotient itself is formed.
            const float rcp = scale > 0.f ? 1.0f / scale : 0.f;
            uint32_t packed[EPT / 4];
#pragma unroll
            for (int w = 0; w < EPT / 4; ++w) packed[w] = 0u;
#pragma unroll
            for (int e = 0; e < EPT; ++e) {
                const float pr = x[e] * rcp;
                float v = rintf(pr);
                if (fabsf(fabsf(pr - v) - 0.5f) < 2.44140625e-4f && scale > 0.f) v = rintf(x[e] / scale);
                v = fminf(fmaxf(v, -127.f), 127.f);
                packed[e / 4] |= (uint32_t)(uint8_t)(int8_t)v << (8 * (e % 4));
            }
            if (r < c.k_eff) {
                // EPT bytes per thread (the arrays are 8-byte aligned: validated on the host)
                int8_t *dst = (which ? c.v_q8 : c.k_q8) + (row0 + r) * D + ch * EPT;
                if constexpr (EPT == 8) *reinterpret_cast<uint2 *>(dst) = make_uint2(packed[0], packed[1]);
                else *reinterpret_cast<uint32_t *>(dst) = packed[0];
                if (ch == 0) (which ? c.v_scale : c.k_scale)[row0 + r] = scale;
            }
        }
}

// Diagnostics only (projection cosine): s = sum of the deleted value rows of a head, for heads with a
// diagnostics record.  grid = (token splits, heads_total), 256 threads = 256 / D row groups x D columns.
template <typename TIN, int D>
__global__ void __launch_bounds__(256) k_vsum(const __grid_constant__ CallDev p)
{
    __shared__ float part[256];
    int ci, lh;
    locate(p, blockIdx.y, ci, lh);
    const CacheDev &c = p.c[ci];
    if (!c.diag || c.T <= c.k_eff) return;
    constexpr int RG = 256 / D > 0 ? 256 / D : 1;         // row groups
    const int col = threadIdx.x % D, rg = threadIdx.x / D;
    const int per = (c.T + gridDim.x - 1) / gridDim.x;
    const int r0 = blockIdx.x * per, r1 = min(c.T, r0 + per);
    const TIN *V = reinterpret_cast<const TIN *>(c.v) + (size_t)lh * c.T * D;
    const uint8_t *keep = p.keep + c.tok_off + (size_t)lh * c.T;
    float acc = 0.f;
    if (rg < RG)
        for (int r = r0 + rg; r < r1; r += RG)
            if (!keep[r]) acc += to_f32(V[(size_t)r * D + col]);
    part[threadIdx.x] = acc;
    __syncthreads();
    if (threadIdx.x < D) {
        float t = 0.f;
        for (int g2 = 0; g2 < RG; ++g2) t += part[g2 * D + threadIdx.x];
        atomicAdd(&p.svec[(size_t)blockIdx.y * D + threadIdx.x], t);
    }
}

// Step a4, streaming part: one pass over V accumulating, per head and token
// split, the Gram matrix of the deleted rows (for R^T R = P G_del P, App. H), the
// Gram matrix of the retained rows (only when k_eff >= d, for the span test) and
// u = sum over deleted j of A_j v_j (for r_bar, Eq. 4).
// grid = (splits, heads_total), 256 threads as a 16x16 grid of (D/16)^2 register tiles.
constexpr int GR_ROWS = 32;

template <typename TIN, int D>
__global__ void __launch_bounds__(256) k_gram(const __grid_constant__ CallDev p)
{
    constexpr int NV = D / 64;               // float4 groups per thread along each axis
    constexpr int MT = 4 * NV;
    __shared__ __align__(16) float Vs[GR_ROWS * D];
    __shared__ float As[GR_ROWS];
    __shared__ int Fs[GR_ROWS];
    int ci, lh;
    locate(p, blockIdx.y, ci, lh);
    const CacheDev &c = p.c[ci];
    const int T = c.T;
    const bool need_k = c.k_eff >= D;
    const TIN *Vh = reinterpret_cast<const TIN *>(c.v) + (size_t)lh * T * D;
    const float *A = p.scores + c.tok_off + (size_t)lh * T;
    const uint8_t *keep = p.keep + c.tok_off + (size_t)lh * T;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;

    const int tiles = (T + GR_ROWS - 1) / GR_ROWS;
    const int per = (tiles + p.splits - 1) / p.splits;
    const int t_begin = blockIdx.x * per, t_end = min(tiles, t_begin + per);

    float accD[MT][MT], accK[MT][MT];
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < MT; ++j) { accD[i][j] = 0.f; accK[i][j] = 0.f; }
    float u = 0.f;

    for (int t = t_begin; t < t_end; ++t) {
        const int r0 = t * GR_ROWS;
        __syncthreads();
        load_rows_f32<TIN, D, 256>(Vs, D, Vh, r0, T, GR_ROWS);
        if (threadIdx.x < GR_ROWS) {
            const int j = r0 + threadIdx.x;
            Fs[threadIdx.x] = j < T ? (int)keep[j] : 2;
            As[threadIdx.x] = j < T ? A[j] : 0.f;
        }
        __syncthreads();
#pragma unroll 1
        for (int r = 0; r < GR_ROWS; ++r) {
            const int f = Fs[r];
            if (f == 2) break;
            if (f == 1 && !need_k) continue;
            float a[MT], b[MT];
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const float4 fa = *reinterpret_cast<const float4 *>(&Vs[r * D + v * 64 + ty * 4]);
                const float4 fb = *reinterpret_cast<const float4 *>(&Vs[r * D + v * 64 + tx * 4]);
                a[4 * v] = fa.x; a[4 * v + 1] = fa.y; a[4 * v + 2] = fa.z; a[4 * v + 3] = fa.w;
                b[4 * v] = fb.x; b[4 * v + 1] = fb.y; b[4 * v + 2] = fb.z; b[4 * v + 3] = fb.w;
            }
            if (f == 0) {
#pragma unroll
                for (int i = 0; i < MT; ++i)
#pragma unroll
                    for (int j = 0; j < MT; ++j) accD[i][j] = fmaf(a[i], b[j], accD[i][j]);
                if (threadIdx.x < D) u = fmaf(As[r], Vs[r * D + threadIdx.x], u);
            } else {
#pragma unroll
                for (int i = 0; i < MT; ++i)
#pragma unroll
                    for (int j = 0; j < MT; ++j) accK[i][j] = fmaf(a[i], b[j], accK[i][j]);
            }
        }
    }
    const size_t slot = (size_t)blockIdx.y * p.splits + blockIdx.x;
    float *gd = p.gram_d + slot * D * D, *gk = p.gram_k + slot * D * D;
#pragma unroll
    for (int i = 0; i < MT; ++i) {
        const int row = (i / 4) * 64 + ty * 4 + (i & 3);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int col = v * 64 + tx * 4;
            *reinterpret_cast<float4 *>(&gd[row * D + col]) =
                make_float4(accD[i][4 * v], accD[i][4 * v + 1], accD[i][4 * v + 2], accD[i][4 * v + 3]);
            if (need_k)
                *reinterpret_cast<float4 *>(&gk[row * D + col]) =
                    make_float4(accK[i][4 * v], accK[i][4 * v + 1], accK[i][4 * v + 2], accK[i][4 * v + 3]);
        }
    }
    if (threadIdx.x < D) p.uvec[slot * D + threadIdx.x] = u;
}

}  // namespace obf
