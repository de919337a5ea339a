// Tuned attention-mass kernel (step a1, Eq. 1 with the softmax of App. L.1) for bf16
// caches with head_dim 128: K is read from HBM exactly once and the logits never
// leave the chip.
//
//   A_j = sum_t softmax_j(q_t . K_j / sqrt(d)),  t over the n_q query rows of the KV head.
//
// A head's T keys are cut into chunks of CH = SUBS * 128 keys.  One chunk is handled
// by one "slot": a group of four warps that owns half of the block's tensor memory
// (256 columns).  For its chunk a slot
//   1. gets S^T = K_chunk Q^T from the tensor cores (tcgen05.mma, 128 keys on the
//      lanes, the NQ = n_q rounded up to 32 queries on the columns, fp32);
//   2. takes the column maxima m_loc[t] over its keys, turns the logits into
//      p = exp2(s * log2(e)/sqrt(d) - m_loc[t]) IN PLACE in tensor memory and sums
//      Z_loc[t] = sum_j p;
//   3. publishes (m_loc, Z_loc); the last slot of the head to arrive combines all
//      chunks into (M_t, Z_t) and raises the head's flag;
//   4. once the flag is up: f_t = exp2(m_loc[t] - M_t) / Z_t and
//      A_j = sum_t f_t p_tj, one key per thread, written to the workspace.
// All slots of a head (its team) run at the same time: the kernel is persistent, a
// block carries two slots, and work is dealt in rounds in which every slot takes
// (head, chunk) = (round * heads_per_round + slot / team, slot % team).  A block's
// two slots belong to different heads, so one computes while the other waits for
// its team.  Waits are bounded (tc_common.cuh).
//
// Block = 10 warps: warp 0 TMA producer (Q per slot, K tiles through a 4-stage ring),
// warp 1 MMA issuer, warps 2..5 slot 0, warps 6..9 slot 1.
#pragma once

#include "tc_common.cuh"

namespace obf {

constexpr int ST_STAGES = 4;
constexpr int ST_TILE_BYTES = 128 * 128 * 2;        // one 128-key tile of K
constexpr int ST_THREADS = 320;
constexpr int ST_MAX_NQ = 160;                      // query columns the shared-memory budget allows
constexpr float ST_LOG2E = 1.4426950408889634f;

__host__ __device__ constexpr size_t score_tc_smem_bytes(int nq_pad)
{
    return 1024 + 2 * (size_t)nq_pad * 256 + (size_t)ST_STAGES * ST_TILE_BYTES +
           2 * (4 * 256 + 256 + 256) * sizeof(float) + 64;
}

struct ScoreItem {
    int cache, lh, chunk, nsv;     // nsv: 128-key tiles of the chunk that hold at least one key
};

// Work of slot `slot` in round `r`; false when the slot idles in that round.
__device__ __forceinline__ bool score_item(const CallDev &p, int r, int slot, ScoreItem &it)
{
    int ci = 0;
#pragma unroll 1
    for (int i = 1; i < p.n_caches; ++i)
        if (r >= p.c[i].sc_round_base) ci = i;
    const CacheDev &c = p.c[ci];
    const int hi = slot / c.sc_team;
    if (hi >= c.sc_hpr) return false;
    const int lh = (r - c.sc_round_base) * c.sc_hpr + hi;
    if (lh >= p.heads_per_cache) return false;
    it.cache = ci;
    it.lh = lh;
    it.chunk = slot - hi * c.sc_team;
    const int left = c.T - it.chunk * p.sc_subs * 128;
    const int tiles = (left + 127) / 128;
    it.nsv = tiles < p.sc_subs ? tiles : p.sc_subs;
    return true;
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Across the 32 lanes of a warp: lane l ends with op over all lanes of element l.
template <bool IS_MAX>
__device__ __forceinline__ float warp_reduce_scatter(float (&v)[32], int lane)
{
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        const bool up = (lane & o) != 0;
#pragma unroll
        for (int i = 0; i < o; ++i) {
            const float send = up ? v[i] : v[i + o];
            const float keep = up ? v[i + o] : v[i];
            const float recv = __shfl_xor_sync(0xffffffffu, send, o);
            v[i] = IS_MAX ? fmaxf(keep, recv) : keep + recv;
        }
    }
    return v[0];
}

__global__ void __launch_bounds__(ST_THREADS, 1) k_score_tc(const __grid_constant__ CallDev p, const __grid_constant__ TcMaps tm)
{
    extern __shared__ uint8_t st_smem_raw[];
    const int NQ = p.sc_nq, SUBS = p.sc_subs, CH = SUBS * 128;
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(st_smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *q_s = base;                                           // 2 x [NQ x 128] bf16, two 64-column halves each
    uint8_t *ring = q_s + 2 * (size_t)NQ * 256;                    // ST_STAGES x 32 KiB
    float *scratch = reinterpret_cast<float *>(ring + ST_STAGES * ST_TILE_BYTES);
    __shared__ uint64_t bar_q_full[2], bar_mma_done[2], bar_tmem_free[2], bar_full[ST_STAGES], bar_empty[ST_STAGES];
    __shared__ uint32_t s_tmem, s_abort, s_last[2];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_blocks = gridDim.x;
    tc::WaitCtx wc{&s_abort, p.status};

    if (tid == 0) {
        s_abort = 0u;
        for (int w = 0; w < 2; ++w) {
            tc::mbar_init(&bar_q_full[w], 1);
            tc::mbar_init(&bar_mma_done[w], 1);
            tc::mbar_init(&bar_tmem_free[w], 4);
        }
        for (int s = 0; s < ST_STAGES; ++s) { tc::mbar_init(&bar_full[s], 1); tc::mbar_init(&bar_empty[s], 1); }
        tc::mbar_init_fence();
    }
    if (warp == 1) tc::tmem_alloc(&s_tmem, 512);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = s_tmem;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint32_t it = 0, nq[2] = {0u, 0u};
            bool dead = false;
            for (int r = 0; r < p.sc_rounds && !dead; ++r) {
                for (int w = 0; w < 2 && !dead; ++w) {
                    ScoreItem item;
                    if (!score_item(p, r, w * n_blocks + (int)blockIdx.x, item)) continue;
                    // the slot's Q buffer is free once the MMAs of its previous chunk are done
                    if (nq[w] > 0 && !tc::mbar_wait(&bar_mma_done[w], (nq[w] - 1) & 1u, wc)) { dead = true; break; }
                    const uint32_t qdst = tc::smem_u32(q_s + (size_t)w * NQ * 256);
                    tc::mbar_expect_tx(&bar_q_full[w], (uint32_t)NQ * 256u);
                    tc::tma_load_3d(qdst, &tm.b[item.cache], &bar_q_full[w], 0, 0, item.lh);
                    tc::tma_load_3d(qdst + (uint32_t)NQ * 128u, &tm.b[item.cache], &bar_q_full[w], 64, 0, item.lh);
                    for (int sub = 0; sub < item.nsv; ++sub, ++it) {
                        const int s = it % ST_STAGES;
                        if (!tc::mbar_wait(&bar_empty[s], ((it / ST_STAGES) & 1u) ^ 1u, wc)) { dead = true; break; }
                        tc::mbar_expect_tx(&bar_full[s], ST_TILE_BYTES);
                        const uint32_t dst = tc::smem_u32(ring + s * ST_TILE_BYTES);
                        const int row0 = item.chunk * CH + sub * 128;
                        tc::tma_load_3d(dst, &tm.a[item.cache], &bar_full[s], 0, row0, item.lh);
                        tc::tma_load_3d(dst + ST_TILE_BYTES / 2, &tm.a[item.cache], &bar_full[s], 64, row0, item.lh);
                    }
                    ++nq[w];
                }
            }
            // nothing this thread started may still be in flight when the block exits
            for (uint32_t j = it > (uint32_t)ST_STAGES ? it - ST_STAGES : 0u; j < it; ++j)
                tc::mbar_wait(&bar_full[j % ST_STAGES], (j / ST_STAGES) & 1u, wc);
            for (int w = 0; w < 2; ++w)
                if (nq[w] > 0) tc::mbar_wait(&bar_q_full[w], (nq[w] - 1) & 1u, wc);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_bf16(128, (uint32_t)NQ, 0, 0);
            uint32_t it = 0, nq[2] = {0u, 0u};
            bool dead = false;
            for (int r = 0; r < p.sc_rounds && !dead; ++r) {
                for (int w = 0; w < 2 && !dead; ++w) {
                    ScoreItem item;
                    if (!score_item(p, r, w * n_blocks + (int)blockIdx.x, item)) continue;
                    if (!tc::mbar_wait(&bar_q_full[w], nq[w] & 1u, wc)) { dead = true; break; }
                    if (!tc::mbar_wait(&bar_tmem_free[w], (nq[w] & 1u) ^ 1u, wc)) { dead = true; break; }
                    tc::tc_fence_after();
                    const uint32_t qaddr = tc::smem_u32(q_s + (size_t)w * NQ * 256);
                    for (int sub = 0; sub < item.nsv; ++sub, ++it) {
                        const int s = it % ST_STAGES;
                        if (!tc::mbar_wait(&bar_full[s], (it / ST_STAGES) & 1u, wc)) { dead = true; break; }
                        tc::tc_fence_after();
                        const uint32_t kaddr = tc::smem_u32(ring + s * ST_TILE_BYTES);
                        const uint32_t acc = tmem + (uint32_t)(w * 256 + sub * NQ);
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            // 16 channels per instruction: 32 bytes along the swizzled row, second half after 4 steps
                            const uint64_t da = tc::smem_desc_sw128(kaddr + (kk >> 2) * (ST_TILE_BYTES / 2) + (kk & 3) * 32, 16, 1024);
                            const uint64_t db = tc::smem_desc_sw128(qaddr + (kk >> 2) * ((uint32_t)NQ * 128u) + (kk & 3) * 32, 16, 1024);
                            tc::umma_bf16(acc, da, db, idesc, kk > 0 ? 1u : 0u);
                        }
                        tc::umma_commit(&bar_empty[s]);
                    }
                    tc::umma_commit(&bar_mma_done[w]);
                    ++nq[w];
                }
            }
        }
    } else {
        // ---------------- slots: softmax statistics, team hand-shake, pooling ----------------
        const int w = (warp - 2) >> 2;                 // slot of this block
        const int wl = (warp - 2) & 3;                 // warp within the slot
        const int q = warp & 3;                        // tensor-memory lane quarter this warp may touch
        const int row = q * 32 + lane;                 // key row inside a 128-key tile
        const int wt = wl * 32 + lane;                 // thread within the slot
        const int bar_id = 1 + w;
        float *s_part = scratch + w * (4 * 256 + 256 + 256);   // [4 warps][256] per-warp column statistics
        float *s_ml = s_part + 4 * 256;                // [256] chunk maxima (log2 domain)
        float *s_ff = s_ml + 256;                      // [256] pooling weights f_t
        const uint32_t tbase = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(w * 256);
        const float sc = ST_LOG2E * rsqrtf(128.0f);
        const int n_cb = NQ / 32;
        uint32_t n_done = 0;

        for (int r = 0; r < p.sc_rounds; ++r) {
            ScoreItem item;
            if (!score_item(p, r, w * n_blocks + (int)blockIdx.x, item)) continue;
            const CacheDev &c = p.c[item.cache];
            const int g = c.head_base + item.lh;
            const int T = c.T, team = c.sc_team;
            const int j0 = item.chunk * CH;
            tc::mbar_wait(&bar_mma_done[w], n_done & 1u, wc);
            tc::tc_fence_after();

            // ---- column maxima over the chunk's keys ----
            for (int cb = 0; cb < n_cb; ++cb) {
                float m[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) m[i] = -INFINITY;
                for (int sub = 0; sub < item.nsv; ++sub) {
                    uint32_t rr[32];
                    tc::tmem_ld32(tbase + (uint32_t)(sub * NQ + cb * 32), rr);
                    tc::tmem_ld_wait();
                    if (j0 + sub * 128 + row < T) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) m[i] = fmaxf(m[i], __uint_as_float(rr[i]));
                    }
                }
                s_part[wl * 256 + cb * 32 + lane] = warp_reduce_scatter<true>(m, lane);
            }
            tc::named_barrier(bar_id, 128);
            for (int t = wt; t < NQ; t += 128)
                s_ml[t] = fmaxf(fmaxf(s_part[t], s_part[256 + t]), fmaxf(s_part[512 + t], s_part[768 + t])) * sc;
            tc::named_barrier(bar_id, 128);

            // ---- p = exp2(s * sc - m_loc) in place, column sums ----
            for (int cb = 0; cb < n_cb; ++cb) {
                float ml[32], z[32];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 v = *reinterpret_cast<const float4 *>(&s_ml[cb * 32 + i * 4]);
                    ml[4 * i] = v.x; ml[4 * i + 1] = v.y; ml[4 * i + 2] = v.z; ml[4 * i + 3] = v.w;
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) z[i] = 0.f;
                for (int sub = 0; sub < item.nsv; ++sub) {
                    uint32_t rr[32];
                    const uint32_t ta = tbase + (uint32_t)(sub * NQ + cb * 32);
                    tc::tmem_ld32(ta, rr);
                    tc::tmem_ld_wait();
                    const bool kv = j0 + sub * 128 + row < T;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float pe = kv ? ex2_approx(fmaf(__uint_as_float(rr[i]), sc, -ml[i])) : 0.f;
                        z[i] += pe;
                        rr[i] = __float_as_uint(pe);
                    }
                    tc::tmem_st32(ta, rr);
                }
                tc::tmem_st_wait();
                s_part[wl * 256 + cb * 32 + lane] = warp_reduce_scatter<false>(z, lane);
            }
            tc::named_barrier(bar_id, 128);

            // ---- publish the chunk's statistics; the last slot of the head combines them ----
            float2 *part = reinterpret_cast<float2 *>(p.sc_part) + (c.sc_part_off + ((size_t)item.lh * team + item.chunk) * NQ);
            float2 *head_st = reinterpret_cast<float2 *>(p.sc_head) + (size_t)g * NQ;
            for (int t = wt; t < p.n_q; t += 128) {
                const float z_loc = (s_part[t] + s_part[256 + t]) + (s_part[512 + t] + s_part[768 + t]);
                __stcg(&part[t], make_float2(s_ml[t], z_loc));
            }
            __threadfence();
            tc::named_barrier(bar_id, 128);
            if (wt == 0) {
                const uint32_t old = atomicAdd(&p.sc_cnt[g], 1u);
                s_last[w] = (old == (uint32_t)(team - 1)) ? 1u : 0u;
                __threadfence();
            }
            tc::named_barrier(bar_id, 128);
            if (s_last[w]) {
                for (int t = wt; t < p.n_q; t += 128) {
                    const float2 *hp = reinterpret_cast<const float2 *>(p.sc_part) + (c.sc_part_off + (size_t)item.lh * team * NQ);
                    float M = -INFINITY;
                    for (int ch = 0; ch < team; ++ch) M = fmaxf(M, __ldcg(&hp[(size_t)ch * NQ + t]).x);
                    float Z = 0.f;
                    for (int ch = 0; ch < team; ++ch) {
                        const float2 v = __ldcg(&hp[(size_t)ch * NQ + t]);
                        Z += v.y * ex2_approx(v.x - M);
                    }
                    if (!(Z > 0.f) || !isfinite(Z) || !isfinite(M)) atomicOr(p.status, OBF_DEV_NONFINITE);
                    __stcg(&head_st[t], make_float2(M, Z));
                }
                __threadfence();
                tc::named_barrier(bar_id, 128);
                if (wt == 0) atomicExch(&p.sc_flag[g], 1u);
            }
            if (wt == 0) {
                // bounded wait for the head's flag
                const uint64_t t0 = tc::global_ns();
                volatile uint32_t *flag = p.sc_flag + g;
                while (*flag == 0u) {
                    if (s_abort) break;
                    if (tc::global_ns() - t0 > tc::WAIT_LIMIT_NS) {
                        s_abort = 1u;
                        atomicOr(p.status, OBF_DEV_TIMEOUT);
                        break;
                    }
                }
                __threadfence();
            }
            tc::named_barrier(bar_id, 128);
            for (int t = wt; t < NQ; t += 128) {
                float f = 0.f;
                if (t < p.n_q) {
                    const float2 hs = __ldcg(&head_st[t]);
                    f = ex2_approx(s_ml[t] - hs.x) / hs.y;
                }
                s_ff[t] = f;
            }
            tc::named_barrier(bar_id, 128);

            // ---- A_j = sum_t f_t p_tj ----
            float *A = p.scores + c.tok_off + (size_t)item.lh * T;
            for (int sub = 0; sub < item.nsv; ++sub) {
                float acc = 0.f;
                for (int cb = 0; cb < n_cb; ++cb) {
                    uint32_t rr[32];
                    tc::tmem_ld32(tbase + (uint32_t)(sub * NQ + cb * 32), rr);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 f = *reinterpret_cast<const float4 *>(&s_ff[cb * 32 + i * 4]);
                        acc = fmaf(__uint_as_float(rr[4 * i]), f.x, acc);
                        acc = fmaf(__uint_as_float(rr[4 * i + 1]), f.y, acc);
                        acc = fmaf(__uint_as_float(rr[4 * i + 2]), f.z, acc);
                        acc = fmaf(__uint_as_float(rr[4 * i + 3]), f.w, acc);
                    }
                }
                const int j = j0 + sub * 128 + row;
                if (j < T) {
                    if (!isfinite(acc)) atomicOr(p.status, OBF_DEV_NONFINITE);
                    A[j] = acc;
                    if (c.scores_out) c.scores_out[(size_t)item.lh * T + j] = acc;
                }
            }
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&bar_tmem_free[w]);
            ++n_done;
        }
    }

    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem, 512);
}

}  // namespace obf
