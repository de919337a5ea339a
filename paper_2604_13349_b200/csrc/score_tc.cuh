// Tuned attention-mass kernel (step a1, Eq. 1 with the softmax of App. L.1) for bf16
// caches with head_dim 128 and up to 256 query rows per KV head (above 128 rows a head is
// worked on as two items of up to 128 rows whose masses are added afterwards).
//
//   A_j = sum_t softmax_j(q_t . K_j / sqrt(d)),  t over the n_q query rows of the KV head.
//
// The softmax normaliser of a query is needed before any key's mass can be pooled, so
// the keys are visited twice.  K comes from HBM once: the second visit follows the first
// closely enough to be served by the L2 cache.
//
//   pass A (statistics)  S = Q K_tile^T on the tensor cores with the QUERIES on the
//       tensor-memory lanes: a thread owns one query and keeps its running maximum m_t
//       and sum z_t = sum_j exp2(s_tj c - m_t) (c = log2(e)/sqrt(d)) over the block's
//       chunk of keys; nothing crosses lanes.  Per (head, chunk) the block publishes
//       (m_t, z_t); the last block of the head to arrive folds all chunks into
//       M'_t = M_t + log2(Z_t) and publishes that.
//   pass B (pooling)     S^T = K_tile Q^T with the KEYS on the lanes: a thread owns one
//       key and sums exp2(s_tj c - M'_t) = softmax_j over all queries of the tile;
//       again nothing crosses lanes, and a key's mass is complete in one thread.
//
// A head's T keys are cut into chunks of 4 tiles of 128 keys; a head's chunks are worked
// on by a team of blocks in the same round.  Rounds are dealt as
// (head, chunk) = (round * heads_per_round + block / team, block % team), and a block
// runs A(i), B(i - ST_LAG) for i = 0, 1, ..: a chunk's second visit comes one round after
// its first, when every block of its team has published (a longer lag pushes the chunk out
// of the L2 cache before its second visit).
// The wait for M' is bounded like every other wait (tc_common.cuh).
//
// Block = 20 warps: warp 0 TMA producer (K tiles through a 4-stage ring, asked into L2 one
// round ahead; Q of a pass is loaded while the pass before it runs, into the buffer of its
// kind: one for the statistics passes, one for the pooling passes, which read Q again),
// warps 1 and 19 MMA issuers, alternate tiles (accumulators in a 4-deep ring of 128 tensor-memory columns),
// warps 2..17 consumers in four groups of four, group g taking the tiles with index g (mod 4), so
// that every scheduler holds one warp of each group and the four are at different points of
// their tiles: a warp owns the 32 tensor-memory lanes of its quarter and walks the 128 columns
// of its tile in four pieces of 32 (load, wait, exponentials); the tile goes back to the MMA
// issuers when its last piece is in registers.  A key's pooled mass is complete in one thread.
// Measured alternatives that were slower: two groups (two warps per scheduler), the load of a
// piece in flight behind the arithmetic of the piece before it (the unrolled code was slower in
// every form), a share of the exponentials evaluated as a polynomial on the FMA pipe (the
// special-function unit is busy about half of the time: it is not what the warps wait for).
// Warp 18 is the messenger: it publishes the chunk statistics the consumers leave in shared
// memory, folds a head's chunks when its block is the last to arrive, and then fetches the
// head's M' for the pooling pass a round later, so that the consumers never wait for global memory.
#pragma once

#include "tc_common.cuh"

namespace obf {

constexpr int ST_TILES = 4;                         // 128-key tiles per chunk
constexpr int ST_CHUNK = ST_TILES * 128;
constexpr int ST_STAGES = 4;                        // K tiles in flight in shared memory
constexpr int ST_TBUF = 4;                          // accumulator tiles in tensor memory
constexpr int ST_LAG = 1;                           // rounds between a chunk's statistics pass and its pooling pass
constexpr int ST_TILE_BYTES = 128 * 128 * 2;
constexpr int ST_GROUPS = 4;                        // consumer groups of four warps, one accumulator tile each
constexpr int ST_CONSUMERS = ST_GROUPS * 128;
constexpr int ST_THREADS = 64 + ST_CONSUMERS + 64;
constexpr int ST_MAX_NQ = 256;                      // two query tiles of 128 rows
constexpr float ST_LOG2E = 1.4426950408889634f;
constexpr size_t ST_SMEM_BYTES = 1024 + (size_t)2 * ST_TILE_BYTES + (size_t)ST_STAGES * ST_TILE_BYTES +
                                 (2 * 2 * ST_GROUPS * 128 + 2 * 128) * sizeof(float) + 64;
static_assert(ST_STAGES == ST_TBUF, "a ring stage is released by the accumulator barrier of the same index");

struct ScoreItem {
    int r, cache, lh, chunk, nt;   // r: round; lh: KV head in the cache; nt: tiles of the chunk that hold at least one key
    int lv, qt;                    // lv = lh * query tiles + qt: the (head, query tile) pair; qt: which 128 query rows
};

// What a block needs of a cache to find its work of a round (kept in shared memory).
struct ScoreTab {
    int round_base, hpr, hi, chunk, T;   // hi, chunk: this block's head slot and chunk inside a round of the cache
};

// Work of this block in round `r`; false when the block idles in that round.
__device__ __forceinline__ bool score_item(const CallDev &p, const ScoreTab *tab, int r, ScoreItem &it)
{
    int ci = 0;
#pragma unroll 1
    for (int i = 1; i < p.n_caches; ++i)
        if (r >= tab[i].round_base) ci = i;
    const ScoreTab c = tab[ci];
    if (c.hi >= c.hpr) return false;
    // a head with more than 128 query rows is dealt as two items, one per 128 rows: softmax rows are independent,
    // so the head's masses are the sum of the two items' masses
    const int lv = (r - c.round_base) * c.hpr + c.hi;
    if (lv >= p.heads_per_cache * p.sc_qt) return false;
    it.r = r;
    it.cache = ci;
    it.lv = lv;
    it.lh = p.sc_qt == 2 ? lv >> 1 : lv;
    it.qt = p.sc_qt == 2 ? lv & 1 : 0;
    it.chunk = c.chunk;
    const int tiles = (c.T - c.chunk * ST_CHUNK + 127) >> 7;
    it.nt = tiles < ST_TILES ? tiles : ST_TILES;
    return true;
}

// The passes of a block in the order it runs them: A(i), B(i - ST_LAG) for i = 0, 1, ..
struct PassIter {
    int i = 0, ph = 0;
};

// Next pass with work for this block: kind 0 = statistics, 1 = pooling.
__device__ __forceinline__ bool next_pass(const CallDev &p, const ScoreTab *tab, int R, PassIter &s, ScoreItem &item, int &kind)
{
    while (s.i < R + ST_LAG) {
        const int ph = s.ph, r = ph == 0 ? s.i : s.i - ST_LAG;
        if (ph == 0) s.ph = 1;
        else { s.ph = 0; ++s.i; }
        if (r < 0 || r >= R) continue;
        if (!score_item(p, tab, r, item)) continue;
        kind = ph;
        return true;
    }
    return false;
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float lg2_approx(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t atom_add_acq_rel_gpu(uint32_t *addr, uint32_t v)
{
    uint32_t old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(addr), "r"(v) : "memory");
    return old;
}

__device__ __forceinline__ void st_relaxed_gpu_u64(unsigned long long *addr, unsigned long long v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(addr), "l"(v) : "memory");
}

__device__ __forceinline__ unsigned long long ld_relaxed_gpu_u64(const unsigned long long *addr)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(addr) : "memory");
    return v;
}

// Pass A on one thread's 32 logits of a piece: running maximum m (log2 domain) and sum z of
// exp2(s c - m) of one query.  With MASKED only the first n_valid columns are keys.
template <bool MASKED>
__device__ __forceinline__ void stats_update(uint32_t (&rr)[32], int n_valid, float sc, float &m, float &z)
{
    if (MASKED) {
#pragma unroll
        for (int e = 0; e < 32; ++e)
            if (e >= n_valid) rr[e] = 0xff800000u;                                     // -inf: no such key
    }
    float t0 = __uint_as_float(rr[0]), t1 = __uint_as_float(rr[1]);
    float t2 = __uint_as_float(rr[2]), t3 = __uint_as_float(rr[3]);
#pragma unroll
    for (int e = 4; e < 32; e += 4) {
        t0 = fmaxf(t0, __uint_as_float(rr[e]));
        t1 = fmaxf(t1, __uint_as_float(rr[e + 1]));
        t2 = fmaxf(t2, __uint_as_float(rr[e + 2]));
        t3 = fmaxf(t3, __uint_as_float(rr[e + 3]));
    }
    const float mn = fmaxf(m, fmaxf(fmaxf(t0, t1), fmaxf(t2, t3)) * sc);
    if (mn > -INFINITY) {
        float z0 = 0.f, z1 = 0.f, z2 = 0.f, z3 = 0.f;
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
            z0 += ex2_approx(fmaf(__uint_as_float(rr[e]), sc, -mn));
            z1 += ex2_approx(fmaf(__uint_as_float(rr[e + 1]), sc, -mn));
            z2 += ex2_approx(fmaf(__uint_as_float(rr[e + 2]), sc, -mn));
            z3 += ex2_approx(fmaf(__uint_as_float(rr[e + 3]), sc, -mn));
        }
        z = z * ex2_approx(m - mn) + ((z0 + z1) + (z2 + z3));
        m = mn;
    }
}

// Pass B on one thread's 32 logits of a piece: the softmax weights of one key under 32 queries, added up.
// mp: M'_t of those queries (shared memory, the same address for every lane).
__device__ __forceinline__ float pool_piece(const uint32_t (&rr)[32], const float *mp, float sc)
{
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        const float4 v = *reinterpret_cast<const float4 *>(mp + e);
        a0 += ex2_approx(fmaf(__uint_as_float(rr[e]), sc, -v.x));
        a1 += ex2_approx(fmaf(__uint_as_float(rr[e + 1]), sc, -v.y));
        a2 += ex2_approx(fmaf(__uint_as_float(rr[e + 2]), sc, -v.z));
        a3 += ex2_approx(fmaf(__uint_as_float(rr[e + 3]), sc, -v.w));
    }
    return (a0 + a1) + (a2 + a3);
}

__global__ void __launch_bounds__(ST_THREADS, 1) k_score_tc(const __grid_constant__ CallDev p, const __grid_constant__ TcMaps tm)
{
    extern __shared__ uint8_t st_smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(st_smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *q_s = base;                                           // 2 x [128 x 128] bf16: Q of a statistics pass, Q of a pooling pass; two 64-column halves each
    uint8_t *ring = q_s + 2 * ST_TILE_BYTES;                       // ST_STAGES x 32 KiB
    float *s_m = reinterpret_cast<float *>(ring + ST_STAGES * ST_TILE_BYTES);   // [2][tile of the chunk][128 queries] tile maxima
    float *s_z = s_m + 2 * ST_GROUPS * 128;                        // [2][tile of the chunk][128 queries] tile sums
    float *s_mp = s_z + 2 * ST_GROUPS * 128;                       // [2][128] M'_t of the head being pooled
    __shared__ uint64_t bar_q_full[2], bar_q_free[2], bar_full[ST_STAGES];
    __shared__ uint64_t bar_t_full[ST_TBUF], bar_t_empty[ST_TBUF];
    __shared__ uint64_t bar_st_ready[2], bar_st_free[2], bar_mp_ready[2], bar_mp_free[2];
    __shared__ ScoreTab s_tab[OBF_MAX_CACHES];
    __shared__ uint32_t s_tmem, s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int R = p.sc_rounds;
    tc::WaitCtx wc{&s_abort, p.status, p.wait_limit_ns};

    if (tid == 0) {
        s_abort = 0u;
        for (int b = 0; b < 2; ++b) { tc::mbar_init(&bar_q_full[b], 1); tc::mbar_init(&bar_q_free[b], 2); }
        for (int s = 0; s < ST_STAGES; ++s) tc::mbar_init(&bar_full[s], 1);
        for (int s = 0; s < ST_TBUF; ++s) {
            tc::mbar_init(&bar_t_full[s], 1);
            tc::mbar_init(&bar_t_empty[s], 4);                  // the four warps of the group that owns the tile
        }
        for (int b = 0; b < 2; ++b) {
            tc::mbar_init(&bar_st_ready[b], ST_CONSUMERS / 32);
            tc::mbar_init(&bar_st_free[b], 1);
            tc::mbar_init(&bar_mp_ready[b], 1);
            tc::mbar_init(&bar_mp_free[b], ST_CONSUMERS / 32);
        }
        tc::mbar_init_fence();
    }
    if (tid >= 64 && tid < 64 + p.n_caches) {
        const CacheDev &c = p.c[tid - 64];
        ScoreTab e;
        e.round_base = c.sc_round_base;
        e.hpr = c.sc_hpr;
        e.hi = (int)blockIdx.x / c.sc_team;
        e.chunk = (int)blockIdx.x - e.hi * c.sc_team;
        e.T = c.T;
        s_tab[tid - 64] = e;
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
            // Q of a pass goes to the buffer of its kind once the MMAs of that buffer's last user are done
            auto load_q = [&](const ScoreItem &item, int kind) -> bool {
                if (nq[kind] > 0 && !tc::mbar_wait(&bar_q_free[kind], (nq[kind] - 1) & 1u, wc, 64)) return false;
                const uint32_t qdst = tc::smem_u32(q_s + kind * ST_TILE_BYTES);
                tc::mbar_expect_tx(&bar_q_full[kind], ST_TILE_BYTES);
                tc::tma_load_3d(qdst, &tm.b[item.cache], &bar_q_full[kind], 0, item.qt * 128, item.lh);      // rows past n_q read as zero
                tc::tma_load_3d(qdst + ST_TILE_BYTES / 2, &tm.b[item.cache], &bar_q_full[kind], 64, item.qt * 128, item.lh);
                ++nq[kind];
                return true;
            };
            PassIter pi;
            ScoreItem item, nxt;
            int kind = 0, nkind = 0;
            bool have = next_pass(p, s_tab, R, pi, item, kind);
            if (have) load_q(item, kind);
            while (have && !dead) {
                if (kind == 0) {
                    // the next statistics pass reads its tiles from HBM: ask for them now
                    ScoreItem nx;
                    if (item.r + 1 < R && score_item(p, s_tab, item.r + 1, nx)) {
                        for (int t = 0; t < nx.nt; ++t) {
                            tc::tma_prefetch_l2_3d(&tm.a[nx.cache], 0, nx.chunk * ST_CHUNK + t * 128, nx.lh);
                            tc::tma_prefetch_l2_3d(&tm.a[nx.cache], 64, nx.chunk * ST_CHUNK + t * 128, nx.lh);
                        }
                    }
                }
                for (int t = 0; t < item.nt; ++t, ++it) {
                    const int s = it % ST_STAGES;
                    // the stage is free once the MMAs of the tile that used it last are done: that is the
                    // same event that hands the accumulator tile to the consumers
                    if (it >= (uint32_t)ST_STAGES) {
                        const uint32_t j = it - ST_STAGES;
                        if (!tc::mbar_wait(&bar_t_full[j % ST_TBUF], (j / ST_TBUF) & 1u, wc, 64)) { dead = true; break; }
                    }
                    tc::mbar_expect_tx(&bar_full[s], ST_TILE_BYTES);
                    const uint32_t dst = tc::smem_u32(ring + s * ST_TILE_BYTES);
                    const int row0 = item.chunk * ST_CHUNK + t * 128;
                    tc::tma_load_3d(dst, &tm.a[item.cache], &bar_full[s], 0, row0, item.lh);
                    tc::tma_load_3d(dst + ST_TILE_BYTES / 2, &tm.a[item.cache], &bar_full[s], 64, row0, item.lh);
                }
                if (dead) break;
                // Q of the next pass, while the tiles just asked for are worked on
                have = next_pass(p, s_tab, R, pi, nxt, nkind);
                if (have && !load_q(nxt, nkind)) dead = true;
                item = nxt;
                kind = nkind;
            }
            // nothing this thread started may still be in flight when the block exits
            for (uint32_t j = it > (uint32_t)ST_STAGES ? it - ST_STAGES : 0u; j < it; ++j)
                tc::mbar_wait(&bar_full[j % ST_STAGES], (j / ST_STAGES) & 1u, wc, 64);
            for (int b = 0; b < 2; ++b)
                if (nq[b] > 0) tc::mbar_wait(&bar_q_full[b], (nq[b] - 1) & 1u, wc, 64);
        }
    } else if (warp == 1 || warp == ST_THREADS / 32 - 1) {
        // ---------------- MMA issuers: two threads, alternate tiles ----------------
        // What an issuer does for a tile (two barrier tests, eight instructions that each hold the thread
        // for about 100 cycles, a commit) takes longer than the tensor cores need for the tile; two
        // issuers on separate warps overlap that.  Tiles are independent: different accumulators and ring
        // stages, and a commit only covers its own thread's instructions.
        if (lane == 0) {
            constexpr uint32_t IDESC = tc::idesc_bf16(128, 128, 0, 0);
            const uint32_t me = warp == 1 ? 0u : 1u;
            uint32_t it = 0, nq[2] = {0u, 0u};
            const uint32_t ring_addr = tc::smem_u32(ring);
            bool dead = false;
            PassIter pi;
            ScoreItem item;
            int kind = 0;
            while (!dead && next_pass(p, s_tab, R, pi, item, kind)) {
                if (!tc::mbar_wait(&bar_q_full[kind], nq[kind] & 1u, wc)) break;
                ++nq[kind];
                // operand descriptors: the k-step only moves the start address (in 16-byte units, low word)
                const uint64_t dq0 = tc::smem_desc_sw128(tc::smem_u32(q_s + kind * ST_TILE_BYTES), 16, 1024);
                bool issued = false;
                for (int t = 0; t < item.nt; ++t) {
                    const uint32_t ti = it + t;
                    if ((ti & 1u) != me) continue;
                    // accumulator tile and ring stage share their index and the parity of their use
                    const uint32_t tb = ti % ST_TBUF, par = (ti / ST_TBUF) & 1u;
                    const bool e_ok = tc::mbar_test(&bar_t_empty[tb], par ^ 1u), f_ok = tc::mbar_test(&bar_full[tb], par);
                    if (!e_ok && !tc::mbar_wait(&bar_t_empty[tb], par ^ 1u, wc)) { dead = true; break; }
                    if (!f_ok && !tc::mbar_wait(&bar_full[tb], par, wc)) { dead = true; break; }
                    tc::tc_fence_after();
                    const uint64_t dk0 = tc::smem_desc_sw128(ring_addr + tb * ST_TILE_BYTES, 16, 1024);
                    const uint32_t acc = tmem + tb * 128u;
                    // pass A: queries on the lanes (S = Q K^T); pass B: keys on the lanes (S^T = K Q^T)
                    const uint64_t da0 = kind == 0 ? dq0 : dk0, db0 = kind == 0 ? dk0 : dq0;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        // 16 channels per instruction: 32 bytes along the swizzled row, second half after 4 steps
                        constexpr uint32_t HALF16 = (ST_TILE_BYTES / 2) >> 4;
                        const uint64_t off16 = (uint64_t)((kk >> 2) * HALF16 + (kk & 3) * 2);
                        tc::umma_bf16(acc, da0 + off16, db0 + off16, IDESC, kk > 0 ? 1u : 0u);
                    }
                    tc::umma_commit(&bar_t_full[tb]);
                    issued = true;
                }
                it += item.nt;
                // the Q buffer is free when both issuers' instructions of the pass are done
                if (!dead) {
                    if (issued) tc::umma_commit(&bar_q_free[kind]);
                    else tc::mbar_arrive(&bar_q_free[kind]);
                }
            }
        }
    } else if (warp < 2 + ST_CONSUMERS / 32) {
        // ---------------- consumers ----------------
        static_assert(ST_TBUF % ST_GROUPS == 0, "an accumulator tile must always belong to the same consumer group");
        const int q = warp & 3;                        // tensor-memory lane quarter this warp may touch
        const int grp = (warp - 2) >> 2;               // tiles with index == grp (mod ST_GROUPS) are this warp's
        const int row = q * 32 + lane;                 // lane of the accumulator tile: a query (pass A) or a key (pass B)
        const uint32_t tlane = tmem + ((uint32_t)(q * 32) << 16);
        const float sc = ST_LOG2E * rsqrtf(128.0f);
        uint32_t it = 0, n_a[2] = {0u, 0u}, n_b[2] = {0u, 0u};

        // The four 32-column pieces of an accumulator tile, `work(piece, registers)` on each; the tile is handed
        // back as soon as its last piece is in registers.
        auto walk_tile = [&](uint32_t ti, auto &&work) {
            const uint32_t tb = ti % ST_TBUF;
            tc::mbar_wait(&bar_t_full[tb], (ti / ST_TBUF) & 1u, wc, 20);
            tc::tc_fence_after();
            const uint32_t ta = tlane + tb * 128u;
            uint32_t rr[32];
#pragma unroll 1
            for (int pc = 0; pc < 4; ++pc) {
                tc::tmem_ld32(ta + 32u * pc, rr);
                tc::tmem_ld_wait();
                if (pc == 3) {
                    tc::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(&bar_t_empty[tb]);
                }
                work(pc, rr);
            }
        };

        for (int i = 0; i < R + ST_LAG; ++i) {
            // ======== pass A of round i: maximum and sum per query over the keys of this group's tiles ========
            ScoreItem item;
            if (i < R && score_item(p, s_tab, i, item)) {
                const int T = s_tab[item.cache].T, buf = i & 1;
                // a chunk has at most as many tiles as there are groups: this group meets at most one of them
                static_assert(ST_GROUPS == ST_TILES, "one tile of a chunk per consumer group");
                float m = -INFINITY, z = 0.f;
                int my_t = -1;
#pragma unroll 1
                for (int t = 0; t < item.nt; ++t) {
                    const uint32_t ti = it + t;
                    if ((int)(ti % ST_GROUPS) != grp) continue;
                    my_t = t;
                    const int key0 = item.chunk * ST_CHUNK + t * 128;                     // key of column 0 of the tile
                    walk_tile(ti, [&](int pc, uint32_t (&rr)[32]) {
                        // two copies of the update: the one that masks missing keys runs for a head's ragged last tile only
                        const int k0 = key0 + 32 * pc;
                        if (k0 + 32 > T) stats_update<true>(rr, T - k0, sc, m, z);
                        else stats_update<false>(rr, 32, sc, m, z);
                    });
                }
                it += item.nt;
                // hand (m, z) of the tile to the messenger, filed under the tile's place in the chunk: the messenger
                // merges a chunk's tiles in that order whichever groups worked on them
                if (n_a[buf] > 0) tc::mbar_wait(&bar_st_free[buf], (n_a[buf] - 1) & 1u, wc, 20);
                if (my_t >= 0) {
                    s_m[(buf * ST_TILES + my_t) * 128 + row] = m;
                    s_z[(buf * ST_TILES + my_t) * 128 + row] = z;
                }
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&bar_st_ready[buf]);
                ++n_a[buf];
            }
            // ======== pass B of round i - ST_LAG: pooled mass per key over all queries of the tile ========
            if (i >= ST_LAG && score_item(p, s_tab, i - ST_LAG, item)) {
                const CacheDev &c = p.c[item.cache];
                const int T = s_tab[item.cache].T, buf = (i - ST_LAG) & 1;
                tc::mbar_wait(&bar_mp_ready[buf], n_b[buf] & 1u, wc, 20);
                const float *mp = s_mp + buf * 128;
                // with two query tiles per head each writes its own plane; a small kernel adds them up afterwards
                float *dst = (item.qt ? p.scores2 : p.scores) + c.tok_off + (size_t)item.lh * T;
                float *out = (c.scores_out && p.sc_qt == 1) ? c.scores_out + (size_t)item.lh * T : nullptr;
#pragma unroll 1
                for (int t = 0; t < item.nt; ++t) {
                    const uint32_t ti = it + t;
                    if ((int)(ti % ST_GROUPS) != grp) continue;
                    float a = 0.f;
                    walk_tile(ti, [&](int pc, uint32_t (&rr)[32]) { a += pool_piece(rr, mp + 32 * pc, sc); });
                    const int j = item.chunk * ST_CHUNK + t * 128 + row;
                    if (j < T) {
                        if (!isfinite(a)) atomicOr(p.status, OBF_DEV_NONFINITE);
                        dst[j] = a;
                        if (out) out[j] = a;
                    }
                }
                it += item.nt;
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&bar_mp_free[buf]);
                ++n_b[buf];
            }
        }
    } else {
        // ---------------- messenger: chunk statistics out, a head's chunks folded by the last block to arrive, M' in ----------------
        uint32_t n_a[2] = {0u, 0u}, n_b[2] = {0u, 0u};
        for (int i = 0; i < R; ++i) {
            ScoreItem item;
            if (!score_item(p, s_tab, i, item)) continue;
            const CacheDev &c = p.c[item.cache];
            const int buf = i & 1, team = c.sc_team;
            const int g = c.head_base * p.sc_qt + item.lv;                     // index of the (head, query tile) pair
            const int nq = min(128, p.n_q - 128 * item.qt);                    // query rows of this item
            tc::mbar_wait(&bar_st_ready[buf], n_a[buf] & 1u, wc, 32);
            float2 *partials = reinterpret_cast<float2 *>(p.sc_part) + (c.sc_part_off + ((size_t)item.lv * team + item.chunk) * 128);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int t = lane + 32 * k;
                const float *sm = s_m + buf * ST_TILES * 128 + t, *sz = s_z + buf * ST_TILES * 128 + t;
                float M = sm[0];
                for (int e = 1; e < item.nt; ++e) M = fmaxf(M, sm[e * 128]);
                float Z = 0.f;
                for (int e = 0; e < item.nt; ++e)
                    if (sm[e * 128] > -INFINITY) Z += sz[e * 128] * ex2_approx(sm[e * 128] - M);
                if (t < nq) __stcg(&partials[t], make_float2(M, Z));
            }
            __syncwarp();
            uint32_t last = 0u;
            if (lane == 0) {
                tc::mbar_arrive(&bar_st_free[buf]);
                // the warp barrier orders the lanes' stores before this release; the acquire side mirrors it
                last = (atom_add_acq_rel_gpu(&p.sc_cnt[g], 1u) == (uint32_t)(team - 1)) ? 1u : 0u;
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            ++n_a[buf];
            if (last) {
                // every lane reads other blocks' statistics below: each orders its own loads behind lane 0's acquire
                asm volatile("fence.acq_rel.gpu;" ::: "memory");
                // this block is the last of its head: fold all chunks, eight chunks of the lane's four queries per sweep
                // (32 loads in flight: the fold is a few round trips long, whatever the team's size)
                const float2 *hp = reinterpret_cast<const float2 *>(p.sc_part) + (c.sc_part_off + (size_t)item.lv * team * 128);
                unsigned long long *words = reinterpret_cast<unsigned long long *>(p.sc_head) + (size_t)g * 128;
                float M[4], Z[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) { M[k] = -INFINITY; Z[k] = 0.f; }
                for (int c0 = 0; c0 < team; c0 += 8) {
                    float2 v[4][8];
#pragma unroll
                    for (int k = 0; k < 4; ++k)
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            v[k][e] = (c0 + e < team && lane + 32 * k < nq) ? __ldcg(&hp[(size_t)(c0 + e) * 128 + lane + 32 * k])
                                                                               : make_float2(-INFINITY, 0.f);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        float Mn = M[k];
#pragma unroll
                        for (int e = 0; e < 8; ++e) Mn = fmaxf(Mn, v[k][e].x);
                        if (Mn > -INFINITY) {
                            Z[k] *= ex2_approx(M[k] - Mn);
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                if (v[k][e].x > -INFINITY) Z[k] += v[k][e].y * ex2_approx(v[k][e].x - Mn);
                            M[k] = Mn;
                        }
                    }
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int t = lane + 32 * k;
                    if (t >= nq) continue;
                    // the keys outside the prompt take their share of the normaliser
                    if (c.lse_extra) fold_lse_extra(c.lse_extra[(size_t)item.lh * p.n_q + 128 * item.qt + t], M[k], Z[k]);
                    float mp = M[k] + lg2_approx(Z[k]);
                    if (!(Z[k] > 0.f) || !isfinite(mp)) {
                        atomicOr(p.status, OBF_DEV_NONFINITE);
                        mp = __int_as_float(0x7fc00000);
                    }
                    // one 64-bit word per query: low = M'_t, high = 1 once it is valid
                    if (!p.debug_drop_publish) st_relaxed_gpu_u64(words + t, (1ull << 32) | __float_as_uint(mp));
                }
            }
            // M'_t of this head for the pooling pass one round on; the team has a round to get there
            {
                const int fb = i & 1;
                if (n_b[fb] > 0) tc::mbar_wait(&bar_mp_free[fb], (n_b[fb] - 1) & 1u, wc, 32);
                const unsigned long long *words = reinterpret_cast<const unsigned long long *>(p.sc_head) + (size_t)g * 128;
                // the four words of this lane are polled together: one round trip, not four
                unsigned long long v[4] = {0ull, 0ull, 0ull, 0ull};
                const uint64_t t0 = tc::global_ns();
                for (;;) {
                    bool all = true;
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (lane + 32 * k < nq && (v[k] >> 32) == 0ull) v[k] = ld_relaxed_gpu_u64(words + lane + 32 * k);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (lane + 32 * k < nq && (v[k] >> 32) == 0ull) all = false;
                    // the warp leaves the loop as one: votes, not per-lane exits
                    if (__all_sync(0xffffffffu, all) || __any_sync(0xffffffffu, *(volatile uint32_t *)&s_abort != 0u)) break;
                    if (__any_sync(0xffffffffu, tc::global_ns() - t0 > p.wait_limit_ns)) {
                        if (lane == 0) {
                            s_abort = 1u;
                            atomicOr(p.status, OBF_DEV_TIMEOUT);
                        }
                        break;
                    }
                    __nanosleep(64);
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int t = lane + 32 * k;
                    // exp2(-inf) = 0 for padding columns
                    s_mp[fb * 128 + t] = t < nq ? __uint_as_float((uint32_t)v[k]) : INFINITY;
                }
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&bar_mp_ready[fb]);
                ++n_b[fb];
            }
        }
    }

    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem, 512);
}

// Heads with two query tiles: the masses of the second tile's rows are added to the first tile's.
// grid = (ceil(T_max / 256), heads_total).
__global__ void __launch_bounds__(256) k_score_join(const __grid_constant__ CallDev p)
{
    int ci, lh;
    locate(p, blockIdx.y, ci, lh);
    const CacheDev &c = p.c[ci];
    const int j = blockIdx.x * 256 + threadIdx.x;
    if (j >= c.T) return;
    const size_t e = c.tok_off + (size_t)lh * c.T + j;
    const float a = p.scores[e] + p.scores2[e];
    p.scores[e] = a;
    if (c.scores_out) c.scores_out[(size_t)lh * c.T + j] = a;
}

}  // namespace obf
