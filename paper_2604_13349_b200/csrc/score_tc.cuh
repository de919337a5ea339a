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
// (head, chunk) = (round * heads_per_round + block / team, block % team).
//
// The two kinds of pass are two STREAMS that run side by side in a block and share only the
// tensor pipe and the special-function unit: the statistics stream walks the block's items
// i = 0, 1, .., the pooling stream walks the same items behind it, item i as soon as the
// head's M' is there (every block of the team has published its statistics of the item and
// the last one has folded them).  Each stream has its own ring of K tiles, its own
// accumulator tiles in tensor memory and its own consumer warps, so a stream that waits
// (for the team, for a tile) leaves the arithmetic units to the other one; the pooling
// stream never asks for a chunk before the statistics stream has brought it into the L2
// cache.  Every wait is bounded (tc_common.cuh).
//
// Block = 20 warps.  Warp 0: TMA producer, one thread that feeds both rings (whichever has
// room) and the three query buffers: Q of item n lives in buffer n mod 3 from the time the
// statistics stream is one item before it until the pooling stream is done with it, so a
// query tile is loaded once and a whole item ahead.  Warps 1 and 19: the MMA issuers of the
// two streams.  An accumulator tile (128 columns) is filled, handed over and given back in two
// halves of 64 columns, so the MMAs of a group's next tile run behind its arithmetic.
// Warps 2..17: consumers, four groups of four (a warp owns the 32 tensor-memory lanes of its
// quarter): groups 0 and 1 take alternate tiles of the statistics stream, groups 2 and 3 of
// the pooling stream; every scheduler holds one warp of each group.  A warp walks the 128
// columns of a tile in four pieces of 32 (load, wait, exponentials).  A key's pooled mass is
// complete in one thread.  A statistics group writes the (maximum, sum) of its tiles of a chunk
// (tiles 0 and 2, or 1 and 3, merged in that order whichever group they fall to) straight to the
// workspace.  Warp 18 is the messenger: once the eight statistics warps have written, it counts
// the block in, folds the head's chunks when its block is the last of the team to arrive, and
// then fetches the head's M' into shared memory for the pooling stream, so that the consumers
// never wait for global memory.
// Measured alternatives that were slower: one sequence of passes A(i), B(i-1) with all four
// groups on the same pass (every group reaches a pass boundary at the same time and the
// special-function unit idles there), the load of a piece in flight behind the arithmetic of the
// piece before it, a share of the exponentials evaluated as a polynomial on the FMA pipe.
#pragma once

#include "tc_common.cuh"

namespace obf {

constexpr int ST_TILES = 4;                         // 128-key tiles per chunk
constexpr int ST_CHUNK = ST_TILES * 128;
constexpr int ST_STREAMS = 2;                       // stream 0: statistics passes, stream 1: pooling passes
constexpr int ST_SBUF = 2;                          // per stream: K tiles in flight in shared memory = accumulator tiles in tensor memory = consumer groups
constexpr int ST_HALVES = 2;                        // an accumulator tile is filled, handed over and given back in halves of 64 columns
constexpr int ST_QBUF = 3;                          // query tiles in shared memory: the pooling item's, the statistics item's, the next one's
constexpr int ST_PART = 2;                          // (maximum, sum) pairs a block publishes per chunk and query: tiles 0+2 and tiles 1+3
constexpr int ST_TILE_BYTES = 128 * 128 * 2;
constexpr int ST_STREAM_WARPS = ST_SBUF * 4;        // consumer warps of a stream: groups of four, a warp per tensor-memory lane quarter
constexpr int ST_CONSUMERS = ST_STREAMS * ST_STREAM_WARPS * 32;
constexpr int ST_THREADS = 64 + ST_CONSUMERS + 64;
constexpr int ST_MAX_NQ = 256;                      // two query tiles of 128 rows
constexpr float ST_LOG2E = 1.4426950408889634f;
constexpr size_t ST_SMEM_BYTES = 1024 + (size_t)ST_QBUF * ST_TILE_BYTES + (size_t)ST_STREAMS * ST_SBUF * ST_TILE_BYTES +
                                 2 * 128 * sizeof(float) + 64;
static_assert(ST_STREAMS * ST_SBUF * 128 == 512, "the accumulator tiles fill the tensor memory");
static_assert(ST_SBUF == 2 && ST_PART == 2, "a group's tiles of a chunk are the even or the odd ones");

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

__device__ __forceinline__ void red_add_release_gpu(uint32_t *addr, uint32_t v)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(addr), "r"(v) : "memory");
}

__device__ __forceinline__ uint32_t ld_acquire_gpu_u32(const uint32_t *addr)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(addr) : "memory");
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
    uint8_t *q_s = base;                                           // ST_QBUF x [128 x 128] bf16 queries, two 64-column halves each
    uint8_t *ring = q_s + ST_QBUF * ST_TILE_BYTES;                 // per stream ST_SBUF stages of 32 KiB
    float *s_mp = reinterpret_cast<float *>(ring + ST_STREAMS * ST_SBUF * ST_TILE_BYTES);   // [2][128] M'_t of the heads being pooled
    __shared__ uint64_t bar_q_full[ST_QBUF], bar_q_free[ST_QBUF], bar_full[ST_STREAMS * ST_SBUF];
    __shared__ uint64_t bar_t_full[ST_STREAMS * ST_SBUF * ST_HALVES], bar_t_empty[ST_STREAMS * ST_SBUF * ST_HALVES];
    __shared__ uint64_t bar_mp_ready[2], bar_mp_free[2];
    __shared__ ScoreTab s_tab[OBF_MAX_CACHES];
    __shared__ uint32_t s_tmem, s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int R = p.sc_rounds;
    tc::WaitCtx wc{&s_abort, p.status, p.wait_limit_ns};

    if (tid == 0) {
        s_abort = 0u;
        for (int b = 0; b < ST_QBUF; ++b) { tc::mbar_init(&bar_q_full[b], 1); tc::mbar_init(&bar_q_free[b], 1); }
        for (int s = 0; s < ST_STREAMS * ST_SBUF; ++s) tc::mbar_init(&bar_full[s], 1);
        for (int s = 0; s < ST_STREAMS * ST_SBUF * ST_HALVES; ++s) {
            tc::mbar_init(&bar_t_full[s], 1);
            tc::mbar_init(&bar_t_empty[s], 4);                  // the four warps of the group that owns the tile
        }
        for (int b = 0; b < 2; ++b) {
            tc::mbar_init(&bar_mp_ready[b], 1);
            tc::mbar_init(&bar_mp_free[b], ST_STREAM_WARPS);
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
        // ---------------- TMA producer: one thread feeds both rings and the query buffers, whichever has room ----------------
        if (lane == 0) {
            struct Feed {
                int r, t;              // round of the item being fed (R: none left), next tile of it
                uint32_t k, n;         // tiles asked for so far; items begun so far
                bool have;
                ScoreItem item;
            };
            Feed f[ST_STREAMS], fq;    // fq walks the items one ahead of the statistics stream and loads their queries
            auto advance = [&](Feed &x) {
                x.have = false;
                while (!x.have && x.r + 1 < R) x.have = score_item(p, s_tab, ++x.r, x.item);
                if (!x.have) x.r = R;
                x.t = 0;
            };
            for (int s = 0; s < ST_STREAMS; ++s) {
                f[s].r = -1;
                f[s].k = f[s].n = 0u;
                advance(f[s]);
            }
            fq.r = -1;
            fq.k = fq.n = 0u;
            advance(fq);
            uint64_t stalled_since = 0;
            while (f[0].have || f[1].have) {
                bool progress = false;
                // Q of item n goes to buffer n mod ST_QBUF once the pooling stream's MMAs of item n - ST_QBUF are done;
                // it is asked for as soon as the statistics stream has begun the item before it
                if (fq.have && fq.n <= f[0].n + (f[0].have ? 0u : 1u) &&
                    (fq.n < (uint32_t)ST_QBUF || tc::mbar_test(&bar_q_free[fq.n % ST_QBUF], (fq.n / ST_QBUF - 1) & 1u))) {
                    const uint32_t qb = fq.n % ST_QBUF;
                    const uint32_t qdst = tc::smem_u32(q_s + qb * ST_TILE_BYTES);
                    tc::mbar_expect_tx(&bar_q_full[qb], ST_TILE_BYTES);
                    tc::tma_load_3d(qdst, &tm.b[fq.item.cache], &bar_q_full[qb], 0, fq.item.qt * 128, fq.item.lh);      // rows past n_q read as zero
                    tc::tma_load_3d(qdst + ST_TILE_BYTES / 2, &tm.b[fq.item.cache], &bar_q_full[qb], 64, fq.item.qt * 128, fq.item.lh);
                    ++fq.n;
                    advance(fq);
                    progress = true;
                }
#pragma unroll 1
                for (int s = 0; s < ST_STREAMS; ++s) {
                    Feed &x = f[s];
                    if (!x.have) continue;
                    // the pooling stream reads a chunk from the L2 cache: it never asks for a chunk before the
                    // statistics stream has asked for all of it
                    if (s == 1 && f[0].r <= x.r) continue;
                    // a ring stage is free once the MMAs of the tile that used it last are done: that is the same
                    // event that hands the tile's last accumulator half to the consumers
                    const uint32_t sb = (uint32_t)s * ST_SBUF + x.k % ST_SBUF;
                    if (x.k >= (uint32_t)ST_SBUF) {
                        const uint32_t j = x.k - ST_SBUF;
                        if (!tc::mbar_test(&bar_t_full[sb * ST_HALVES + ST_HALVES - 1], (j / ST_SBUF) & 1u)) continue;
                    }
                    if (s == 0 && x.t == 0) {
                        // the next statistics item reads its tiles from HBM: ask for them now
                        ScoreItem nx;
                        if (x.r + 1 < R && score_item(p, s_tab, x.r + 1, nx)) {
                            for (int t = 0; t < nx.nt; ++t) {
                                tc::tma_prefetch_l2_3d(&tm.a[nx.cache], 0, nx.chunk * ST_CHUNK + t * 128, nx.lh);
                                tc::tma_prefetch_l2_3d(&tm.a[nx.cache], 64, nx.chunk * ST_CHUNK + t * 128, nx.lh);
                            }
                        }
                    }
                    tc::mbar_expect_tx(&bar_full[sb], ST_TILE_BYTES);
                    const uint32_t dst = tc::smem_u32(ring + sb * ST_TILE_BYTES);
                    const int row0 = x.item.chunk * ST_CHUNK + x.t * 128;
                    tc::tma_load_3d(dst, &tm.a[x.item.cache], &bar_full[sb], 0, row0, x.item.lh);
                    tc::tma_load_3d(dst + ST_TILE_BYTES / 2, &tm.a[x.item.cache], &bar_full[sb], 64, row0, x.item.lh);
                    ++x.k;
                    progress = true;
                    if (x.t == 0) ++x.n;
                    if (++x.t == x.item.nt) advance(x);
                }
                if (progress) {
                    stalled_since = 0;
                    continue;
                }
                // nothing has room: bounded like every other wait
                if (s_abort) break;
                const uint64_t now = tc::global_ns();
                if (stalled_since == 0) stalled_since = now;
                else if (now - stalled_since > p.wait_limit_ns) {
                    s_abort = 1u;
                    atomicOr(p.status, OBF_DEV_TIMEOUT);
                    break;
                }
                __nanosleep(32);
            }
            // nothing this thread started may still be in flight when the block exits
            for (int s = 0; s < ST_STREAMS; ++s)
                for (uint32_t j = f[s].k > (uint32_t)ST_SBUF ? f[s].k - ST_SBUF : 0u; j < f[s].k; ++j)
                    tc::mbar_wait(&bar_full[s * ST_SBUF + j % ST_SBUF], (j / ST_SBUF) & 1u, wc, 64);
            for (uint32_t j = fq.n > (uint32_t)ST_QBUF ? fq.n - ST_QBUF : 0u; j < fq.n; ++j)
                tc::mbar_wait(&bar_q_full[j % ST_QBUF], (j / ST_QBUF) & 1u, wc, 64);
        }
    } else if (warp == 1 || warp == ST_THREADS / 32 - 1) {
        // ---------------- MMA issuers: one thread per stream ----------------
        if (lane == 0) {
            constexpr uint32_t IDESC = tc::idesc_bf16(128, 128 / ST_HALVES, 0, 0);
            const int s = warp == 1 ? 0 : 1;
            uint32_t k = 0, n = 0;
            const uint32_t ring_addr = tc::smem_u32(ring);
            bool dead = false;
            for (int r = 0; r < R && !dead; ++r) {
                ScoreItem item;
                if (!score_item(p, s_tab, r, item)) continue;
                const uint32_t qb = n % ST_QBUF;
                if (!tc::mbar_wait(&bar_q_full[qb], (n / ST_QBUF) & 1u, wc)) break;
                ++n;
                // operand descriptors: the k-step only moves the start address (in 16-byte units, low word)
                const uint64_t dq0 = tc::smem_desc_sw128(tc::smem_u32(q_s + qb * ST_TILE_BYTES), 16, 1024);
                for (int t = 0; t < item.nt && !dead; ++t, ++k) {
                    // accumulator tile and ring stage share their index and the parity of their use
                    const uint32_t sb = (uint32_t)s * ST_SBUF + k % ST_SBUF, par = (k / ST_SBUF) & 1u;
                    if (!tc::mbar_test(&bar_full[sb], par) && !tc::mbar_wait(&bar_full[sb], par, wc)) { dead = true; break; }
                    const uint64_t dk0 = tc::smem_desc_sw128(ring_addr + sb * ST_TILE_BYTES, 16, 1024);
                    // The tile's 128 accumulator columns are filled in two halves of 64, each with its own pair of
                    // barriers: the consumers give a half back while they still work on the other one.
#pragma unroll 1
                    for (uint32_t h = 0; h < (uint32_t)ST_HALVES; ++h) {
                        const uint32_t hb = sb * ST_HALVES + h;
                        if (!tc::mbar_test(&bar_t_empty[hb], par ^ 1u) && !tc::mbar_wait(&bar_t_empty[hb], par ^ 1u, wc)) { dead = true; break; }
                        tc::tc_fence_after();
                        const uint32_t acc = tmem + sb * 128u + h * (128u / ST_HALVES);
                        // the 64 rows of the column operand that make this half: 128 bytes a row inside both channel halves
                        const uint64_t hoff = (uint64_t)((h * (128u / ST_HALVES) * 128u) >> 4);
                        // statistics: queries on the lanes (S = Q K^T), the half's columns are keys;
                        // pooling: keys on the lanes (S^T = K Q^T), the half's columns are queries
                        const uint64_t da0 = s == 0 ? dq0 : dk0, db0 = (s == 0 ? dk0 : dq0) + hoff;
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            // 16 channels per instruction: 32 bytes along the swizzled row, second half after 4 steps
                            constexpr uint32_t HALF16 = (ST_TILE_BYTES / 2) >> 4;
                            const uint64_t off16 = (uint64_t)((kk >> 2) * HALF16 + (kk & 3) * 2);
                            tc::umma_bf16(acc, da0 + off16, db0 + off16, IDESC, kk > 0 ? 1u : 0u);
                        }
                        tc::umma_commit(&bar_t_full[hb]);
                    }
                }
                // the item's query buffer may be loaded again once the pooling stream's instructions on it are done
                if (s == 1 && !dead) tc::umma_commit(&bar_q_free[qb]);
            }
        }
    } else if (warp < 2 + ST_CONSUMERS / 32) {
        // ---------------- consumers ----------------
        const int q = warp & 3;                        // tensor-memory lane quarter this warp may touch
        const int grp = (warp - 2) >> 2;               // groups 0, 1: statistics stream; groups 2, 3: pooling stream
        const int s = grp / ST_SBUF, gs = grp % ST_SBUF;   // stream, and which of the stream's tiles are this group's
        const int row = q * 32 + lane;                 // lane of the accumulator tile: a query (statistics) or a key (pooling)
        const uint32_t tlane = tmem + ((uint32_t)(q * 32) << 16);
        const float sc = ST_LOG2E * rsqrtf(128.0f);
        uint32_t k = 0;

        // The four 32-column pieces of an accumulator tile, `work(piece, registers)` on each; a half of the tile is
        // handed back as soon as its second piece is in registers.
        auto walk_tile = [&](uint32_t kt, auto &&work) {
            const uint32_t sb = (uint32_t)s * ST_SBUF + kt % ST_SBUF;
            const uint32_t ta = tlane + sb * 128u;
            uint32_t rr[32];
#pragma unroll 1
            for (int pc = 0; pc < 4; ++pc) {
                const uint32_t hb = sb * ST_HALVES + (uint32_t)(pc >> 1);
                if ((pc & 1) == 0) {
                    tc::mbar_wait(&bar_t_full[hb], (kt / ST_SBUF) & 1u, wc, 20);
                    tc::tc_fence_after();
                }
                tc::tmem_ld32(ta + 32u * pc, rr);
                tc::tmem_ld_wait();
                if (pc & 1) {
                    // the half's second piece is in registers: the half goes back to the MMA issuer
                    tc::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(&bar_t_empty[hb]);
                }
                work(pc, rr);
            }
        };

        if (s == 0) {
            // ======== statistics stream: maximum and sum per query over the keys of this group's tiles of a chunk ========
            for (int i = 0; i < R; ++i) {
                ScoreItem item;
                if (!score_item(p, s_tab, i, item)) continue;
                const CacheDev &c = p.c[item.cache];
                const int T = s_tab[item.cache].T;
                float m = -INFINITY, z = 0.f;
#pragma unroll 1
                for (int t = 0; t < item.nt; ++t) {
                    if ((int)((k + t) % ST_SBUF) != gs) continue;
                    const int key0 = item.chunk * ST_CHUNK + t * 128;                     // key of column 0 of the tile
                    walk_tile(k + t, [&](int pc, uint32_t (&rr)[32]) {
                        // two copies of the update: the one that masks missing keys runs for a head's ragged last tile only
                        const int k0 = key0 + 32 * pc;
                        if (k0 + 32 > T) stats_update<true>(rr, T - k0, sc, m, z);
                        else stats_update<false>(rr, 32, sc, m, z);
                    });
                }
                // this group's tiles are the even or the odd ones of the chunk; (m, z) goes to the workspace under that
                // parity, so that the fold meets the same pairs in the same order whichever group worked on them
                const int slot = (int)((gs + k) % ST_SBUF);
                float2 *partials = reinterpret_cast<float2 *>(p.sc_part) +
                                   (c.sc_part_off + (((size_t)item.lv * c.sc_team + item.chunk) * ST_PART + slot) * 128);
                __stcg(&partials[row], make_float2(m, z));
                k += item.nt;
                // the warp counts itself in for the (head, query tile): the warp barrier orders the lanes' stores before
                // lane 0's release, and nobody waits for the counter's answer
                __syncwarp();
                if (lane == 0 && !p.debug_drop_publish) red_add_release_gpu(&p.sc_cnt[c.head_base * p.sc_qt + item.lv], 1u);
            }
        } else {
            // ======== pooling stream: pooled mass per key over all queries of the item ========
            uint32_t n_h[2] = {0u, 0u};
            for (int i = 0; i < R; ++i) {
                ScoreItem item;
                if (!score_item(p, s_tab, i, item)) continue;
                const CacheDev &c = p.c[item.cache];
                const int T = s_tab[item.cache].T, buf = i & 1;
                tc::mbar_wait(&bar_mp_ready[buf], n_h[buf] & 1u, wc, 20);
                const float *mp = s_mp + buf * 128;
                // with two query tiles per head each writes its own plane; a small kernel adds them up afterwards
                float *dst = (item.qt ? p.scores2 : p.scores) + c.tok_off + (size_t)item.lh * T;
                float *out = (c.scores_out && p.sc_qt == 1) ? c.scores_out + (size_t)item.lh * T : nullptr;
#pragma unroll 1
                for (int t = 0; t < item.nt; ++t) {
                    if ((int)((k + t) % ST_SBUF) != gs) continue;
                    float a = 0.f;
                    walk_tile(k + t, [&](int pc, uint32_t (&rr)[32]) { a += pool_piece(rr, mp + 32 * pc, sc); });
                    const int j = item.chunk * ST_CHUNK + t * 128 + row;
                    if (j < T) {
                        if (!isfinite(a)) atomicOr(p.status, OBF_DEV_NONFINITE);
                        dst[j] = a;
                        if (out) out[j] = a;
                    }
                }
                k += item.nt;
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&bar_mp_free[buf]);
                ++n_h[buf];
            }
        }
    } else {
        // ---------------- messenger: waits for the head's team, folds its statistics, M' into shared memory ----------------
        // Every block of a team folds for itself (the same pairs in the same order: the same bits), so nothing but the
        // statistics warps' counter stands between a team's statistics and a block's pooling.
        uint32_t n_b[2] = {0u, 0u};
        for (int i = 0; i < R; ++i) {
            ScoreItem item;
            if (!score_item(p, s_tab, i, item)) continue;
            const CacheDev &c = p.c[item.cache];
            const int team = c.sc_team, fb = i & 1;
            const int g = c.head_base * p.sc_qt + item.lv;                     // index of the (head, query tile) pair
            const int nq = min(128, p.n_q - 128 * item.qt);                    // query rows of this item
            // the pooling warps are done with what this buffer held two items back
            if (n_b[fb] > 0) tc::mbar_wait(&bar_mp_free[fb], (n_b[fb] - 1) & 1u, wc, 32);
            // every statistics warp of every block of the team has written its pairs of this (head, query tile)
            {
                const uint32_t want = (uint32_t)team * ST_STREAM_WARPS;
                const uint64_t t0 = tc::global_ns();
                for (;;) {
                    uint32_t ok = 1u;
                    if (lane == 0) {
                        ok = ld_acquire_gpu_u32(&p.sc_cnt[g]) >= want ? 1u : 0u;
                        if (!ok && (s_abort != 0u || tc::global_ns() - t0 > p.wait_limit_ns)) {
                            if (s_abort == 0u) {
                                s_abort = 1u;
                                atomicOr(p.status, OBF_DEV_TIMEOUT);
                            }
                            ok = 2u;
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);                     // the warp leaves the loop as one
                    if (ok) break;
                    __nanosleep(64);
                }
                // every lane reads other blocks' statistics below: each orders its own loads behind lane 0's acquire
                asm volatile("fence.acq_rel.gpu;" ::: "memory");
            }
            // fold all chunks' pairs, eight pairs of the lane's four queries per sweep (32 loads in flight)
            const float2 *hp = reinterpret_cast<const float2 *>(p.sc_part) + (c.sc_part_off + (size_t)item.lv * team * ST_PART * 128);
            const int n_pairs = team * ST_PART;
            float M[4], Z[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) { M[k] = -INFINITY; Z[k] = 0.f; }
            for (int c0 = 0; c0 < n_pairs; c0 += 8) {
                float2 v[4][8];
#pragma unroll
                for (int k = 0; k < 4; ++k)
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        v[k][e] = (c0 + e < n_pairs && lane + 32 * k < nq) ? __ldcg(&hp[(size_t)(c0 + e) * 128 + lane + 32 * k])
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
                float mp = INFINITY;                                           // exp2(-inf) = 0 for padding columns
                if (t < nq) {
                    // the keys outside the prompt take their share of the normaliser
                    if (c.lse_extra) fold_lse_extra(c.lse_extra[(size_t)item.lh * p.n_q + 128 * item.qt + t], M[k], Z[k]);
                    mp = M[k] + lg2_approx(Z[k]);
                    if (!(Z[k] > 0.f) || !isfinite(mp)) {
                        atomicOr(p.status, OBF_DEV_NONFINITE);
                        mp = __int_as_float(0x7fc00000);
                    }
                }
                s_mp[fb * 128 + t] = mp;
            }
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&bar_mp_ready[fb]);
            ++n_b[fb];
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
