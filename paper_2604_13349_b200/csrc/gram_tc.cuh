// Tuned streaming pass of Orthogonal BackFill for bf16 caches with head_dim 128:
// one pass over V on the tensor cores.
//
// Per (cache, layer, KV head) it produces what the dense algebra needs:
//   G_del  = sum over deleted j of v_j v_j^T          (R^T R = P G_del P, Eq. 3 in the Gram form of App. H)
//   u      = sum over deleted j of A_j v_j            (r_bar = P u / (A_del + eps), Eq. 4)
//   G_keep = sum over retained j of v_j v_j^T         (only when k_eff >= d: decides whether span(V_keep) = R^d, Eq. 2)
//
// Work decomposition.  Every head owns nsub_del tiles of 128 tokens of V followed by
// nsub_keep tiles of 128 rows of the compacted V_keep (read back from v_out).  All
// tiles of the call form one sequence, cut into gridDim.x runs of tc_per tiles; block b
// streams run b.  A run crosses head and kind boundaries; each maximal stretch of
// one (head, kind) inside a run is a segment and yields one partial Gram matrix
// (and one partial u), stored in slot (b - first block touching that head and kind).
//
// Block = 18 warps:
//   warp 0        TMA producer: 128 x 128 bf16 tiles (two 128-byte-swizzled column halves) into a 6-stage ring
//   warp 1        issues tcgen05.mma: G (+)= tile^T tile, both operands MN-major views of the same tile,
//                 accumulators (128 lanes x 128 columns fp32) double-buffered in tensor memory
//   warps 2..13   fix-up, three groups of four warps taking tiles in turn: zero the retained rows of a
//                 V tile in shared memory and accumulate u on the CUDA cores; the attention mass of the
//                 group's next tile (-1 marks a retained token) is fetched while the current one is processed
//   warps 14..17  epilogue: tensor memory -> partial Gram matrix in the workspace
#pragma once

#include "tc_common.cuh"

namespace obf {

constexpr int GT_KEEP_TILES_MAX = 2;                // retained-row tiles per head that enter G_keep (span test)
constexpr int GT_STAGES = 6;
constexpr int GT_TILE = 128;                       // tokens per tile
constexpr int GT_TILE_BYTES = GT_TILE * 128 * 2;   // 32 KiB
constexpr int GT_GROUPS = 3;                       // fix-up groups of four warps, taking tiles in turn
// A ring stage must always be fixed up by the same group: a thread may wait for a barrier phase only if it
// also waited for the phase before (waiting on a parity assumes the previous phase is over).
static_assert(GT_STAGES % GT_GROUPS == 0, "every ring stage must belong to one fix-up group");
constexpr int GT_FIX_THREADS = 128 * GT_GROUPS;
constexpr int GT_THREADS = 64 + GT_FIX_THREADS + 128;
constexpr size_t GT_SMEM_BYTES = 1024 + (size_t)GT_STAGES * GT_TILE_BYTES + GT_GROUPS * 8 * 128 * sizeof(float) +
                                 GT_GROUPS * 2 * 128 * sizeof(float) + 256;

// Walks the segments of one block's run of tiles.
struct TileRun {
    long long pos, end;        // current and one-past-last index in the call-wide tile sequence
    int ci;
    __device__ __forceinline__ void init(const CallDev &p, int block)
    {
        pos = (long long)block * p.tc_per;
        end = pos + p.tc_per;
        if (end > p.tc_total_sub) end = p.tc_total_sub;
        ci = 0;
    }
    // Next segment: cache, local head, kind (0 deleted / 1 retained), first tile, tile count, partial slot.
    __device__ __forceinline__ bool next(const CallDev &p, int &cache, int &lh, int &kind, int &sub0, int &nsub, int &slot)
    {
        if (pos >= end) return false;
        while (ci + 1 < p.n_caches && pos >= p.c[ci + 1].sub_base) ++ci;
        const CacheDev &c = p.c[ci];
        const int per_head = c.nsub_del + c.nsub_keep;
        const long long rel = pos - c.sub_base;
        lh = (int)(rel / per_head);
        const int o = (int)(rel - (long long)lh * per_head);
        kind = o >= c.nsub_del ? 1 : 0;
        sub0 = kind ? o - c.nsub_del : o;
        const int left_in_seg = (kind ? c.nsub_keep : c.nsub_del) - sub0;
        const long long left_in_run = end - pos;
        nsub = left_in_seg < left_in_run ? left_in_seg : (int)left_in_run;
        const long long seg_start = pos - sub0;
        slot = (int)(pos / p.tc_per - seg_start / p.tc_per);
        cache = ci;
        pos += nsub;
        return true;
    }
};

// One tile of a run, with what the fix-up warps need to know about its segment.
struct TileInfo {
    int cache, lh, kind, sub, slot;
    bool first, last;          // first / last tile of its segment within this run
};

struct TileIter {
    TileRun run;
    int cache, lh, kind, sub0, nsub, slot, t;
    __device__ __forceinline__ void init(const CallDev &p, int block) { run.init(p, block); nsub = 0; t = 0; }
    __device__ __forceinline__ bool next(const CallDev &p, TileInfo &ti)
    {
        if (t >= nsub) {
            if (!run.next(p, cache, lh, kind, sub0, nsub, slot)) return false;
            t = 0;
        }
        ti.cache = cache; ti.lh = lh; ti.kind = kind; ti.sub = sub0 + t; ti.slot = slot;
        ti.first = t == 0;
        ti.last = t == nsub - 1;
        ++t;
        return true;
    }
};

__global__ void __launch_bounds__(GT_THREADS, 1) k_gram_tc(const __grid_constant__ CallDev p, const __grid_constant__ TcMaps tm)
{
    constexpr int D = 128;
    extern __shared__ uint8_t gt_smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(gt_smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *tiles = base;                                                // GT_STAGES x 32 KiB, 1024-byte aligned
    float *u_red = reinterpret_cast<float *>(tiles + GT_STAGES * GT_TILE_BYTES);   // [GT_GROUPS][8][128]
    // [GT_GROUPS][2][128] per token of a group's current / next tile: attention mass, -1 for a retained token, 0 beyond T
    float *s_a = u_red + GT_GROUPS * 8 * 128;
    __shared__ uint64_t bar_full[GT_STAGES], bar_ready[GT_STAGES], bar_empty[GT_STAGES];
    __shared__ uint64_t bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t s_tmem, s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    tc::WaitCtx wc{&s_abort, p.status, p.wait_limit_ns};

    if (tid == 0) {
        s_abort = 0u;
        for (int s = 0; s < GT_STAGES; ++s) {
            tc::mbar_init(&bar_full[s], 1);
            tc::mbar_init(&bar_ready[s], 4);
            tc::mbar_init(&bar_empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) { tc::mbar_init(&bar_acc_full[b], 1); tc::mbar_init(&bar_acc_empty[b], 4); }
        tc::mbar_init_fence();
    }
    if (warp == 1) tc::tmem_alloc(&s_tmem, 256);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = s_tmem;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            TileRun run;
            run.init(p, blockIdx.x);
            int cache, lh, kind, sub0, nsub, slot;
            uint32_t it = 0;
            while (run.next(p, cache, lh, kind, sub0, nsub, slot)) {
                const CUtensorMap *map = kind ? &tm.b[cache] : &tm.a[cache];
                for (int t = 0; t < nsub; ++t, ++it) {
                    const int s = it % GT_STAGES;
                    const uint32_t ph = (it / GT_STAGES) & 1u;
                    if (!tc::mbar_wait(&bar_empty[s], ph ^ 1u, wc)) break;
                    tc::mbar_expect_tx(&bar_full[s], GT_TILE_BYTES);
                    const uint32_t dst = tc::smem_u32(tiles + s * GT_TILE_BYTES);
                    tc::tma_load_3d(dst, map, &bar_full[s], 0, (sub0 + t) * GT_TILE, lh);
                    tc::tma_load_3d(dst + GT_TILE_BYTES / 2, map, &bar_full[s], 64, (sub0 + t) * GT_TILE, lh);
                }
                if (s_abort) break;
            }
            // nothing this thread started may still be in flight when the block exits
            const uint32_t issued = it;
            for (uint32_t j = issued > (uint32_t)GT_STAGES ? issued - GT_STAGES : 0u; j < issued; ++j)
                tc::mbar_wait(&bar_full[j % GT_STAGES], (j / GT_STAGES) & 1u, wc);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t IDESC = tc::idesc_bf16(128, 128, 1, 1);
            TileRun run;
            run.init(p, blockIdx.x);
            int cache, lh, kind, sub0, nsub, slot;
            uint32_t it = 0, seg = 0;
            while (run.next(p, cache, lh, kind, sub0, nsub, slot)) {
                const uint32_t buf = seg & 1u;
                if (!tc::mbar_wait(&bar_acc_empty[buf], ((seg >> 1) & 1u) ^ 1u, wc)) break;
                tc::tc_fence_after();
                const uint32_t acc = tmem + buf * 128u;
                for (int t = 0; t < nsub; ++t, ++it) {
                    const int s = it % GT_STAGES;
                    if (!tc::mbar_wait(&bar_ready[s], (it / GT_STAGES) & 1u, wc)) break;
                    tc::tc_fence_after();
                    const uint32_t tile = tc::smem_u32(tiles + s * GT_TILE_BYTES);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        // 16 tokens per instruction: rows kk*16.. of the tile, both 64-column halves
                        const uint64_t dv = tc::smem_desc_sw128(tile + kk * 2048, GT_TILE_BYTES / 2, 1024);
                        tc::umma_bf16(acc, dv, dv, IDESC, (t > 0 || kk > 0) ? 1u : 0u);
                    }
                    tc::umma_commit(&bar_empty[s]);
                }
                tc::umma_commit(&bar_acc_full[buf]);
                ++seg;
                if (s_abort) break;
            }
        }
    } else if (warp < 2 + GT_FIX_THREADS / 32) {
        // ---------------- fix-up: zero retained rows, accumulate u ----------------
        // GT_GROUPS groups of four warps take the tiles of the run in turn, so that several tiles are
        // fixed up at the same time; each group keeps its own partial u.
        const int f = tid - 64;
        const int grp = f >> 7, fl = f & 127;      // group, thread within the group
        const int cg = fl & 15, rg = fl >> 4;      // 16-byte column group, row group (8 of them)
        const uint32_t col_off = (uint32_t)(cg >> 3) * (GT_TILE_BYTES / 2);
        float *u_red_g = u_red + grp * 8 * 128;
        const int bar_id = 1 + grp;
        // attention mass of token fl of a tile as k_select left it: -1 marks a retained token
        auto fetch = [&](const TileInfo &ti) -> float {
            if (ti.kind != 0) return 0.f;
            const CacheDev &c = p.c[ti.cache];
            const int j = ti.sub * GT_TILE + fl;
            if (j >= c.T) return 0.f;
            return __ldg(p.scores + c.tok_off + (size_t)ti.lh * c.T + j);
        };
        TileIter iter, ahead;
        iter.init(p, blockIdx.x);
        ahead.init(p, blockIdx.x);
        // the group looks at every tile of the run (to see where segments start and end) but fixes up
        // only tiles with index == grp (mod GT_GROUPS); the masses of its next tile are requested one tile early
        TileInfo cur, pre;
        bool has_cur = iter.next(p, cur);
        // `ahead` stands on the group's next own tile
        bool has_pre = true;
        for (int sk = 0; sk <= grp && has_pre; ++sk) has_pre = ahead.next(p, pre);
        float a_own = has_pre ? fetch(pre) : 0.f;   // mass for the group's next own tile
        uint32_t it = 0, n_own = 0;
        float u[8];
        float *s_ag = s_a + grp * 2 * 128;
        while (has_cur) {
            const bool own = (it % GT_GROUPS) == (uint32_t)grp;
            if (cur.first) {
#pragma unroll
                for (int e = 0; e < 8; ++e) u[e] = 0.f;
            }
            if (own) {
                const int s = it % GT_STAGES;
                float *sa = s_ag + (n_own & 1u) * 128;
                sa[fl] = a_own;
                // the group's next own tile: its masses are in flight while this tile is processed
                for (int sk = 0; sk < GT_GROUPS && has_pre; ++sk) has_pre = ahead.next(p, pre);
                if (has_pre) a_own = fetch(pre);
                tc::mbar_wait(&bar_full[s], (it / GT_STAGES) & 1u, wc);
                tc::named_barrier(bar_id, 128);        // sa is complete
                if (cur.kind == 0) {
                    uint8_t *tile = tiles + s * GT_TILE_BYTES + col_off;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int r = rg + 8 * i;
                        const float a = sa[r];
                        const bool kept = a < 0.f;
                        const float am = kept ? 0.f : a;
                        uint4 *ptr = reinterpret_cast<uint4 *>(tile + r * 128 + (((cg & 7) ^ (r & 7)) << 4));
                        const uint4 raw = *ptr;
                        if (kept) *ptr = make_uint4(0u, 0u, 0u, 0u);
                        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            u[2 * e] = fmaf(am, __uint_as_float(w[e] << 16), u[2 * e]);
                            u[2 * e + 1] = fmaf(am, __uint_as_float(w[e] & 0xFFFF0000u), u[2 * e + 1]);
                        }
                    }
                    tc::fence_async_smem();
                }
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&bar_ready[s]);
                ++n_own;
            }
            if (cur.kind == 0 && cur.last) {
                // the group's u over its 8 row groups, in a fixed order
                const int g = p.c[cur.cache].head_base + cur.lh;
                tc::named_barrier(bar_id, 128);
#pragma unroll
                for (int e = 0; e < 8; ++e) u_red_g[rg * 128 + cg * 8 + e] = u[e];
                tc::named_barrier(bar_id, 128);
                float sum = 0.f;
#pragma unroll
                for (int r = 0; r < 8; ++r) sum += u_red_g[r * 128 + fl];
                p.uvec[(((size_t)g * p.gram_slots + cur.slot) * GT_GROUPS + grp) * D + fl] = sum;
            }
            has_cur = iter.next(p, cur);
            ++it;
        }
    } else {
        // ---------------- epilogue: accumulator -> workspace ----------------
        const int q = warp & 3;                    // lane quarter this warp may read
        const int row = q * 32 + lane;
        TileRun run;
        run.init(p, blockIdx.x);
        int cache, lh, kind, sub0, nsub, slot;
        uint32_t seg = 0;
        while (run.next(p, cache, lh, kind, sub0, nsub, slot)) {
            const int g = p.c[cache].head_base + lh;
            const uint32_t buf = seg & 1u;
            tc::mbar_wait(&bar_acc_full[buf], (seg >> 1) & 1u, wc);
            tc::tc_fence_after();
            float *dst = (kind ? p.gram_k : p.gram_d) + ((size_t)g * p.gram_slots + slot) * D * D + (size_t)row * D;
#pragma unroll 1
            for (int cb = 0; cb < 4; ++cb) {
                uint32_t r[32];
                tc::tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + buf * 128u + cb * 32u, r);
                tc::tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    *reinterpret_cast<float4 *>(dst + cb * 32 + e * 4) =
                        make_float4(__uint_as_float(r[4 * e]), __uint_as_float(r[4 * e + 1]),
                                    __uint_as_float(r[4 * e + 2]), __uint_as_float(r[4 * e + 3]));
            }
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&bar_acc_empty[buf]);
            ++seg;
        }
    }

    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem, 256);
}

}  // namespace obf
