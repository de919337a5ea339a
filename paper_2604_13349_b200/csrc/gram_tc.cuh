// Tuned streaming pass of Orthogonal BackFill for bf16 caches with head_dim 128:
// one pass over V on the tensor cores that needs no selection result.
//
// With Q an orthonormal basis of the retained values' span and P = I - Q Q^T (Eq. 2-3), every
// retained row satisfies P v = 0.  Sums over the deleted rows may therefore run over ALL rows:
//   R^T R = P G_del P = P G_all P,          G_all = sum over all j of v_j v_j^T   (Eq. 3, Gram form of App. H)
//   r_bar = P u_del / (A_del + eps),        u_del = u_all - sum over retained j of A_j v_j,  u_all = sum_j A_j v_j   (Eq. 4)
// The pass produces G_all and u_all per (cache, layer, KV head) from V and the attention masses alone; the few
// retained rows are taken out of u (and out of the trace of G) by the dense algebra, which reads them anyway.
// It can thus run beside the selection and the gather instead of after them.
//
// (Whether span(V_keep) = R^d, Eq. 2, is decided by k_span_test from the gathered rows themselves.)
//
// Work decomposition.  Every head owns ceil(T / 128) tiles of 128 tokens of V.  All tiles of a launch form one sequence, cut into
// gridDim.x runs of `per` tiles; block b streams run b.  A run crosses head boundaries; each maximal stretch of
// one head inside a run is a segment and yields one partial Gram matrix (and one partial u), stored in slot
// (b - first block touching that head).
//
// Block = 10 warps:
//   warp 0       TMA producer: 128 x 128 bf16 tiles (two 128-byte-swizzled column halves) into a ring
//   warp 1       issues tcgen05.mma: [G | u] (+)= tile^T [tile | a] in ONE instruction per 16 tokens (N = 144): the
//                B operand is the value tile followed, as a third 64-column block of the same MN-major layout, by
//                the tile's 128 masses as bf16 columns: high, middle and low part of the fp32 mass (their sum is
//                the mass exactly, and bf16 x bf16 products are exact in fp32), so that the CUDA cores never read
//                a value tile; the three columns exist once per mass level (common.cuh: u_level), a token filling
//                those of its own level; accumulators double-buffered in tensor memory
//   warps 2..4   masses: warp w serves ring stage w; it fetches the 128 masses of its next tile early, splits them
//                and writes the columns into the stage's mass block (rows of 128 bytes, 128-byte swizzle)
//   warps 6..9   epilogue: tensor memory -> partial Gram matrix and partial u in the workspace
#pragma once

#include "tc_common.cuh"

namespace obf {

constexpr int GT_STAGES = 3;
constexpr int GT_TILE = 128;                       // tokens per tile
constexpr int GT_TILE_BYTES = GT_TILE * 128 * 2;   // 32 KiB
constexpr int GT_ABLOCK_BYTES = GT_TILE * 128;     // mass block: [128 tokens][64 columns] bf16 like a column block of the tile; columns 3 * level + part in use
constexpr int GT_STAGE_BYTES = GT_TILE_BYTES + GT_ABLOCK_BYTES;   // the mass block sits right behind its value tile
constexpr int GT_NU = 16;                          // columns of the mass block that enter the MMA
static_assert(3 * U_LEVELS <= GT_NU, "the mass columns must fit the MMA's extra columns");
constexpr int GT_THREADS = 64 + 128 + 128;
constexpr size_t GT_SMEM_BYTES = 1024 + (size_t)GT_STAGES * GT_STAGE_BYTES + 64;
constexpr uint32_t GT_TMEM_COLS = 512;             // 2 accumulators of 128 + 16 columns at a stride of 256
constexpr uint32_t GT_TMEM_STRIDE = 256;

// Walks the segments of one block's run of tiles.
struct TileRun {
    long long pos, end;        // current and one-past-last index in the launch-wide tile sequence
    int ci, per;
    __device__ __forceinline__ void init(const CallDev &p, int block)
    {
        per = p.tc_per;
        const long long total = p.tc_total_sub;
        pos = (long long)block * per;
        end = pos + per;
        if (end > total) end = total;
        ci = 0;
    }
    __device__ __forceinline__ long long base_of(const CacheDev &c) const { return c.sub_base; }
    // Next segment: cache, local head, first tile, tile count, partial slot.
    __device__ __forceinline__ bool next(const CallDev &p, int &cache, int &lh, int &sub0, int &nsub, int &slot)
    {
        for (;;) {
            if (pos >= end) return false;
            while (ci + 1 < p.n_caches && pos >= base_of(p.c[ci + 1])) ++ci;
            const CacheDev &c = p.c[ci];
            const int per_head = c.nsub_del;
            const long long rel = pos - base_of(c);
            lh = (int)(rel / per_head);
            sub0 = (int)(rel - (long long)lh * per_head);
            const int left_in_seg = per_head - sub0;
            const long long left_in_run = end - pos;
            nsub = left_in_seg < left_in_run ? left_in_seg : (int)left_in_run;
            const long long seg_start = pos - sub0;
            slot = (int)(pos / per - seg_start / per);
            cache = ci;
            pos += nsub;
            // the span test ran first and found this head's retained values to span R^d: nothing of it is needed
            // (every role of the block walks the segments through here and skips the same ones)
            if (p.skip_full && (p.hflag[c.head_base + lh] & HFLAG_SPAN_FULL)) continue;
            return true;
        }
    }
};

// G_all and u_all from V.
// One block per multiprocessor; the launch bound of three only caps the registers at 64 per thread, so that the
// blocks of the selection and the gather, which run on a side stream at the same time, find registers beside it.
__global__ void __launch_bounds__(GT_THREADS, 3) k_gram_tc(const __grid_constant__ CallDev p, const __grid_constant__ TcMaps tm)
{
    constexpr int D = 128;
    extern __shared__ uint8_t gt_smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(gt_smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *tiles = base;                                                // GT_STAGES x (32 KiB tile + 16 KiB mass block), 1024-byte aligned
    __shared__ uint64_t bar_full[GT_STAGES], bar_ready[GT_STAGES], bar_empty[GT_STAGES];
    __shared__ uint64_t bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t s_tmem, s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    tc::WaitCtx wc{&s_abort, p.status, p.wait_limit_ns};

    if (tid == 0) {
        s_abort = 0u;
        for (int s = 0; s < GT_STAGES; ++s) {
            tc::mbar_init(&bar_full[s], 1);
            tc::mbar_init(&bar_ready[s], 1);
            tc::mbar_init(&bar_empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) { tc::mbar_init(&bar_acc_full[b], 1); tc::mbar_init(&bar_acc_empty[b], 4); }
        tc::mbar_init_fence();
    }
    if (warp == 1) tc::tmem_alloc(&s_tmem, GT_TMEM_COLS);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = s_tmem;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            TileRun run;
            run.init(p, blockIdx.x);
            int cache, lh, sub0, nsub, slot;
            uint32_t it = 0;
            while (run.next(p, cache, lh, sub0, nsub, slot)) {
                const CUtensorMap *map = &tm.a[cache];
                for (int t = 0; t < nsub; ++t, ++it) {
                    const int s = it % GT_STAGES;
                    const uint32_t ph = (it / GT_STAGES) & 1u;
                    if (!tc::mbar_wait(&bar_empty[s], ph ^ 1u, wc)) break;
                    tc::mbar_expect_tx(&bar_full[s], GT_TILE_BYTES);
                    const uint32_t dst = tc::smem_u32(tiles + s * GT_STAGE_BYTES);
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
            constexpr uint32_t idesc = tc::idesc_bf16(128, 128 + GT_NU, 1, 1);
            TileRun run;
            run.init(p, blockIdx.x);
            int cache, lh, sub0, nsub, slot;
            uint32_t it = 0, seg = 0;
            bool dead = false;
            while (!dead && run.next(p, cache, lh, sub0, nsub, slot)) {
                const uint32_t buf = seg & 1u;
                if (!tc::mbar_wait(&bar_acc_empty[buf], ((seg >> 1) & 1u) ^ 1u, wc)) break;
                tc::tc_fence_after();
                const uint32_t acc = tmem + buf * GT_TMEM_STRIDE;
                for (int t = 0; t < nsub; ++t, ++it) {
                    const int s = it % GT_STAGES;
                    const uint32_t ph = (it / GT_STAGES) & 1u;
                    if (!tc::mbar_wait(&bar_full[s], ph, wc)) { dead = true; break; }
                    if (!tc::mbar_wait(&bar_ready[s], ph, wc)) { dead = true; break; }
                    tc::tc_fence_after();
                    const uint32_t tile = tc::smem_u32(tiles + s * GT_STAGE_BYTES);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        // 16 tokens per instruction: rows kk*16.. of the tile; the column blocks of 64 follow one another
                        // at 16 KiB: two of the value tile and, for the B operand, the mass block
                        const uint64_t dv = tc::smem_desc_sw128(tile + kk * 2048, GT_TILE_BYTES / 2, 1024);
                        tc::umma_bf16(acc, dv, dv, idesc, (t > 0 || kk > 0) ? 1u : 0u);
                    }
                    tc::umma_commit(&bar_empty[s]);
                }
                if (dead) break;
                tc::umma_commit(&bar_acc_full[buf]);
                ++seg;
                if (s_abort) break;
            }
        }
    } else if (warp < 6) {
        // ---------------- masses: three bf16 columns per level and tile ----------------
        // One warp per ring stage, each on its own: warp w serves the tiles with index w (mod GT_STAGES), so that the
        // masses of several tiles are under way at once (one tile costs a round trip to the stage's barrier, the
        // stores and a proxy fence).
        const int mw = warp - 2;
        if (mw < GT_STAGES) {
            TileRun run;
            run.init(p, blockIdx.x);
            int cache, lh, sub0, nsub, slot;
            // position of the walk: tile `t` of the current segment, `it` in the run
            bool have = run.next(p, cache, lh, sub0, nsub, slot);
            int t = 0;
            uint32_t it = 0;
            auto step = [&]() {
                ++it;
                if (++t >= nsub) { have = run.next(p, cache, lh, sub0, nsub, slot); t = 0; }
            };
            // moves the walk to this warp's next tile at or after the current position
            auto seek = [&]() {
                while (have && (it % GT_STAGES) != (uint32_t)mw) step();
            };
            // masses of tokens lane, lane + 32, .. of the tile the walk stands on
            auto fetch = [&](float (&a)[4]) {
                const CacheDev &c = p.c[cache];
                const float *A = p.scores + c.tok_off + (size_t)lh * c.T;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int j = (sub0 + t) * GT_TILE + lane + 32 * e;
                    a[e] = j < c.T ? __ldg(A + j) : 0.f;
                }
            };
            seek();
            float a_next[4] = {0.f, 0.f, 0.f, 0.f};
            if (have) fetch(a_next);
            uint8_t *ab = tiles + mw * GT_STAGE_BYTES + GT_TILE_BYTES;     // this stage's mass block
            while (have) {
                float a[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) a[e] = a_next[e];
                const uint32_t ph = (it / GT_STAGES) & 1u;
                // this warp's next tile: its masses are in flight while the current ones are written
                step();
                seek();
                if (have) fetch(a_next);
                if (!tc::mbar_wait(&bar_empty[mw], ph ^ 1u, wc)) break;   // the stage's last user is done with its mass block
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int k = lane + 32 * e;
                    const __nv_bfloat16 hi = __float2bfloat16_rn(a[e]);
                    const float r1 = a[e] - __bfloat162float(hi);
                    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
                    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
                    const uint32_t part[3] = {(uint32_t)__bfloat16_as_ushort(hi), (uint32_t)__bfloat16_as_ushort(mid),
                                              (uint32_t)__bfloat16_as_ushort(lo)};
                    const int lev = u_level(a[e]);
                    // columns 0..15 of the token's row: column 3 * lev + i holds part i, the others zero
                    uint32_t w[8];
#pragma unroll
                    for (int n2 = 0; n2 < 8; ++n2) {
                        const int n0 = 2 * n2, n1 = 2 * n2 + 1;
                        const uint32_t v0 = (n0 / 3 == lev && n0 < 3 * U_LEVELS) ? part[n0 % 3] : 0u;
                        const uint32_t v1 = (n1 / 3 == lev && n1 < 3 * U_LEVELS) ? part[n1 % 3] : 0u;
                        w[n2] = v0 | (v1 << 16);
                    }
                    // the two 16-byte chunks of columns 0..7 and 8..15 sit at chunk (0 or 1) XOR (token mod 8) of the row
                    uint8_t *rowp = ab + k * 128;
                    *reinterpret_cast<uint4 *>(rowp + ((0 ^ (k & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    *reinterpret_cast<uint4 *>(rowp + ((1 ^ (k & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
                }
                tc::fence_async_smem();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&bar_ready[mw]);
            }
        }
    } else {
        // ---------------- epilogue: accumulators -> workspace ----------------
        const int q = warp & 3;                    // lane quarter this warp may read
        const int row = q * 32 + lane;
        TileRun run;
        run.init(p, blockIdx.x);
        int cache, lh, sub0, nsub, slot;
        uint32_t seg = 0;
        while (run.next(p, cache, lh, sub0, nsub, slot)) {
            const int g = p.c[cache].head_base + lh;
            const uint32_t buf = seg & 1u;
            if (!tc::mbar_wait(&bar_acc_full[buf], (seg >> 1) & 1u, wc)) break;
            tc::tc_fence_after();
            const uint32_t tl = tmem + ((uint32_t)(q * 32) << 16);
            float *dst = p.gram_d + ((size_t)g * p.gram_slots + slot) * D * D + (size_t)row * D;
#pragma unroll 1
            for (int cb = 0; cb < 4; ++cb) {
                uint32_t r[32];
                tc::tmem_ld32(tl + buf * GT_TMEM_STRIDE + cb * 32u, r);
                tc::tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    *reinterpret_cast<float4 *>(dst + cb * 32 + e * 4) =
                        make_float4(__uint_as_float(r[4 * e]), __uint_as_float(r[4 * e + 1]),
                                    __uint_as_float(r[4 * e + 2]), __uint_as_float(r[4 * e + 3]));
            }
            {
                // u of value channel `row`, per mass level: three columns add up the products with the three parts of the masses
                uint32_t r[32];
                tc::tmem_ld32(tl + buf * GT_TMEM_STRIDE + 128u, r);
                tc::tmem_ld_wait();
#pragma unroll
                for (int l = 0; l < U_LEVELS; ++l)
                    p.uvec[(((size_t)g * p.gram_slots + slot) * U_LEVELS + l) * D + row] =
                        (__uint_as_float(r[3 * l]) + __uint_as_float(r[3 * l + 1])) + __uint_as_float(r[3 * l + 2]);
            }
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&bar_acc_empty[buf]);
            ++seg;
        }
    }

    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem, GT_TMEM_COLS);
}

}  // namespace obf
