// Host side of the C ABI declared in include/obf.h: argument validation,
// workspace layout, kernel dispatch.  Allocates no device memory.
#include <atomic>
#include <cstdio>
#include <cstring>

#include "algebra.cuh"
#include "common.cuh"
#include "generic.cuh"
#include "gram_tc.cuh"
#include "merge.cuh"
#include "score_tc.cuh"
#include "span_test.cuh"

namespace obf {

static thread_local int32_t g_last_launches = 0;
static thread_local bool g_keep_status = false;

// Optional per-launch timing (obf_compress_profiled): an event after every launch.
struct Profiler {
    cudaEvent_t ev[OBF_MAX_PHASES + 1];
    const char *names[OBF_MAX_PHASES];
    int n = 0;
    bool active = false;
};
static thread_local Profiler g_prof;
static thread_local const char *g_phase_names[OBF_MAX_PHASES];
static thread_local int g_phase_count = 0;

// A second stream per host thread and device for work that may overlap the main stream's, with the two events
// of the fork and the join.  Created on first use; no device memory is involved.
struct SideStream {
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, rows_done = nullptr, join = nullptr;
    int device = -1;
};

static SideStream *side_stream()
{
    static thread_local SideStream ss[16];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 16) return nullptr;
    SideStream &s = ss[dev];
    if (s.device != dev) {
        if (cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&s.join, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&s.rows_done, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        s.device = dev;
    }
    return &s;
}

static inline void mark(cudaStream_t st, const char *name)
{
    ++g_last_launches;
    if (g_prof.active && g_prof.n < OBF_MAX_PHASES) {
        g_prof.names[g_prof.n] = name;
        cudaEventRecord(g_prof.ev[++g_prof.n], st);
    }
}

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
    size_t off_status, off_scores, off_keep, off_stats, off_sums, off_lscores, off_scores2;
    size_t off_gram_d, off_gram_k, off_uvec, off_delta, off_hflag, off_svec, off_assign;
    size_t total;
    int splits;
    int heads_total;
    size_t tok_total;
    size_t tok_off[OBF_MAX_CACHES];
    // tuned bf16 / head_dim 128 path
    bool tuned;
    int gram_slots;                 // partial Gram matrices stored per head
    int tc_per, tc_blocks;          // tiles per block and blocks of the tensor-core pass over V
    long long tc_total_sub;
    int nsub_del[OBF_MAX_CACHES];
    long long sub_base[OBF_MAX_CACHES];
    // tensor-core score kernel
    bool sc_on;
    int sc_nq, sc_subs, sc_blocks, sc_rounds, sc_qt;
    int sc_team[OBF_MAX_CACHES], sc_hpr[OBF_MAX_CACHES], sc_round_base[OBF_MAX_CACHES];
    size_t sc_part_off[OBF_MAX_CACHES], sc_part_pairs;
    size_t off_sc_part, off_sc_head, off_sc_sync;
};

// Streaming multiprocessors of the current device (148 on a B200 when no device can be asked).
static int sm_count()
{
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return 148; }
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = 148;
        }
        cached[dev] = n;
    }
    return cached[dev];
}

// The tensor-core kernels cover bf16 caches with head_dim 128 and at least one full 128-token tile.
static bool tuned_path_applies(const obf_params_t *p, const obf_cache_t *caches, int32_t n)
{
    if (p->dtype != OBF_BF16 || p->head_dim != 128 || (p->flags & OBF_FLAG_GENERIC_PATH)) return false;
    for (int i = 0; i < n; ++i)
        if (caches[i].T < GT_TILE) return false;
    return true;
}

static int choose_splits(int heads_total, int T_max)
{
    int s = (2 * 148 + heads_total - 1) / heads_total;
    const int tiles = (T_max + GR_ROWS - 1) / GR_ROWS;
    if (s > tiles) s = tiles;
    if (s > 16) s = 16;
    if (s < 1) s = 1;
    return s;
}

// Retained positions of a cache: the protected prefix plus at most `budget` of the other positions.
static inline int k_eff_of(const obf_params_t *p, const obf_cache_t &c)
{
    const int s = (int)OBF_FLAG_SINK_OF(p->flags) < c.T ? (int)OBF_FLAG_SINK_OF(p->flags) : c.T;
    return s + (c.budget < c.T - s ? c.budget : c.T - s);
}

static obf_status_t validate_shapes(const obf_params_t *p, const obf_cache_t *caches, int32_t n, int rank)
{
    if (!p || !caches) return OBF_ERR_INVALID_ARG;
    if (n < 1) return OBF_ERR_INVALID_ARG;
    if (n > OBF_MAX_CACHES) return OBF_ERR_UNSUPPORTED;
    if (p->layers < 1 || p->kv_heads < 1 || p->q_heads < 1 || p->n_obs < 1) return OBF_ERR_INVALID_ARG;
    if (p->q_heads % p->kv_heads != 0) return OBF_ERR_INVALID_ARG;
    if (p->head_dim != 64 && p->head_dim != 128) return OBF_ERR_UNSUPPORTED;
    if (p->dtype != OBF_F32 && p->dtype != OBF_BF16) return OBF_ERR_UNSUPPORTED;
    if (rank < 0 || rank > p->head_dim) return OBF_ERR_INVALID_ARG;
    if (!(p->eps >= 0.f)) return OBF_ERR_INVALID_ARG;
    if ((long long)p->layers * p->kv_heads * n > (1 << 24)) return OBF_ERR_UNSUPPORTED;
    for (int i = 0; i < n; ++i) {
        if (caches[i].T < 1 || caches[i].T > OBF_MAX_T) return OBF_ERR_INVALID_ARG;
        if (caches[i].budget < 1) return OBF_ERR_INVALID_ARG;
        // the layerwise selector keeps a layer's summed masses in shared memory
        if ((p->flags & OBF_FLAG_LAYERWISE) && caches[i].T > SEL_SMEM_MAX_T) return OBF_ERR_UNSUPPORTED;
    }
    return OBF_OK;
}

static void make_layout(const obf_params_t *p, const obf_cache_t *caches, int32_t n, int rank, Layout &L)
{
    const int hpc = p->layers * p->kv_heads;
    const int d = p->head_dim;
    const int n_q = (p->q_heads / p->kv_heads) * p->n_obs;
    L.heads_total = hpc * n;
    size_t tok = 0;
    int T_max = 1;
    for (int i = 0; i < n; ++i) {
        L.tok_off[i] = tok;
        tok += (size_t)hpc * caches[i].T;
        if (caches[i].T > T_max) T_max = caches[i].T;
    }
    L.tok_total = tok;
    L.splits = choose_splits(L.heads_total, T_max);
    L.tuned = tuned_path_applies(p, caches, n);
    L.gram_slots = L.splits;
    L.tc_per = 0; L.tc_blocks = 0; L.tc_total_sub = 0;
    if (L.tuned && rank > 0) {
        long long total = 0;
        for (int i = 0; i < n; ++i) {
            L.nsub_del[i] = (caches[i].T + GT_TILE - 1) / GT_TILE;
            L.sub_base[i] = total;
            total += (long long)hpc * L.nsub_del[i];
        }
        const long long sms = sm_count();
        const long long want = total < sms ? total : sms;
        L.tc_total_sub = total;
        L.tc_per = (int)((total + want - 1) / want);
        L.tc_blocks = (int)((total + L.tc_per - 1) / L.tc_per);
        int slots = 1;
        for (int i = 0; i < n; ++i) {
            const int a = (L.nsub_del[i] + L.tc_per - 1) / L.tc_per + 1;
            if (a > slots) slots = a;
        }
        L.gram_slots = slots;
    }
    L.sc_on = false;
    L.sc_nq = L.sc_subs = L.sc_blocks = L.sc_rounds = 0;
    L.sc_qt = 1;
    L.sc_part_pairs = 0;
    if (L.tuned && n_q <= ST_MAX_NQ) {
        // more than 128 query rows per head: two work items per head, one per 128 rows
        L.sc_qt = (n_q + 127) / 128;
        const int hpc_real = hpc;
        const int hpc = hpc_real * L.sc_qt;
        // chunks of ST_TILES 128-key tiles, one per block and round; a head's team must fit in one round
        L.sc_nq = 128;
        L.sc_subs = ST_TILES;
        long long blocks_wanted = 0;
        for (int i = 0; i < n; ++i) {
            L.sc_team[i] = (caches[i].T + ST_CHUNK - 1) / ST_CHUNK;
            blocks_wanted += (long long)hpc * L.sc_team[i];
        }
        const long long sms = sm_count();
        L.sc_blocks = (int)(blocks_wanted < sms ? blocks_wanted : sms);
        bool fits = true;
        int rounds = 0;
        size_t pairs = 0;
        for (int i = 0; i < n; ++i) {
            if (L.sc_team[i] > L.sc_blocks) { fits = false; break; }
            L.sc_hpr[i] = L.sc_blocks / L.sc_team[i];
            if (L.sc_hpr[i] > hpc) L.sc_hpr[i] = hpc;
            L.sc_round_base[i] = rounds;
            rounds += (hpc + L.sc_hpr[i] - 1) / L.sc_hpr[i];
            L.sc_part_off[i] = pairs;
            pairs += (size_t)hpc * L.sc_team[i] * 128;
        }
        L.sc_on = fits;
        L.sc_rounds = rounds;
        L.sc_part_pairs = pairs;
    }
    size_t o = 0;
    L.off_status = o; o += 256;
    L.off_scores = o; o = align_up(o + tok * sizeof(float), 256);
    L.off_keep = o;   o = align_up(o + tok, 256);
    L.off_stats = o;  o = align_up(o + (size_t)L.heads_total * n_q * 2 * sizeof(float), 256);
    L.off_sums = o;   o = align_up(o + (size_t)L.heads_total * 4 * sizeof(float), 256);
    L.off_scores2 = o;
    if (L.sc_on && L.sc_qt == 2) o = align_up(o + tok * sizeof(float), 256);
    L.off_lscores = o;
    if (p->flags & OBF_FLAG_LAYERWISE) o = align_up(o + tok / p->kv_heads * sizeof(float), 256);
    L.off_sc_part = L.off_sc_head = L.off_sc_sync = o;
    if (L.sc_on) {
        L.off_sc_part = o; o = align_up(o + L.sc_part_pairs * 2 * sizeof(float), 256);
        // sc_head and sc_cnt are cleared together before every launch
        L.off_sc_head = o; o = align_up(o + (size_t)L.heads_total * L.sc_qt * 128 * sizeof(unsigned long long), 256);
        L.off_sc_sync = o; o = align_up(o + (size_t)L.heads_total * L.sc_qt * sizeof(uint32_t), 256);
    }
    L.off_gram_d = L.off_gram_k = L.off_uvec = L.off_delta = L.off_hflag = L.off_svec = o;
    if (rank > 0) {
        const size_t gsz = (size_t)L.heads_total * L.gram_slots * d * d * sizeof(float);
        L.off_gram_d = o; o = align_up(o + gsz, 256);
        L.off_gram_k = o; if (!L.tc_per) o = align_up(o + gsz, 256);   // the tuned path forms G_keep inside the span test
        L.off_uvec = o;   o = align_up(o + (size_t)L.heads_total * L.gram_slots * (L.tc_per ? U_LEVELS : 1) * d * sizeof(float), 256);
        L.off_delta = o;  o = align_up(o + (size_t)L.heads_total * d * sizeof(float), 256);
        L.off_hflag = o;  o = align_up(o + (size_t)L.heads_total * sizeof(uint32_t), 256);
        L.off_svec = o;   o = align_up(o + (size_t)L.heads_total * d * sizeof(float), 256);
    }
    L.off_assign = o;
    if (p->flags & OBF_FLAG_MERGE) o = align_up(o + tok * sizeof(int32_t), 256);
    L.total = o;
}

static bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

#define OBF_CUDA_TRY(expr)                                                        \
    do {                                                                          \
        cudaError_t e_ = (expr);                                                  \
        if (e_ != cudaSuccess) {                                                  \
            std::fprintf(stderr, "obf: %s failed: %s\n", #expr, cudaGetErrorString(e_)); \
            return OBF_ERR_CUDA;                                                  \
        }                                                                         \
    } while (0)

template <typename K>
static obf_status_t set_smem(K kernel, size_t bytes)
{
    OBF_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    OBF_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared));
    return OBF_OK;
}

// cuTensorMapEncodeTiled, looked up through the runtime so that the library does not link the driver.
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn tensor_map_encoder()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return nullptr;
        }
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// Tensor map of a bf16 array [heads, rows, 128] for box_rows x 64-column boxes with the
// 128-byte swizzle; rows past `rows` read as zero.
static obf_status_t encode_rows_map(CUtensorMap *m, const void *ptr, uint64_t rows, uint64_t heads, uint32_t box_rows = GT_TILE)
{
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return OBF_ERR_CUDA;
    cuuint64_t dims[3] = {128, rows, heads};
    cuuint64_t strides[2] = {128 * 2, rows * 128 * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t es[3] = {1, 1, 1};
    const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        std::fprintf(stderr, "obf: cuTensorMapEncodeTiled failed with %d\n", (int)r);
        return OBF_ERR_CUDA;
    }
    return OBF_OK;
}

// Streaming pass of OBF on the tensor cores (bf16, head_dim 128): Gram matrix and mass-weighted sum over all rows
// of V (needs the masses, not the selection).
static obf_status_t launch_gram_tc(const CallDev &cd, const Layout &L, cudaStream_t st)
{
    static thread_local TcMaps m;
    if (L.tc_blocks == 0) return OBF_OK;
    const uint64_t hpc = (uint64_t)cd.heads_per_cache;
    for (int i = 0; i < cd.n_caches; ++i) {
        const obf_status_t s = encode_rows_map(&m.a[i], cd.c[i].v, (uint64_t)cd.c[i].T, hpc);
        if (s != OBF_OK) return s;
    }
    OBF_CUDA_TRY(cudaFuncSetAttribute(k_gram_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GT_SMEM_BYTES));
    // the whole shared-memory capacity, so that the side stream's blocks find room beside this kernel's
    OBF_CUDA_TRY(cudaFuncSetAttribute(k_gram_tc, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared));
    k_gram_tc<<<L.tc_blocks, GT_THREADS, GT_SMEM_BYTES, st>>>(cd, m);
    mark(st, "k_gram_tc");
    return OBF_OK;
}

// Attention mass on the tensor cores (bf16, head_dim 128): one persistent launch.
static obf_status_t launch_score_tc(const CallDev &cd, const Layout &L, cudaStream_t st)
{
    static thread_local TcMaps maps;
    const uint64_t hpc = (uint64_t)cd.heads_per_cache;
    for (int i = 0; i < cd.n_caches; ++i) {
        obf_status_t s = encode_rows_map(&maps.a[i], cd.c[i].k, (uint64_t)cd.c[i].T, hpc);
        if (s != OBF_OK) return s;
        if ((s = encode_rows_map(&maps.b[i], cd.c[i].q, (uint64_t)cd.n_q, hpc)) != OBF_OK) return s;
    }
    const size_t smem = ST_SMEM_BYTES;
    OBF_CUDA_TRY(cudaFuncSetAttribute(k_score_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    OBF_CUDA_TRY(cudaMemsetAsync(cd.sc_head, 0, (L.off_sc_sync - L.off_sc_head) + (size_t)cd.heads_total * L.sc_qt * sizeof(uint32_t), st));
    // The blocks of a head's team wait for one another, so the whole grid has to be resident at once: a
    // cooperative launch starts only when it is (the grid never exceeds one block per multiprocessor).
    void *args[2] = {const_cast<CallDev *>(&cd), &maps};
    OBF_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(k_score_tc), dim3(L.sc_blocks), dim3(ST_THREADS),
                                             args, smem, st));
    mark(st, "k_score_tc");
    if (L.sc_qt == 2) {
        int T_max = 1;
        for (int i = 0; i < cd.n_caches; ++i) T_max = cd.c[i].T > T_max ? cd.c[i].T : T_max;
        dim3 gj((T_max + 255) / 256, cd.heads_total);
        k_score_join<<<gj, 256, 0, st>>>(cd);
        mark(st, "k_score_join");
    }
    return OBF_OK;
}

template <typename TIN, int D>
static obf_status_t launch_generic(const CallDev &cd, const Layout &L, int T_max, int k_max, cudaStream_t st)
{
    const int heads = cd.heads_total;
    const size_t sm_sc = score_smem_bytes<D>();
    obf_status_t s;
    if (L.sc_on) {
        if ((s = launch_score_tc(cd, L, st)) != OBF_OK) return s;
    } else {
        if ((s = set_smem(k_score_stats<TIN, D>, sm_sc)) != OBF_OK) return s;
        if ((s = set_smem(k_score_pool<TIN, D>, sm_sc)) != OBF_OK) return s;
        dim3 g1((cd.n_q + SC_TILE - 1) / SC_TILE, heads);
        k_score_stats<TIN, D><<<g1, SC_NT, sm_sc, st>>>(cd);
        mark(st, "k_score_stats");
        dim3 g2((T_max + SC_TILE - 1) / SC_TILE, heads);
        k_score_pool<TIN, D><<<g2, SC_NT, sm_sc, st>>>(cd);
        mark(st, "k_score_pool");
    }
    // The tuned pass over V needs the masses but not the selection (it sums over all rows, gram_tc.cuh): it runs
    // on the caller's stream while selection and gather run on a side stream of the library.  (Not while
    // profiling per launch, where every kernel is timed alone.)
    const bool tuned_obf = cd.rank > 0 && L.tc_per > 0;
    // With OBF_FLAG_EARLY_OUT the span test comes first and the pass over V skips what it found full: one stream.
    SideStream *side = (tuned_obf && !g_prof.active && !cd.skip_full) ? side_stream() : nullptr;
    cudaStream_t sel = side ? side->stream : st;       // stream of selection and gather
    if (side) {
        OBF_CUDA_TRY(cudaEventRecord(side->fork, st));
        OBF_CUDA_TRY(cudaStreamWaitEvent(side->stream, side->fork, 0));
        if ((s = launch_gram_tc(cd, L, st)) != OBF_OK) return s;
    }
    if (cd.layerwise) {
        // masses of a layer's KV heads added up, then every head's block selects on its layer's sums
        const int n_layers = heads / cd.kv_heads;
        const size_t sm_sel = (size_t)T_max * sizeof(uint32_t);
        dim3 gl((T_max + 255) / 256, n_layers);
        k_layer_sum<<<gl, 256, 0, sel>>>(cd);
        mark(sel, "k_layer_sum");
        const int sms = sm_count();
        if (heads > 2 * sms && heads <= 4 * sms) {
            if ((s = set_smem(k_select_smem<512, true>, sm_sel)) != OBF_OK) return s;
            k_select_smem<512, true><<<heads, 512, sm_sel, sel>>>(cd);
        } else {
            if ((s = set_smem(k_select_smem<1024, true>, sm_sel)) != OBF_OK) return s;
            k_select_smem<1024, true><<<heads, 1024, sm_sel, sel>>>(cd);
        }
    } else if (T_max <= SEL_SMEM_MAX_T) {
        const size_t sm_sel = (size_t)T_max * sizeof(uint32_t);
        // blocks of 1024 threads fit twice on an SM; when the heads then need a second, nearly empty wave,
        // blocks of 512 threads (four per SM) finish sooner
        const int sms = sm_count();
        if (heads > 2 * sms && heads <= 4 * sms) {
            if ((s = set_smem(k_select_smem<512>, sm_sel)) != OBF_OK) return s;
            k_select_smem<512><<<heads, 512, sm_sel, sel>>>(cd);
        } else {
            if ((s = set_smem(k_select_smem<1024>, sm_sel)) != OBF_OK) return s;
            k_select_smem<1024><<<heads, 1024, sm_sel, sel>>>(cd);
        }
    } else {
        k_select<<<heads, SEL_NT, 0, sel>>>(cd);
    }
    mark(sel, "k_select");
    dim3 g4((k_max + GATHER_ROWS - 1) / GATHER_ROWS, heads);
    if (side) {
        // the values first: the rest of the call needs them
        k_gather<D * (int)sizeof(TIN), 1><<<g4, 256, 0, sel>>>(cd);
        mark(sel, "k_gather");
        OBF_CUDA_TRY(cudaEventRecord(side->rows_done, side->stream));
        if constexpr (sizeof(TIN) == 2 && D == 128) {
            // the span test reads the gathered rows only (it forms G_keep itself): it runs here, beside the pass over
            // V, whose persistent blocks leave room for one of its blocks per multiprocessor
            const size_t sm_span = span_smem_bytes<D>();
            if ((s = set_smem(k_span_test<D, true>, sm_span)) != OBF_OK) return s;
            k_span_test<D, true><<<heads, ST_NT, sm_span, sel>>>(cd);
            mark(sel, "k_span_test");
        }
        OBF_CUDA_TRY(cudaEventRecord(side->join, side->stream));
        // the keys are needed by nothing that follows: they are copied on the caller's stream once the pass over V
        // is over (it is bound by HBM), while the span test finishes on the side stream
        OBF_CUDA_TRY(cudaStreamWaitEvent(st, side->rows_done, 0));
        k_gather<D * (int)sizeof(TIN), 2><<<g4, 256, 0, st>>>(cd);
        ++g_last_launches;
        OBF_CUDA_TRY(cudaStreamWaitEvent(st, side->join, 0));
    } else {
        k_gather<D * (int)sizeof(TIN)><<<g4, 256, 0, sel>>>(cd);
        mark(sel, "k_gather");
    }
    if (cd.rank > 0) {
        const size_t sm_alg = algebra_smem_bytes<D>(cd.alg_rows, cd.rank, cd.fast_iters);
        if ((s = set_smem(k_obf_algebra<TIN, D>, sm_alg)) != OBF_OK) return s;
        if (tuned_obf) {
            if constexpr (sizeof(TIN) == 2 && D == 128) {
                if (cd.skip_full) {
                    // the span test before the pass over V, which then skips the heads whose retained values span R^d
                    const size_t sm_span0 = span_smem_bytes<D>();
                    if ((s = set_smem(k_span_test<D, true>, sm_span0)) != OBF_OK) return s;
                    k_span_test<D, true><<<heads, ST_NT, sm_span0, st>>>(cd);
                    mark(st, "k_span_test");
                }
            }
            if (!side && (s = launch_gram_tc(cd, L, st)) != OBF_OK) return s;
        } else {
            dim3 g5(cd.splits, heads);
            k_gram<TIN, D><<<g5, 256, 0, st>>>(cd);
            mark(st, "k_gram");
        }
        bool any_diag = false;
        for (int i = 0; i < cd.n_caches; ++i) any_diag = any_diag || cd.c[i].diag != nullptr;
        if (any_diag) {
            // the projection cosine of the diagnostics needs the plain sum of the deleted values: one more pass over V
            OBF_CUDA_TRY(cudaMemsetAsync(cd.svec, 0, (size_t)heads * D * sizeof(float), st));
            dim3 gv((T_max + 2047) / 2048, heads);
            k_vsum<TIN, D><<<gv, 256, 0, st>>>(cd);
            mark(st, "k_vsum");
        }
        const size_t sm_span = span_smem_bytes<D>();
        if (side || cd.skip_full) {
            // the span test has been enqueued already: on the side stream (this stream has waited for it) or, with
            // OBF_FLAG_EARLY_OUT, before the pass over V
        } else if constexpr (sizeof(TIN) == 2 && D == 128) {
            if (tuned_obf) {
                // the tuned path forms G_keep inside the span test, from the gathered rows
                if ((s = set_smem(k_span_test<D, true>, sm_span)) != OBF_OK) return s;
                k_span_test<D, true><<<heads, ST_NT, sm_span, st>>>(cd);
            } else {
                if ((s = set_smem(k_span_test<D>, sm_span)) != OBF_OK) return s;
                k_span_test<D><<<heads, ST_NT, sm_span, st>>>(cd);
            }
        } else {
            if ((s = set_smem(k_span_test<D>, sm_span)) != OBF_OK) return s;
            k_span_test<D><<<heads, ST_NT, sm_span, st>>>(cd);
        }
        if (!side && !cd.skip_full) mark(st, "k_span_test");
        k_obf_algebra<TIN, D><<<heads, ALG_NT, sm_alg, st>>>(cd);
        mark(st, "k_obf_algebra");
    }
    if (cd.merge) {
        // cache-merging baseline (App. E): route the deleted positions, then add their values into the retained rows
        const size_t sm_mg = merge_smem_bytes<D>();
        if ((s = set_smem(k_merge_assign<TIN, D>, sm_mg)) != OBF_OK) return s;
        dim3 ga((T_max + MG_TILE - 1) / MG_TILE, heads);
        k_merge_assign<TIN, D><<<ga, 256, sm_mg, st>>>(cd);
        mark(st, "k_merge_assign");
        dim3 gm((k_max + 7) / 8, heads);
        k_merge_apply<TIN, D><<<gm, 256, 0, st>>>(cd);
        mark(st, "k_merge_apply");
    }
    bool any_q8 = false;
    for (int i = 0; i < cd.n_caches; ++i) any_q8 = any_q8 || cd.c[i].k_q8 != nullptr;
    if (any_q8) {
        constexpr int QB = qr_block_rows<TIN, D>();
        dim3 gq((k_max + QB - 1) / QB, heads);
        k_quantize_rows<TIN, D><<<gq, 256, 0, st>>>(cd);
        mark(st, "k_quantize_rows");
    }
    OBF_CUDA_TRY(cudaGetLastError());
    return OBF_OK;
}

static obf_status_t run(const obf_params_t *p, const obf_cache_t *caches, int32_t n, int rank,
                        void *workspace, size_t workspace_bytes, void *stream)
{
    g_last_launches = 0;
    obf_status_t s = validate_shapes(p, caches, n, rank);
    if (s != OBF_OK) return s;
    for (int i = 0; i < n; ++i) {
        const obf_cache_t &c = caches[i];
        if (!c.k || !c.v || !c.q_obs || !c.k_out || !c.v_out || !c.idx_out) return OBF_ERR_INVALID_ARG;
        if (misaligned(c.k) || misaligned(c.v) || misaligned(c.q_obs) || misaligned(c.k_out) ||
            misaligned(c.v_out) || (reinterpret_cast<uintptr_t>(c.idx_out) & 3u))
            return OBF_ERR_INVALID_ARG;
        if (c.diag_out && (reinterpret_cast<uintptr_t>(c.diag_out) & 3u)) return OBF_ERR_INVALID_ARG;
        if (c.scores_out && (reinterpret_cast<uintptr_t>(c.scores_out) & 3u)) return OBF_ERR_INVALID_ARG;
        if (c.delta_out && (reinterpret_cast<uintptr_t>(c.delta_out) & 3u)) return OBF_ERR_INVALID_ARG;
        if (c.lse_extra && (reinterpret_cast<uintptr_t>(c.lse_extra) & 3u)) return OBF_ERR_INVALID_ARG;
        // the int8 copy of the relay: all four arrays or none
        const int n_q8 = (c.k_q8_out != nullptr) + (c.v_q8_out != nullptr) + (c.k_scale_out != nullptr) + (c.v_scale_out != nullptr);
        if (n_q8 != 0 && n_q8 != 4) return OBF_ERR_INVALID_ARG;
        if (n_q8 && ((reinterpret_cast<uintptr_t>(c.k_scale_out) & 3u) || (reinterpret_cast<uintptr_t>(c.v_scale_out) & 3u) ||
                     (reinterpret_cast<uintptr_t>(c.k_q8_out) & 7u) || (reinterpret_cast<uintptr_t>(c.v_q8_out) & 7u)))
            return OBF_ERR_INVALID_ARG;
    }
    Layout L;
    make_layout(p, caches, n, rank, L);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < L.total)
        return OBF_ERR_WORKSPACE;
    if (p->flags & OBF_FLAG_TEST_WAIT_EXPIRES) {
        // the test hook is for tiny calls on the tuned score kernel only
        if (!L.sc_on || L.heads_total > 4) return OBF_ERR_INVALID_ARG;
        for (int i = 0; i < n; ++i)
            if (caches[i].T > 2048) return OBF_ERR_INVALID_ARG;
    }

    CallDev cd;
    std::memset(&cd, 0, sizeof(cd));
    const int hpc = p->layers * p->kv_heads;
    int T_max = 1, k_max = 1;
    for (int i = 0; i < n; ++i) {
        CacheDev &c = cd.c[i];
        c.k = caches[i].k; c.v = caches[i].v; c.q = caches[i].q_obs;
        c.k_out = caches[i].k_out; c.v_out = caches[i].v_out; c.idx_out = caches[i].idx_out;
        c.diag = caches[i].diag_out; c.scores_out = caches[i].scores_out; c.delta_out = caches[i].delta_out;
        c.lse_extra = caches[i].lse_extra;
        c.k_q8 = caches[i].k_q8_out; c.v_q8 = caches[i].v_q8_out;
        c.k_scale = caches[i].k_scale_out; c.v_scale = caches[i].v_scale_out;
        c.assign_out = caches[i].assign_out;
        c.T = caches[i].T;
        c.k_eff = k_eff_of(p, caches[i]);
        c.head_base = i * hpc;
        c.tok_off = L.tok_off[i];
        c.nsub_del = L.tc_per ? L.nsub_del[i] : 0;
        c.sub_base = L.tc_per ? L.sub_base[i] : 0;
        c.sc_team = L.sc_on ? L.sc_team[i] : 0;
        c.sc_hpr = L.sc_on ? L.sc_hpr[i] : 0;
        c.sc_round_base = L.sc_on ? L.sc_round_base[i] : 0;
        c.sc_part_off = L.sc_on ? L.sc_part_off[i] : 0;
        if (c.T > T_max) T_max = c.T;
        if (c.k_eff > k_max) k_max = c.k_eff;
    }
    cd.n_caches = n;
    cd.heads_per_cache = hpc;
    cd.heads_total = L.heads_total;
    cd.n_q = (p->q_heads / p->kv_heads) * p->n_obs;
    cd.d = p->head_dim;
    cd.rank = rank;
    cd.splits = L.splits;
    cd.gram_slots = L.gram_slots;
    cd.tc_per = L.tc_per;
    cd.gram_all = L.tc_per ? 1 : 0;
    cd.u_levels = L.tc_per ? U_LEVELS : 1;
    cd.tc_total_sub = L.tc_total_sub;
    cd.sc_nq = L.sc_on ? L.sc_nq : 0;
    cd.sc_qt = L.sc_on ? L.sc_qt : 1;
    cd.sc_subs = L.sc_subs;
    cd.sc_rounds = L.sc_rounds;
    cd.eps = p->eps;
    char *ws = static_cast<char *>(workspace);
    cd.status = reinterpret_cast<uint32_t *>(ws + L.off_status);
    cd.scores = reinterpret_cast<float *>(ws + L.off_scores);
    cd.keep = reinterpret_cast<uint8_t *>(ws + L.off_keep);
    cd.stats = reinterpret_cast<float *>(ws + L.off_stats);
    cd.sums = reinterpret_cast<float *>(ws + L.off_sums);
    cd.lscores = reinterpret_cast<float *>(ws + L.off_lscores);
    cd.scores2 = reinterpret_cast<float *>(ws + L.off_scores2);
    cd.kv_heads = p->kv_heads;
    cd.layerwise = (p->flags & OBF_FLAG_LAYERWISE) ? 1 : 0;
    cd.n_sink = (int32_t)OBF_FLAG_SINK_OF(p->flags);
    cd.fast_iters = (p->flags & OBF_FLAG_FAST_PATH) ? 3 : 0;
    cd.attn_inject = (p->flags & OBF_FLAG_ATTN_INJECT) ? 1 : 0;
    cd.skip_full = (p->flags & OBF_FLAG_EARLY_OUT) && L.tc_per > 0 && rank > 0 ? 1 : 0;
    cd.alg_rows = k_max < p->head_dim ? k_max : p->head_dim;
    cd.wait_limit_ns = tc::WAIT_LIMIT_NS;
    cd.debug_drop_publish = 0;
    if (p->flags & OBF_FLAG_TEST_WAIT_EXPIRES) {
        cd.wait_limit_ns = 20000000ull;
        cd.debug_drop_publish = 1;
    }
    cd.sc_part = reinterpret_cast<float *>(ws + L.off_sc_part);
    cd.sc_head = reinterpret_cast<float *>(ws + L.off_sc_head);
    cd.sc_cnt = reinterpret_cast<uint32_t *>(ws + L.off_sc_sync);
    cd.gram_d = reinterpret_cast<float *>(ws + L.off_gram_d);
    cd.gram_k = reinterpret_cast<float *>(ws + L.off_gram_k);
    cd.uvec = reinterpret_cast<float *>(ws + L.off_uvec);
    cd.delta = reinterpret_cast<float *>(ws + L.off_delta);
    cd.hflag = reinterpret_cast<uint32_t *>(ws + L.off_hflag);
    cd.svec = reinterpret_cast<float *>(ws + L.off_svec);
    cd.assign = reinterpret_cast<int32_t *>(ws + L.off_assign);
    cd.merge = (p->flags & OBF_FLAG_MERGE) ? 1 : 0;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!g_keep_status) OBF_CUDA_TRY(cudaMemsetAsync(cd.status, 0, 256, st));     // a slab of a larger job adds to the job's status
    if (g_prof.active) cudaEventRecord(g_prof.ev[0], st);

    if (p->dtype == OBF_F32) {
        return p->head_dim == 64 ? launch_generic<float, 64>(cd, L, T_max, k_max, st)
                                 : launch_generic<float, 128>(cd, L, T_max, k_max, st);
    }
    return p->head_dim == 64 ? launch_generic<__nv_bfloat16, 64>(cd, L, T_max, k_max, st)
                             : launch_generic<__nv_bfloat16, 128>(cd, L, T_max, k_max, st);
}

}  // namespace obf

using namespace obf;

extern "C" {

// The rank a call runs with: the cache-merging baseline replaces the back-fill.
static inline int effective_rank(const obf_params_t *p) { return (p->flags & OBF_FLAG_MERGE) ? 0 : p->rank; }

obf_status_t obf_workspace_bytes(const obf_params_t *params, const obf_cache_t *caches, int32_t n_caches,
                                 size_t *bytes)
{
    if (!bytes) return OBF_ERR_INVALID_ARG;
    obf_status_t s = validate_shapes(params, caches, n_caches, params ? params->rank : 0);
    if (s != OBF_OK) return s;
    Layout L;
    make_layout(params, caches, n_caches, effective_rank(params), L);
    *bytes = L.total;
    return OBF_OK;
}

obf_status_t obf_compress(const obf_params_t *params, const obf_cache_t *caches, int32_t n_caches,
                          void *workspace, size_t workspace_bytes, void *stream)
{
    if (!params) return OBF_ERR_INVALID_ARG;
    return run(params, caches, n_caches, effective_rank(params), workspace, workspace_bytes, stream);
}

obf_status_t evict_only(const obf_params_t *params, const obf_cache_t *caches, int32_t n_caches,
                        void *workspace, size_t workspace_bytes, void *stream)
{
    if (!params) return OBF_ERR_INVALID_ARG;
    obf_params_t pe = *params;
    pe.flags &= ~(uint32_t)OBF_FLAG_MERGE;                 // eviction only: nothing is merged either
    return run(&pe, caches, n_caches, 0, workspace, workspace_bytes, stream);
}

struct HostArena {
    size_t k[OBF_MAX_CACHES], v[OBF_MAX_CACHES], q[OBF_MAX_CACHES];
    size_t k_out[OBF_MAX_CACHES], v_out[OBF_MAX_CACHES], idx[OBF_MAX_CACHES];
    size_t diag[OBF_MAX_CACHES], scores[OBF_MAX_CACHES], delta[OBF_MAX_CACHES], lse[OBF_MAX_CACHES];
    size_t ws, ws_bytes, total;
};

static void host_arena_layout(const obf_params_t *p, const obf_cache_t *caches, int32_t n, HostArena &H)
{
    const size_t e = p->dtype == OBF_F32 ? 4 : 2;
    const size_t hpc = (size_t)p->layers * p->kv_heads, d = p->head_dim;
    size_t o = 0;
    for (int i = 0; i < n; ++i) {
        const size_t T = caches[i].T, ke = (size_t)k_eff_of(p, caches[i]);
        H.k[i] = o; o = align_up(o + hpc * T * d * e, 256);
        H.v[i] = o; o = align_up(o + hpc * T * d * e, 256);
        H.q[i] = o; o = align_up(o + (size_t)p->layers * p->q_heads * p->n_obs * d * e, 256);
        H.k_out[i] = o; o = align_up(o + hpc * ke * d * e, 256);
        H.v_out[i] = o; o = align_up(o + hpc * ke * d * e, 256);
        H.idx[i] = o; o = align_up(o + hpc * ke * 4, 256);
        H.diag[i] = o; o = align_up(o + hpc * sizeof(obf_diag_t), 256);
        H.scores[i] = o; if (caches[i].scores_out) o = align_up(o + hpc * T * 4, 256);
        H.delta[i] = o; o = align_up(o + hpc * d * 4, 256);
        H.lse[i] = o; if (caches[i].lse_extra) o = align_up(o + (size_t)p->layers * p->q_heads * p->n_obs * 4, 256);
    }
    Layout L;
    make_layout(p, caches, n, effective_rank(p), L);
    H.ws = o; H.ws_bytes = L.total; o += L.total;
    H.total = o;
}

obf_status_t obf_host_arena_bytes(const obf_params_t *params, const obf_cache_t *caches, int32_t n_caches,
                                  size_t *bytes)
{
    if (!bytes) return OBF_ERR_INVALID_ARG;
    obf_status_t s = validate_shapes(params, caches, n_caches, params ? params->rank : 0);
    if (s != OBF_OK) return s;
    HostArena H;
    host_arena_layout(params, caches, n_caches, H);
    *bytes = H.total;
    return OBF_OK;
}

// Streams and events of the host-staged call: copies in, copies out, and per slab of layers the two
// hand-overs (inputs on the device, results ready).  Created on first use per host thread and device.
constexpr int HOST_SLABS_MAX = 8;
struct HostPipe {
    cudaStream_t cin = nullptr, cout = nullptr;
    cudaEvent_t start = nullptr, in_done[HOST_SLABS_MAX], comp_done[HOST_SLABS_MAX], out_done = nullptr;
    int device = -1;
};

static HostPipe *host_pipe()
{
    static thread_local HostPipe hp[16];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 16) return nullptr;
    HostPipe &h = hp[dev];
    if (h.device != dev) {
        bool ok = cudaStreamCreateWithFlags(&h.cin, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&h.cout, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&h.start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&h.out_done, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < HOST_SLABS_MAX; ++i)
            ok = cudaEventCreateWithFlags(&h.in_done[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&h.comp_done[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) { cudaGetLastError(); return nullptr; }
        h.device = dev;
    }
    return &h;
}

// The layers are cut into slabs that go through copy-in, compute and copy-out as a pipeline: the PCIe link
// carries slab s + 1 in and slab s - 1 out while the kernels work on slab s (layers are independent and
// contiguous in every array).  The kernels of all slabs run on the caller's stream, one slab after the other.
obf_status_t obf_compress_host(const obf_params_t *params, const obf_cache_t *caches, int32_t n_caches,
                               void *device_arena, size_t arena_bytes, void *stream)
{
    obf_status_t s = validate_shapes(params, caches, n_caches, params ? params->rank : 0);
    if (s != OBF_OK) return s;
    for (int i = 0; i < n_caches; ++i) {
        const obf_cache_t &c = caches[i];
        if (!c.k || !c.v || !c.q_obs || !c.k_out || !c.v_out || !c.idx_out) return OBF_ERR_INVALID_ARG;
        if (c.k_q8_out || c.v_q8_out || c.k_scale_out || c.v_scale_out || c.assign_out) return OBF_ERR_UNSUPPORTED;   // device entry points only
    }
    HostArena H;
    host_arena_layout(params, caches, n_caches, H);
    if (!device_arena || (reinterpret_cast<uintptr_t>(device_arena) & 255u) || arena_bytes < H.total)
        return OBF_ERR_WORKSPACE;
    char *base = static_cast<char *>(device_arena);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t e = params->dtype == OBF_F32 ? 4 : 2;
    const size_t H_kv = (size_t)params->kv_heads, d = params->head_dim;
    HostPipe *hp = host_pipe();
    if (!hp) return OBF_ERR_CUDA;
    const int n_slabs = params->layers < 4 ? params->layers : 4;
    // nothing of this call may start before what the caller's stream already holds (an earlier call on the arena)
    OBF_CUDA_TRY(cudaEventRecord(hp->start, st));
    OBF_CUDA_TRY(cudaStreamWaitEvent(hp->cin, hp->start, 0));
    OBF_CUDA_TRY(cudaStreamWaitEvent(hp->cout, hp->start, 0));
    for (int sl = 0; sl < n_slabs; ++sl) {
        const size_t l0 = (size_t)params->layers * sl / n_slabs, l1 = (size_t)params->layers * (sl + 1) / n_slabs;
        const size_t nl = l1 - l0;
        obf_params_t ps = *params;
        ps.layers = (int32_t)nl;
        obf_cache_t dev[OBF_MAX_CACHES];
        for (int i = 0; i < n_caches; ++i) {
            const obf_cache_t &c = caches[i];
            const size_t T = c.T, ke = (size_t)k_eff_of(params, c);
            const size_t kv_l = H_kv * T * d * e, q_l = (size_t)params->q_heads * params->n_obs * d * e;
            const size_t o_l = H_kv * ke * d * e;
            dev[i] = c;
            dev[i].k = base + H.k[i] + l0 * kv_l; dev[i].v = base + H.v[i] + l0 * kv_l; dev[i].q_obs = base + H.q[i] + l0 * q_l;
            dev[i].k_out = base + H.k_out[i] + l0 * o_l; dev[i].v_out = base + H.v_out[i] + l0 * o_l;
            dev[i].idx_out = reinterpret_cast<int32_t *>(base + H.idx[i]) + l0 * H_kv * ke;
            dev[i].diag_out = c.diag_out ? reinterpret_cast<obf_diag_t *>(base + H.diag[i]) + l0 * H_kv : nullptr;
            dev[i].scores_out = c.scores_out ? reinterpret_cast<float *>(base + H.scores[i]) + l0 * H_kv * T : nullptr;
            dev[i].delta_out = c.delta_out ? reinterpret_cast<float *>(base + H.delta[i]) + l0 * H_kv * d : nullptr;
            const size_t lse_l = (size_t)params->q_heads * params->n_obs;
            dev[i].lse_extra = c.lse_extra ? reinterpret_cast<const float *>(base + H.lse[i]) + l0 * lse_l : nullptr;
            if (c.lse_extra)
                OBF_CUDA_TRY(cudaMemcpyAsync(const_cast<float *>(dev[i].lse_extra), c.lse_extra + l0 * lse_l,
                                             nl * lse_l * sizeof(float), cudaMemcpyHostToDevice, hp->cin));
            OBF_CUDA_TRY(cudaMemcpyAsync(const_cast<void *>(dev[i].k), static_cast<const char *>(c.k) + l0 * kv_l, nl * kv_l,
                                         cudaMemcpyHostToDevice, hp->cin));
            OBF_CUDA_TRY(cudaMemcpyAsync(const_cast<void *>(dev[i].v), static_cast<const char *>(c.v) + l0 * kv_l, nl * kv_l,
                                         cudaMemcpyHostToDevice, hp->cin));
            OBF_CUDA_TRY(cudaMemcpyAsync(const_cast<void *>(dev[i].q_obs), static_cast<const char *>(c.q_obs) + l0 * q_l,
                                         nl * q_l, cudaMemcpyHostToDevice, hp->cin));
        }
        OBF_CUDA_TRY(cudaEventRecord(hp->in_done[sl], hp->cin));
        OBF_CUDA_TRY(cudaStreamWaitEvent(st, hp->in_done[sl], 0));
        g_keep_status = sl > 0;
        s = run(&ps, dev, n_caches, effective_rank(&ps), base + H.ws, H.ws_bytes, stream);
        g_keep_status = false;
        if (s != OBF_OK) { cudaStreamSynchronize(hp->cin); cudaStreamSynchronize(st); cudaStreamSynchronize(hp->cout); return s; }
        OBF_CUDA_TRY(cudaEventRecord(hp->comp_done[sl], st));
        OBF_CUDA_TRY(cudaStreamWaitEvent(hp->cout, hp->comp_done[sl], 0));
        for (int i = 0; i < n_caches; ++i) {
            const obf_cache_t &c = caches[i];
            const size_t T = c.T, ke = (size_t)k_eff_of(params, c);
            const size_t o_l = H_kv * ke * d * e;
            OBF_CUDA_TRY(cudaMemcpyAsync(static_cast<char *>(c.k_out) + l0 * o_l, dev[i].k_out, nl * o_l, cudaMemcpyDeviceToHost, hp->cout));
            OBF_CUDA_TRY(cudaMemcpyAsync(static_cast<char *>(c.v_out) + l0 * o_l, dev[i].v_out, nl * o_l, cudaMemcpyDeviceToHost, hp->cout));
            OBF_CUDA_TRY(cudaMemcpyAsync(c.idx_out + l0 * H_kv * ke, dev[i].idx_out, nl * H_kv * ke * 4, cudaMemcpyDeviceToHost, hp->cout));
            if (c.diag_out)
                OBF_CUDA_TRY(cudaMemcpyAsync(c.diag_out + l0 * H_kv, dev[i].diag_out, nl * H_kv * sizeof(obf_diag_t),
                                             cudaMemcpyDeviceToHost, hp->cout));
            if (c.scores_out)
                OBF_CUDA_TRY(cudaMemcpyAsync(c.scores_out + l0 * H_kv * T, dev[i].scores_out, nl * H_kv * T * 4,
                                             cudaMemcpyDeviceToHost, hp->cout));
            if (c.delta_out)
                OBF_CUDA_TRY(cudaMemcpyAsync(c.delta_out + l0 * H_kv * d, dev[i].delta_out, nl * H_kv * d * 4,
                                             cudaMemcpyDeviceToHost, hp->cout));
        }
    }
    OBF_CUDA_TRY(cudaEventRecord(hp->out_done, hp->cout));
    OBF_CUDA_TRY(cudaStreamWaitEvent(st, hp->out_done, 0));
    OBF_CUDA_TRY(cudaStreamSynchronize(st));
    return OBF_OK;
}

obf_status_t obf_last_device_status(const void *workspace, void *stream, uint32_t *device_status)
{
    if (!workspace || !device_status) return OBF_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t v = 0;
    OBF_CUDA_TRY(cudaMemcpyAsync(&v, workspace, sizeof(v), cudaMemcpyDeviceToHost, st));
    OBF_CUDA_TRY(cudaStreamSynchronize(st));
    *device_status = v;
    return (v & (OBF_DEV_NONFINITE | OBF_DEV_NO_CONVERGE | OBF_DEV_TIMEOUT | OBF_DEV_INTERNAL)) ? OBF_ERR_DEVICE_STATUS : OBF_OK;
}

obf_status_t obf_compress_profiled(const obf_params_t *params, const obf_cache_t *caches, int32_t n_caches,
                                   void *workspace, size_t workspace_bytes, void *stream,
                                   float *phase_ms, int32_t *n_phases)
{
    if (!params || !phase_ms || !n_phases) return OBF_ERR_INVALID_ARG;
    for (int i = 0; i <= OBF_MAX_PHASES; ++i) OBF_CUDA_TRY(cudaEventCreate(&g_prof.ev[i]));
    // One untimed pass first: while the device works on it the host enqueues the timed pass, so that
    // the events of the timed pass are not separated by host-side launch latency.
    obf_status_t s = run(params, caches, n_caches, effective_rank(params), workspace, workspace_bytes, stream);
    if (s != OBF_OK) {
        for (int i = 0; i <= OBF_MAX_PHASES; ++i) cudaEventDestroy(g_prof.ev[i]);
        return s;
    }
    g_prof.n = 0;
    g_prof.active = true;
    s = run(params, caches, n_caches, effective_rank(params), workspace, workspace_bytes, stream);
    g_prof.active = false;
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    *n_phases = 0;
    if (s == OBF_OK && e == cudaSuccess) {
        for (int i = 0; i < g_prof.n; ++i) {
            cudaEventElapsedTime(&phase_ms[i], g_prof.ev[i], g_prof.ev[i + 1]);
            g_phase_names[i] = g_prof.names[i];
        }
        g_phase_count = g_prof.n;
        *n_phases = g_prof.n;
    }
    for (int i = 0; i <= OBF_MAX_PHASES; ++i) cudaEventDestroy(g_prof.ev[i]);
    if (e != cudaSuccess) return OBF_ERR_CUDA;
    return s;
}

const char *obf_phase_name(int32_t phase)
{
    return (phase >= 0 && phase < g_phase_count) ? g_phase_names[phase] : "";
}

const char *obf_status_string(obf_status_t status)
{
    switch (status) {
    case OBF_OK: return "ok";
    case OBF_ERR_INVALID_ARG: return "invalid argument";
    case OBF_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case OBF_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case OBF_ERR_CUDA: return "CUDA runtime error";
    case OBF_ERR_DEVICE_STATUS: return "device reported a numerical or timeout condition";
    }
    return "unknown status";
}

int32_t obf_last_launch_count(void) { return g_last_launches; }

}  // extern "C"

// ---------------------------------------------------------------------------
// evict_only with library-owned scratch, for callers that cannot allocate.
// ---------------------------------------------------------------------------
namespace {

// The scratch itself.  In host code this name is only a handle for the runtime,
// not an address a kernel could use; the device address is looked up per device.
static __device__ __align__(256) unsigned char g_static_scratch[OBF_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
// Device address of the array, per device ordinal; null until resolved.  Host threads that make their first call
// on a device at the same time may each resolve it: they store the same value, and the atomic makes that well defined.
std::atomic<void *> g_static_scratch_addr[kMaxDevices];

// Device address of the scratch array on the current device; resolved on the first call per device.
obf_status_t static_scratch_ptr(void **out)
{
    int dev = -1;
    OBF_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return OBF_ERR_UNSUPPORTED;
    void *ptr = g_static_scratch_addr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        OBF_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        if (!ptr) return OBF_ERR_CUDA;
        g_static_scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return OBF_OK;
}

}  // namespace

extern "C" obf_status_t evict_only_static(const obf_params_t *params, const obf_cache_t *caches,
                                          int32_t n_caches, void *stream)
{
    obf_status_t s = validate_shapes(params, caches, n_caches, 0);
    if (s != OBF_OK) return s;
    obf_params_t pe = *params;
    pe.flags &= ~(uint32_t)OBF_FLAG_MERGE;                 // eviction only: nothing is merged either
    params = &pe;
    Layout L;
    make_layout(params, caches, n_caches, 0, L);
    if (L.total > (size_t)OBF_STATIC_SCRATCH_BYTES) {
        std::fprintf(stderr,
                     "obf: evict_only_static: this call needs %zu bytes of scratch but the built-in array holds "
                     "%zu; use evict_only with a caller-provided workspace\n",
                     L.total, (size_t)OBF_STATIC_SCRATCH_BYTES);
        return OBF_ERR_WORKSPACE;
    }
    void *scratch = nullptr;
    if ((s = static_scratch_ptr(&scratch)) != OBF_OK) return s;
    // run() clears the status word at the head of the scratch; every other region is
    // written by an earlier kernel of the same call before a later one reads it.
    return run(params, caches, n_caches, 0, scratch, (size_t)OBF_STATIC_SCRATCH_BYTES, stream);
}

extern "C" obf_status_t obf_static_scratch_status(void *stream, uint32_t *device_status)
{
    void *scratch = nullptr;
    obf_status_t s = static_scratch_ptr(&scratch);
    if (s != OBF_OK) return s;
    return obf_last_device_status(scratch, stream, device_status);
}
