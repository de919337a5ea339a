/*
 * obf.h - C ABI of the relay-boundary prompt-KV compressor for NVIDIA B200 (sm_100a).
 *
 * One call compresses the prompt KV cache of one or more agents at the relay
 * boundary.  For every (cache, layer, KV head), independently (Section 4.4):
 *
 *   a1  score    A_j = sum over the observation queries t mapped to this KV head of
 *                softmax_j(q_t . K_j / sqrt(head_dim))            (Eq. 1; softmax form of App. L.1)
 *   a2  select   the k_eff = min(budget, T) positions of largest A_j, equal masses
 *                resolved towards the lower position, emitted in ascending
 *                position order                                   (Section 4.3.2; Section 3.1)
 *   a3  gather   K_keep = K[idx,:], V_keep = V[idx,:]             (Algorithm 2, last step)
 *   a4  OBF      orthonormal basis of span(V_keep) (Eq. 2); residual of the deleted
 *                values against that span (Eq. 3); its top-`rank` right singular
 *                subspace C; attention-weighted residual mean r_bar (Eq. 4);
 *                Delta = (r_bar C^T) C (Eq. 5); delta = A_del/(A_keep+eps) * Delta
 *                (Eq. 6); V_out = V_keep + delta on every retained row, keys
 *                untouched (Eq. 7; Algorithm 3)
 *
 * All pointers in obf_cache_t are DEVICE pointers unless a function says
 * otherwise.  The caller owns every buffer, including the workspace; the
 * library allocates no device memory, enqueues all work on `stream`, never
 * synchronises (except obf_last_device_status and the *_host entry point's
 * final wait, as documented) and does not touch the inputs after the enqueued
 * work has completed.  Inputs are read-only and must not alias outputs.
 *
 * Layout (row-major, contiguous, 16-byte aligned base pointers):
 *   k, v      [layers, kv_heads, T, head_dim]
 *   q_obs     [layers, q_heads, n_obs, head_dim]   q head = kv_head * G + g, G = q_heads / kv_heads
 *   k_out,
 *   v_out     [layers, kv_heads, k_eff, head_dim]  same dtype as the inputs
 *   idx_out   [layers, kv_heads, k_eff] int32      ascending positions in [0, T)
 *
 * Numerics: bf16 products accumulated in fp32; softmax, pooling, selection
 * keys and all OBF algebra in fp32; V_out is the fp32 sum rounded once to the
 * output dtype (bit-exact copy of V_keep wherever delta == 0).  K_out is always
 * a bit-exact copy.
 *
 * Errors: anything detectable on the host (null or misaligned pointer, bad
 * shape, budget < 1, rank outside [0, head_dim], unsupported head_dim or dtype,
 * workspace too small) returns a code before anything is enqueued.  Conditions
 * only the device can see are ORed into a status word in the workspace (and
 * into obf_diag_t.status of the head concerned); obf_last_device_status reads
 * it.  A head that hits one keeps its eviction-only result (the skip rule in
 * the footnote to Eq. 7).
 */
#ifndef OBF_H_
#define OBF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    OBF_OK = 0,
    OBF_ERR_INVALID_ARG = 1,    /* null/misaligned pointer, bad shape, budget, rank, n_caches    */
    OBF_ERR_UNSUPPORTED = 2,    /* head_dim not in {64,128}, unknown dtype, too many caches       */
    OBF_ERR_WORKSPACE = 3,      /* workspace null, misaligned or smaller than obf_workspace_bytes */
    OBF_ERR_CUDA = 4,           /* a CUDA runtime call failed (launch, attribute, copy)           */
    OBF_ERR_DEVICE_STATUS = 5   /* the device status word is non-zero (obf_last_device_status)    */
} obf_status_t;

typedef enum { OBF_F32 = 0, OBF_BF16 = 1 } obf_dtype_t;

/* Bits of the device status word / obf_diag_t.status. */
#define OBF_DEV_NONFINITE   0x1u   /* a score or softmax normaliser was not finite                 */
#define OBF_DEV_NO_CONVERGE 0x2u   /* the eigen-iteration hit its sweep limit                      */
#define OBF_DEV_TIMEOUT     0x4u   /* a bounded on-device wait expired                             */
#define OBF_DEV_INTERNAL    0x8u   /* an internal consistency check failed (position out of range) */
#define OBF_DEV_SKIPPED     0x100u /* informational (diag only): OBF skipped, delta = 0            */
#define OBF_DEV_SPAN_FULL   0x200u /* informational (diag only): span(V_keep) is all of R^d        */

/* obf_params_t.flags */
#define OBF_FLAG_GENERIC_PATH 0x1u /* run the shape-generic kernels even where the tuned bf16 path applies */
#define OBF_FLAG_LAYERWISE    0x2u /* layerwise selector (Section 3.2 retention rule, second form; Algorithm 2,
                                      granularity L): the retained positions of a layer are TopK_B of the masses
                                      summed over its KV heads and are shared by those heads (idx_out repeats them
                                      per head); gather and OBF then run per head with the head's own masses.
                                      Needs every T <= 16384, else OBF_ERR_UNSUPPORTED                          */

#define OBF_FLAG_FAST_PATH    0x4u /* the principal subspace of the residual comes from three steps of the Gram
                                      subspace iteration of App. H, C <- orth(C R^T R), started at the first rows of
                                      the identity (the paper leaves the start open), instead of the exact
                                      eigenvectors: an approximation whose error depends on the residual's spectrum.
                                      diag: lam_1 / lam_rho are Rayleigh quotients, lam_next is 0                  */
#define OBF_FLAG_ATTN_INJECT  0x8u /* Attn-inject (App. D.2, alternative designs): the vector delta of Eq. 6 is added in
                                      proportion to each retained position's attention mass instead of uniformly,
                                      V*_t = V_t + k_eff * A_t / (A_keep + eps) * delta (the shares average one).
                                      delta_out and the diagnostics are those of the uniform injection             */
#define OBF_FLAG_MERGE        0x10u /* cache-merging baseline instead of Orthogonal BackFill (App. E, the comparison
                                      method): after selection and gather every deleted position is routed to the
                                      retained position with the most similar key (cosine; ties: lowest position) and
                                      V*_t = V_t + sum over the j routed to t of A_j / (A_t + eps) V_j.  params->rank is
                                      ignored; delta_out stays zero                                                */
#define OBF_FLAG_EARLY_OUT    0x20u /* the span test before the pass over V (tuned bf16 path, rank > 0): a head whose
                                      retained values span R^d has delta = 0 whatever its deleted values are (Eq. 3),
                                      so that pass skips it.  Same outputs bit for bit; the call's kernels then run
                                      one after the other on `stream` instead of beside one another.  Pays when most
                                      heads have budgets of head_dim or more; without the flag every head's values
                                      are streamed                                                                 */
#define OBF_FLAG_SINK(n) (((uint32_t)(n) & 0xFFu) << 8)
                                   /* protected sink prefix (App. F of the paper: the compressors protect the first s
                                      indices of the cache; the eligible set of Section 3.2 leaves the sink out): the
                                      first n <= 255 positions of every cache are retained besides the budget and are no
                                      candidates of the selection, so k_eff = min(n, T) + min(budget, T - min(n, T));
                                      size the outputs with that k_eff                                            */
#define OBF_FLAG_SINK_OF(flags) (((flags) >> 8) & 0xFFu)
#define OBF_FLAG_TEST_WAIT_EXPIRES 0x10000u
                                   /* test hook for the bounded device-side waits of the tuned score kernel: no block
                                      publishes a head's softmax normalisers and the wait limit drops from one second to
                                      20 ms, so every wait for them runs out, the kernels return by themselves, the
                                      status word carries OBF_DEV_TIMEOUT and the outputs hold valid positions but no
                                      meaningful selection.  Accepted only for at most 4 (layer, KV head) pairs in all,
                                      every T <= 2048, on the tuned bf16 / head_dim 128 path; else
                                      OBF_ERR_INVALID_ARG                                                         */

#define OBF_MAX_CACHES 32          /* caches per call                                              */
#define OBF_MAX_T (1 << 20)        /* prompt positions per cache                                   */

typedef struct {              /* shared by all caches of one call                                   */
    int32_t layers, kv_heads, q_heads;  /* q_heads % kv_heads == 0                                  */
    int32_t head_dim;                   /* 64 or 128                                                */
    int32_t n_obs;                      /* observation queries per query head (>= 1)                */
    int32_t rank;                       /* pca_rank of Section 4.4; 0 = eviction only               */
    int32_t dtype;                      /* obf_dtype_t of k, v, q_obs, k_out, v_out                 */
    float   eps;                        /* the epsilon of Eq. 4 and Eq. 6 (the paper uses 1e-12)    */
    uint32_t flags;                     /* OBF_FLAG_*                                               */
} obf_params_t;

typedef struct {              /* per (layer, KV head) diagnostics (App. K.2 names in brackets)      */
    float a_keep, a_del;      /* attention mass on retained / deleted positions (Eq. 6)             */
    float alpha;              /* a_del / (a_keep + eps)                              [DR]           */
    float rcr;                /* ||R||_F^2 / (||V_del||_F^2 + eps)                   [RCR]          */
    float delta_norm;         /* ||delta||_2                                         [IVN]          */
    float kth_score;          /* smallest retained mass among the candidates of the selection       */
    float next_score;         /* largest deleted mass, -1 if nothing is deleted                     */
    float lam_1, lam_rho, lam_next; /* eigenvalues of R^T R: largest, last kept, first dropped      */
    int32_t span_rank;        /* numerical dimension m of span(V_keep) (-1: not evaluated)          */
    int32_t rho_eff;          /* number of principal directions actually used                       */
    uint32_t status;          /* OBF_DEV_* bits                                                     */
    float revr;               /* sum of the rho_eff kept eigenvalues of R^T R over their total  [REVR]; PCR is 1 - rcr */
    float pc;                 /* cosine between the sum of the deleted values and the sum of their projections onto
                                 span(V_keep)  [PC]; 0 when OBF does not run for the head; costs one more pass over V,
                                 made only when diag_out is given                                        */
} obf_diag_t;

typedef struct {              /* one agent's prompt cache; T and budget may differ between caches   */
    const void *k, *v;        /* [layers, kv_heads, T, head_dim]                                    */
    const void *q_obs;        /* [layers, q_heads, n_obs, head_dim]                                 */
    int32_t T;                /* prompt positions, 1 <= T <= OBF_MAX_T                              */
    int32_t budget;           /* >= 1; k_eff = min(budget, T) (more with OBF_FLAG_SINK, see there)  */
    void *k_out, *v_out;      /* [layers, kv_heads, k_eff, head_dim]                                */
    int32_t *idx_out;         /* [layers, kv_heads, k_eff]                                          */
    obf_diag_t *diag_out;     /* optional [layers, kv_heads], or NULL                               */
    float *scores_out;        /* optional [layers, kv_heads, T] attention mass A (Eq. 1), or NULL   */
    float *delta_out;         /* optional [layers, kv_heads, head_dim] injected vector (Eq. 6), or NULL */
    const float *lse_extra;   /* optional device [layers, q_heads, n_obs] fp32, or NULL: per observation query the
                                 natural log of the sum of exp(q.k / sqrt(d)) over the keys OUTSIDE the prompt that the
                                 model's softmax also ran over (earlier agents' relay, the latent positions before it:
                                 Section 3.1 defines the weights of Eq. 1 as a softmax over the whole cache, App. L.1
                                 restates it over the prompt).  Those keys take their share of every row's
                                 normaliser, so a row's weights over the prompt add up to less than one.  NULL or
                                 minus infinity: softmax over the prompt keys alone                          */
    /* Optional int8 copy of the compacted relay (post-hoc quantisation stacked on the compression, App. E, Table 7;
       the paper fixes no quantiser: symmetric, one fp32 scale per retained row, scale = max|x| / 127, code =
       round-half-even(x / scale), a row of zeros has scale 0).  All four NULL, or all four device pointers:
       k_q8_out, v_q8_out int8 [layers, kv_heads, k_eff, head_dim]; k_scale_out, v_scale_out fp32
       [layers, kv_heads, k_eff]; the int8 arrays 8-byte aligned, the scales 4-byte aligned.  The codes are taken
       from k_out / v_out as the call leaves them (v_out after the injection of Eq. 7), which are still written. */
    int8_t *k_q8_out, *v_q8_out;
    float *k_scale_out, *v_scale_out;
    int32_t *assign_out;      /* optional device [layers, kv_heads, T], or NULL; with OBF_FLAG_MERGE: the slot
                                 (0 .. k_eff-1) every deleted position was routed to, -1 for retained positions   */
} obf_cache_t;

/*
 * Size in bytes of the scratch workspace obf_compress / evict_only need for
 * this call shape (Eq. 1's masses, selection flags, the d x d Gram matrices of
 * Eq. 3 and App. H).  Host-only; enqueues nothing.  Pointers inside `caches`
 * are not inspected, only T and budget.
 */
obf_status_t obf_workspace_bytes(const obf_params_t *params, const obf_cache_t *caches,
                                 int32_t n_caches, size_t *bytes);

/*
 * Phi_OBF (Algorithm 3) on every (cache, layer, KV head).  `params`/`caches`
 * are host structs (copied before return); `workspace` is device memory of at
 * least obf_workspace_bytes(), 256-byte aligned, private to this call until
 * the enqueued work completes; `stream` is a cudaStream_t passed as void*.
 * With rank > 0 on the tuned path the selection, the gather of the values and
 * the span test run on a stream of the library (created on first use per host
 * thread and device) that forks from and joins `stream` inside the call,
 * beside the pass over V: everything the call does is ordered on `stream`.
 *
 * Calls that overlap on one device (different streams or host threads, each
 * with its own workspace) are legal but do not speed each other up: the tuned
 * score kernel's blocks wait for one another, so it is launched cooperatively
 * and starts only when the whole grid (one block per multiprocessor) can be
 * resident; until then it waits for whatever else holds the multiprocessors.
 * Every device-side wait is bounded (one second): if one ever runs out the
 * kernels return by themselves, the status word carries OBF_DEV_TIMEOUT (see
 * obf_last_device_status) and the outputs hold valid positions but no
 * meaningful selection.
 */
obf_status_t obf_compress(const obf_params_t *params, const obf_cache_t *caches, int32_t n_caches,
                          void *workspace, size_t workspace_bytes, void *stream);

/*
 * Phi_Attn with headwise granularity (Algorithm 2): steps a1-a3 only.
 * Identical to obf_compress with rank = 0 (params->rank is ignored).
 */
obf_status_t evict_only(const obf_params_t *params, const obf_cache_t *caches, int32_t n_caches,
                        void *workspace, size_t workspace_bytes, void *stream);

/*
 * Size of the device arena obf_compress_host needs (device copies of every
 * input and output of the call plus the workspace).
 */
obf_status_t obf_host_arena_bytes(const obf_params_t *params, const obf_cache_t *caches,
                                  int32_t n_caches, size_t *bytes);

/*
 * Same operation for callers whose caches live in HOST memory (Algorithm 1's
 * relay hand-off when the cache is staged on the host).  Every pointer inside
 * `caches` is a host pointer (pinned memory makes the copies asynchronous);
 * `device_arena` is device memory of at least obf_host_arena_bytes(),
 * 256-byte aligned.  Copies k, v, q_obs to the device, compresses, and copies
 * k_out, v_out, idx_out (and the optional outputs that are not NULL) back,
 * as a pipeline over slabs of layers: the copies run on two streams that
 * the library creates on first use (per host thread and device), the
 * kernels on `stream`; work already enqueued on `stream` is waited for
 * first.  Returns after everything has finished.  The injected vectors can
 * differ from obf_compress on the same data in the last fp32 digits (a slab
 * adds its partial sums up in another order than the whole call).
 */
obf_status_t obf_compress_host(const obf_params_t *params, const obf_cache_t *caches, int32_t n_caches,
                               void *device_arena, size_t arena_bytes, void *stream);

/*
 * Waits for `stream`, reads the status word the last call left in `workspace`
 * and stores it in *device_status.  Returns OBF_ERR_DEVICE_STATUS if any of
 * the error bits (OBF_DEV_NONFINITE, OBF_DEV_NO_CONVERGE, OBF_DEV_TIMEOUT,
 * OBF_DEV_INTERNAL) is set.
 */
obf_status_t obf_last_device_status(const void *workspace, void *stream, uint32_t *device_status);

/*
 * obf_compress with per-kernel device timing, for profiling only.  Enqueues the
 * same kernels as obf_compress (params->rank == 0 gives evict_only's), with a
 * CUDA event recorded between consecutive launches, waits for the stream and
 * writes the elapsed milliseconds of each launch to phase_ms[0 .. *n_phases-1]
 * (host array with room for OBF_MAX_PHASES floats).  obf_phase_name(i) names
 * launch i of the last profiled call of this thread.
 */
#define OBF_MAX_PHASES 16
obf_status_t obf_compress_profiled(const obf_params_t *params, const obf_cache_t *caches, int32_t n_caches,
                                   void *workspace, size_t workspace_bytes, void *stream,
                                   float *phase_ms, int32_t *n_phases);
const char *obf_phase_name(int32_t phase);

/*
 * evict_only for callers that cannot obtain a workspace.  (The paper has no
 * counterpart: this entry point exists for deployment reasons only.)
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they
 * need a compression: a serving process whose start-up code handed every byte
 * of device memory to its own pool, a plug-in that runs under another
 * framework's allocator and must not allocate behind its back, or a latency
 * critical loop that cannot take the device-wide synchronisation an allocation
 * implies.  For them the scratch memory lives inside the library: a fixed
 * array of OBF_STATIC_SCRATCH_BYTES bytes in the library's device image, which
 * every GPU that loads the library holds until the process exits.  The caller
 * passes only inputs and outputs (all device pointers, as for evict_only).
 *
 * - Computes exactly what evict_only computes (steps a1-a3; params->rank is
 *   ignored) and returns the same codes, plus OBF_ERR_WORKSPACE - with a
 *   message on stderr naming both sizes - when the call shape needs more
 *   scratch than OBF_STATIC_SCRATCH_BYTES (obf_workspace_bytes with rank 0
 *   tells how much a shape needs).
 * - Calls no cudaMalloc, cudaFree or any other allocating routine.
 * - The first call on each device resolves the array's device address
 *   (cudaGetSymbolAddress, with that device current); make that first call
 *   before starting any stream capture on the device.  Host threads may make
 *   their first calls at the same time (the address is kept in an atomic).
 * - All calls on one device share the one array and it keeps whatever the
 *   previous call left; the call clears the part that has to start at zero
 *   (the status word) and overwrites the rest before reading it.  Two calls
 *   whose work overlaps on the GPU (different streams, or different host
 *   threads) race on the array: serialise them.
 * - obf_static_scratch_status reads the status word of the last such call.
 */
#define OBF_STATIC_SCRATCH_BYTES (8u << 20)
obf_status_t evict_only_static(const obf_params_t *params, const obf_cache_t *caches, int32_t n_caches,
                               void *stream);
obf_status_t obf_static_scratch_status(void *stream, uint32_t *device_status);

/* Static, never NULL. */
const char *obf_status_string(obf_status_t status);

/* Number of kernels the last obf_compress / evict_only call of this thread enqueued. */
int32_t obf_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* OBF_H_ */
