/*
 * CPU oracle for relay-boundary prompt-KV compression: headwise (or layerwise)
 * attention-mass eviction followed by Orthogonal BackFill (OBF).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, fp64,
 * step-by-step statement of the paper's definitions (Eq. 1-7, Algorithms 2-3),
 * used by the tests, by the smoke check and by the benchmark's CPU-baseline
 * leg.  It shares no code with the CUDA path and the CUDA path never calls it.
 *
 * Inputs are float32 (bf16 inputs are up-cast exactly by the caller); every
 * arithmetic step is carried out in double.  One (layer, KV head) is one
 * independent problem (Section 4.4 applies every step per layer and KV head).
 *
 * Pin status (see tests, all CPU-only):
 *   scores      pinned: row-sum invariant, equal-key closed form, T=2 sigmoid
 *               closed form, library softmax, permutation equivariance;
 *               with out-of-prompt mass: minus infinity gives the plain masses,
 *               an appended key whose mass is dropped gives the same masses,
 *               library log-sum-exp
 *   top-k       pinned: brute-force full sort on tiny inputs, library stable
 *               argsort, planted exact ties
 *   sink prefix pinned: protected positions always retained, the rest equals
 *               the plain top-k of the remaining positions (library argsort)
 *   layerwise   pinned: one KV head reduces to the headwise result, identical
 *               heads reduce to the headwise result, library argsort of the
 *               summed masses, retained set shared by the heads of a layer
 *   gather      pinned: bitwise copies
 *   span basis  pinned: orthonormality, annihilation of V_keep, library
 *               pseudo-inverse projector, library matrix rank
 *   eigen/C     pinned: library SVD of the explicit residual, Max-P closed
 *               form, codimension-1 closed form, hand-worked planted example
 *   scaling     pinned: single-query identity from the error-bound appendix,
 *               hand-worked planted example
 *   merging     pinned: library cosine / argmax statement (numpy), every deleted
 *               position routed exactly once, mass-weighted value sums conserved,
 *               a duplicate of a retained key is routed to it
 *   attn-inject pinned: equal masses give the uniform injection, the shares add up
 *               to the number of retained positions, library statement
 *   int8 relay  pinned: round-trip error at most half a step per element, the
 *               largest element of a row maps to +-127, library rounding
 *               (numpy rint in float32), zero rows
 * No function here is "parity unpinned".
 */
#include <math.h>
#include <float.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    double a_keep;       /* sum of attention mass over retained positions (Eq. 6)          */
    double a_del;        /* sum of attention mass over deleted positions (Eq. 6)           */
    double alpha;        /* a_del / (a_keep + eps)                                          */
    double vdel_fro2;    /* ||V_del||_F^2                                                   */
    double r_fro2;       /* ||R||_F^2                                                       */
    double rcr;          /* r_fro2 / (vdel_fro2 + eps)   (App. K.2)                         */
    double rbar_norm;    /* ||r_bar||_2                                                     */
    double delta_norm;   /* ||delta||_2  (IVN, App. K.2)                                    */
    double kth_score;    /* k_eff-th largest attention mass                                 */
    double next_score;   /* (k_eff+1)-th largest attention mass, or -1 if none              */
    double lam_rho;      /* eigenvalue rho_eff of R^T R (smallest one kept), 0 if none      */
    double lam_next;     /* eigenvalue rho_eff+1 of R^T R (largest one dropped), 0 if none  */
    double lam_1;        /* largest eigenvalue of R^T R                                     */
    int32_t span_rank;   /* numerical rank m of span(V_keep)                                */
    int32_t rho_eff;     /* min(pca_rank, numerical rank of R)                              */
    int32_t n_del;       /* number of deleted positions                                     */
    int32_t skipped;     /* 1 if OBF was skipped for this head (footnote to Eq. 7)          */
    double revr;         /* kept share of the residual's squared singular values (REVR, App. K.2) */
    double pc;           /* cosine between the sum of the deleted values and the sum of their projections
                            onto span(V_keep) (PC, App. K.2); 0 when OBF does not run          */
} obf_oracle_diag_t;

/* ------------------------------------------------------------------ */
/* Step O1 - attention mass, Eq. 1 with the softmax of App. L.1        */
/* ------------------------------------------------------------------ */
/*
 * A_j = sum over the n_q query rows t of softmax_j(q_t . K_j / sqrt(d)).
 * The n_q rows are all observation queries of all query heads that share this
 * KV head (Eq. 1's sum extended over the GQA group).  Softmax runs over the T
 * prompt keys only, natural exponential, maximum subtracted first.
 */
/*
 * lse_extra (may be NULL): per query row t the natural logarithm of the sum of exp(logit) over the keys
 * OUTSIDE the prompt that the model's softmax also ran over (Section 3.1: the attention weights are a softmax
 * over the whole cache; the prompt is one part of it).  The normaliser then is the prompt's sum plus
 * exp(lse_extra[t]), so a row's weights over the prompt add up to less than one.  NULL or minus infinity:
 * the softmax over the prompt keys alone (App. L.1).
 */
void obf_oracle_scores_ext(const float *K, const float *Q, const float *lse_extra, int T, int d, int n_q, double *A)
{
    double *s = (double *)malloc((size_t)T * sizeof(double));
    const double scale = 1.0 / sqrt((double)d);
    for (int j = 0; j < T; ++j) A[j] = 0.0;
    for (int t = 0; t < n_q; ++t) {
        const float *q = Q + (size_t)t * d;
        const double extra = lse_extra ? (double)lse_extra[t] : -INFINITY;
        double mx = extra;
        for (int j = 0; j < T; ++j) {
            const float *k = K + (size_t)j * d;
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += (double)q[c] * (double)k[c];
            s[j] = acc * scale;
            if (s[j] > mx) mx = s[j];
        }
        double Z = extra > -INFINITY ? exp(extra - mx) : 0.0;
        for (int j = 0; j < T; ++j) { s[j] = exp(s[j] - mx); Z += s[j]; }
        for (int j = 0; j < T; ++j) A[j] += s[j] / Z;
    }
    free(s);
}

void obf_oracle_scores(const float *K, const float *Q, int T, int d, int n_q, double *A)
{
    obf_oracle_scores_ext(K, Q, NULL, T, d, n_q, A);
}

/* ------------------------------------------------------------------ */
/* Step O2 - TopK_B with deterministic ties                            */
/* ------------------------------------------------------------------ */
typedef struct { double a; int32_t j; } score_pos_t;

static int cmp_score_desc_index_asc(const void *x, const void *y)
{
    const score_pos_t *p = (const score_pos_t *)x, *q = (const score_pos_t *)y;
    if (p->a > q->a) return -1;
    if (p->a < q->a) return 1;
    return (p->j > q->j) - (p->j < q->j);      /* equal mass: lower position first */
}

static int cmp_int_asc(const void *x, const void *y)
{
    int32_t a = *(const int32_t *)x, b = *(const int32_t *)y;
    return (a > b) - (a < b);
}

/*
 * The first n_sink positions are protected (the sink prefix of App. F, "Right
 * padding": the compressors protect the first s indices of the cache); they are
 * no candidates of the selection (the eligible set of Section 3.2 leaves them
 * out) and are retained besides the budget.  The other positions are ordered by
 * (mass descending, position ascending) and the first min(budget, T - n_sink)
 * of them are kept.  Returns k_eff = min(n_sink, T) + that many, the retained
 * positions as an ascending index list (Section 3.1: a retained cache is a
 * subsequence i_1 < ... < i_m).  kth/next receive the smallest retained and the
 * largest deleted mass among the candidates (-1 when there is none).
 */
int obf_oracle_topk_sink(const double *A, int T, int budget, int n_sink, int32_t *idx, double *kth, double *next)
{
    int s = n_sink < T ? n_sink : T;
    if (s < 0) s = 0;
    const int nc = T - s;                                  /* candidates */
    int kc = budget < nc ? budget : nc;
    if (kc < 0) kc = 0;
    score_pos_t *sp = (score_pos_t *)malloc((size_t)(nc > 0 ? nc : 1) * sizeof(score_pos_t));
    for (int j = s; j < T; ++j) { sp[j - s].a = A[j]; sp[j - s].j = j; }
    qsort(sp, (size_t)nc, sizeof(score_pos_t), cmp_score_desc_index_asc);
    for (int r = 0; r < s; ++r) idx[r] = r;
    for (int r = 0; r < kc; ++r) idx[s + r] = sp[r].j;
    if (kth)  *kth  = kc > 0 ? sp[kc - 1].a : -1.0;
    if (next) *next = kc < nc ? sp[kc].a : -1.0;
    qsort(idx, (size_t)(s + kc), sizeof(int32_t), cmp_int_asc);
    free(sp);
    return s + kc;
}

/* TopK_B with every position eligible. */
int obf_oracle_topk(const double *A, int T, int budget, int32_t *idx, double *kth, double *next)
{
    return obf_oracle_topk_sink(A, T, budget, 0, idx, kth, next);
}

/* ------------------------------------------------------------------ */
/* Step O6 - orthonormal basis of span(V_keep), Eq. 2                  */
/* ------------------------------------------------------------------ */
/*
 * X is k x d (rows are retained value states).  Writes an orthonormal basis of
 * the row space as the rows of Qb (at most min(k,d) rows of length d) and
 * returns its dimension m.  Gram-Schmidt with largest-remaining-row pivoting
 * and a second orthogonalisation pass; a direction is accepted while the
 * largest remaining row norm exceeds max(k,d) * DBL_EPSILON times the largest
 * original row norm.  Eq. 2 needs any orthonormal basis of that span: only the
 * span enters the method (through Q Q^T), so the pivot order is free.
 */
int obf_oracle_span_basis(const double *X, int k, int d, double *Qb)
{
    if (k <= 0) return 0;
    double *W = (double *)malloc((size_t)k * d * sizeof(double));
    memcpy(W, X, (size_t)k * d * sizeof(double));
    int mmax = k < d ? k : d;
    int m = 0;
    double ref = 0.0;
    const double tol = (double)(k > d ? k : d) * DBL_EPSILON;
    while (m < mmax) {
        int p = -1; double best = 0.0;
        for (int i = 0; i < k; ++i) {
            double n2 = 0.0;
            for (int c = 0; c < d; ++c) n2 += W[(size_t)i * d + c] * W[(size_t)i * d + c];
            if (n2 > best) { best = n2; p = i; }
        }
        if (p < 0) break;
        double nrm = sqrt(best);
        if (m == 0) ref = nrm;
        if (nrm <= tol * ref) break;
        double *q = Qb + (size_t)m * d;
        for (int c = 0; c < d; ++c) q[c] = W[(size_t)p * d + c] / nrm;
        for (int pass = 0; pass < 2; ++pass) {            /* re-orthogonalise against earlier rows */
            for (int r = 0; r < m; ++r) {
                const double *qr = Qb + (size_t)r * d;
                double dot = 0.0;
                for (int c = 0; c < d; ++c) dot += q[c] * qr[c];
                for (int c = 0; c < d; ++c) q[c] -= dot * qr[c];
            }
            double n2 = 0.0;
            for (int c = 0; c < d; ++c) n2 += q[c] * q[c];
            double inv = 1.0 / sqrt(n2);
            for (int c = 0; c < d; ++c) q[c] *= inv;
        }
        for (int i = 0; i < k; ++i) {                     /* deflate every remaining row */
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += W[(size_t)i * d + c] * q[c];
            for (int c = 0; c < d; ++c) W[(size_t)i * d + c] -= dot * q[c];
        }
        ++m;
    }
    free(W);
    return m;
}

/* ------------------------------------------------------------------ */
/* Step O9 - symmetric eigen-decomposition (cyclic Jacobi)             */
/* ------------------------------------------------------------------ */
/*
 * S is n x n symmetric (destroyed).  On return lam[0] >= lam[1] >= ... and row
 * i of E is the unit eigenvector of lam[i].  Classical cyclic Jacobi rotations
 * until every off-diagonal entry is negligible against its diagonal pair.
 */
void obf_oracle_sym_eig(double *S, int n, double *lam, double *E)
{
    double *U = (double *)calloc((size_t)n * n, sizeof(double));   /* columns = eigenvectors */
    for (int i = 0; i < n; ++i) U[(size_t)i * n + i] = 1.0;
    double fro = 0.0;
    for (int i = 0; i < n * n; ++i) fro += S[i] * S[i];
    const double floor_abs = DBL_EPSILON * DBL_EPSILON * sqrt(fro);   /* noise floor in null directions */
    for (int sweep = 0; sweep < 100; ++sweep) {
        int rotated = 0;
        for (int p = 0; p < n - 1; ++p) {
            for (int q = p + 1; q < n; ++q) {
                double apq = S[(size_t)p * n + q];
                double app = S[(size_t)p * n + p], aqq = S[(size_t)q * n + q];
                if (apq == 0.0) continue;
                if (fabs(apq) <= DBL_EPSILON * 1e-3 * sqrt(fabs(app) * fabs(aqq)) + floor_abs) {
                    S[(size_t)p * n + q] = S[(size_t)q * n + p] = 0.0;
                    continue;
                }
                rotated = 1;
                double theta = (aqq - app) / (2.0 * apq);
                double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
                double c = 1.0 / sqrt(t * t + 1.0), s = t * c;
                for (int r = 0; r < n; ++r) {             /* columns p, q */
                    double arp = S[(size_t)r * n + p], arq = S[(size_t)r * n + q];
                    S[(size_t)r * n + p] = c * arp - s * arq;
                    S[(size_t)r * n + q] = s * arp + c * arq;
                }
                for (int r = 0; r < n; ++r) {             /* rows p, q */
                    double apr = S[(size_t)p * n + r], aqr = S[(size_t)q * n + r];
                    S[(size_t)p * n + r] = c * apr - s * aqr;
                    S[(size_t)q * n + r] = s * apr + c * aqr;
                }
                for (int r = 0; r < n; ++r) {
                    double urp = U[(size_t)r * n + p], urq = U[(size_t)r * n + q];
                    U[(size_t)r * n + p] = c * urp - s * urq;
                    U[(size_t)r * n + q] = s * urp + c * urq;
                }
            }
        }
        if (!rotated) break;
    }
    /* selection sort, descending */
    int *ord = (int *)malloc((size_t)n * sizeof(int));
    for (int i = 0; i < n; ++i) ord[i] = i;
    for (int i = 0; i < n; ++i) {
        int b = i;
        for (int j = i + 1; j < n; ++j)
            if (S[(size_t)ord[j] * n + ord[j]] > S[(size_t)ord[b] * n + ord[b]]) b = j;
        int tmp = ord[i]; ord[i] = ord[b]; ord[b] = tmp;
    }
    for (int i = 0; i < n; ++i) {
        lam[i] = S[(size_t)ord[i] * n + ord[i]];
        for (int r = 0; r < n; ++r) E[(size_t)i * n + r] = U[(size_t)r * n + ord[i]];
    }
    free(ord);
    free(U);
}

/* ------------------------------------------------------------------ */
/* One (layer, KV head): Algorithm 2 (headwise) + Algorithm 3          */
/* ------------------------------------------------------------------ */
/*
 * K, V : [T, d] float32;  Q : [n_q, d] float32.
 * idx  : [k_eff] ascending retained positions.
 * K_out, V_out : [k_eff, d] double (K_out rows are exact copies; V_out = V_keep + delta).
 * Optional (may be NULL): A [T], delta [d] (scaled injection), rbar [d],
 * Delta [d] (unscaled direction, Eq. 5), eigvals [d] (of R^T R, descending),
 * proj [d*d] (C^T C, the projector onto the residual principal subspace), diag.
 * Returns k_eff.
 */
static int backfill_given_selection(const float *K, const float *V, const double *A_in,
                                    int T, int d, int k, int rank, double eps,
                                    const int32_t *idx, double kth_score, double next_score,
                                    double *K_out, double *V_out,
                                    double *delta_out, double *rbar_out, double *Delta_out,
                                    double *eigvals_out, double *proj_out, obf_oracle_diag_t *diag, int fast_iters);

int obf_oracle_head_ex(const float *K, const float *V, const float *Q,
                       int T, int d, int n_q, int budget, int rank, double eps,
                       int32_t *idx, double *K_out, double *V_out,
                       double *A_out, double *delta_out, double *rbar_out, double *Delta_out,
                       double *eigvals_out, double *proj_out, obf_oracle_diag_t *diag, int n_sink, int fast_iters);

int obf_oracle_head_sink(const float *K, const float *V, const float *Q,
                         int T, int d, int n_q, int budget, int rank, double eps,
                         int32_t *idx, double *K_out, double *V_out,
                         double *A_out, double *delta_out, double *rbar_out, double *Delta_out,
                         double *eigvals_out, double *proj_out, obf_oracle_diag_t *diag, int n_sink)
{
    return obf_oracle_head_ex(K, V, Q, T, d, n_q, budget, rank, eps, idx, K_out, V_out, A_out, delta_out, rbar_out,
                              Delta_out, eigvals_out, proj_out, diag, n_sink, 0);
}

/* fast_iters > 0: the principal subspace comes from that many steps of the Gram subspace iteration of App. H
 * instead of the exact eigen-decomposition (see backfill_given_selection). */
int obf_oracle_head_lse(const float *K, const float *V, const float *Q, const float *lse_extra,
                        int T, int d, int n_q, int budget, int rank, double eps,
                        int32_t *idx, double *K_out, double *V_out,
                        double *A_out, double *delta_out, double *rbar_out, double *Delta_out,
                        double *eigvals_out, double *proj_out, obf_oracle_diag_t *diag, int n_sink, int fast_iters);

int obf_oracle_head_ex(const float *K, const float *V, const float *Q,
                       int T, int d, int n_q, int budget, int rank, double eps,
                       int32_t *idx, double *K_out, double *V_out,
                       double *A_out, double *delta_out, double *rbar_out, double *Delta_out,
                       double *eigvals_out, double *proj_out, obf_oracle_diag_t *diag, int n_sink, int fast_iters)
{
    return obf_oracle_head_lse(K, V, Q, NULL, T, d, n_q, budget, rank, eps, idx, K_out, V_out, A_out, delta_out,
                               rbar_out, Delta_out, eigvals_out, proj_out, diag, n_sink, fast_iters);
}

/* lse_extra: out-of-prompt softmax mass per query row (see obf_oracle_scores_ext), or NULL. */
int obf_oracle_head_lse(const float *K, const float *V, const float *Q, const float *lse_extra,
                        int T, int d, int n_q, int budget, int rank, double eps,
                        int32_t *idx, double *K_out, double *V_out,
                        double *A_out, double *delta_out, double *rbar_out, double *Delta_out,
                        double *eigvals_out, double *proj_out, obf_oracle_diag_t *diag, int n_sink, int fast_iters)
{
    /* O1: attention mass */
    double *A = (double *)malloc((size_t)T * sizeof(double));
    obf_oracle_scores_ext(K, Q, lse_extra, T, d, n_q, A);
    if (A_out) memcpy(A_out, A, (size_t)T * sizeof(double));

    /* O2: headwise TopK_B, ascending index list */
    double kth = 0.0, next = -1.0;
    int k = obf_oracle_topk_sink(A, T, budget, n_sink, idx, &kth, &next);

    backfill_given_selection(K, V, A, T, d, k, rank, eps, idx, kth, next, K_out, V_out,
                             delta_out, rbar_out, Delta_out, eigvals_out, proj_out, diag, fast_iters);
    free(A);
    return k;
}

int obf_oracle_head(const float *K, const float *V, const float *Q,
                    int T, int d, int n_q, int budget, int rank, double eps,
                    int32_t *idx, double *K_out, double *V_out,
                    double *A_out, double *delta_out, double *rbar_out, double *Delta_out,
                    double *eigvals_out, double *proj_out, obf_oracle_diag_t *diag)
{
    return obf_oracle_head_sink(K, V, Q, T, d, n_q, budget, rank, eps, idx, K_out, V_out, A_out, delta_out, rbar_out,
                                Delta_out, eigvals_out, proj_out, diag, 0);
}

/*
 * Everything after the selection (last step of Algorithm 2, then Algorithm 3) for one (layer, KV head):
 * A_in are this head's own attention masses, idx the k retained positions (ascending), whichever
 * granularity chose them.  kth_score / next_score are passed through to the diagnostics.
 */
static int backfill_given_selection(const float *K, const float *V, const double *A_in,
                                    int T, int d, int k, int rank, double eps,
                                    const int32_t *idx, double kth_score, double next_score,
                                    double *K_out, double *V_out,
                                    double *delta_out, double *rbar_out, double *Delta_out,
                                    double *eigvals_out, double *proj_out, obf_oracle_diag_t *diag, int fast_iters)
{
    obf_oracle_diag_t dg;
    memset(&dg, 0, sizeof(dg));
    dg.kth_score = kth_score;
    dg.next_score = next_score;
    double *A = (double *)malloc((size_t)T * sizeof(double));
    memcpy(A, A_in, (size_t)T * sizeof(double));

    /* O3: gather (Algorithm 2, last step) */
    for (int r = 0; r < k; ++r)
        for (int c = 0; c < d; ++c) {
            K_out[(size_t)r * d + c] = (double)K[(size_t)idx[r] * d + c];
            V_out[(size_t)r * d + c] = (double)V[(size_t)idx[r] * d + c];
        }

    if (delta_out)   for (int c = 0; c < d; ++c) delta_out[c] = 0.0;
    if (rbar_out)    for (int c = 0; c < d; ++c) rbar_out[c] = 0.0;
    if (Delta_out)   for (int c = 0; c < d; ++c) Delta_out[c] = 0.0;
    if (eigvals_out) for (int c = 0; c < d; ++c) eigvals_out[c] = 0.0;
    if (proj_out)    for (int c = 0; c < d * d; ++c) proj_out[c] = 0.0;

    /* deleted positions, ascending (Algorithm 3: P_del = P \ P_keep) */
    int N = T - k;
    dg.n_del = N;
    char *keep = (char *)calloc((size_t)T, 1);
    for (int r = 0; r < k; ++r) keep[idx[r]] = 1;

    /* O5: demand sums (Eq. 6) - also reported for eviction-only heads */
    for (int j = 0; j < T; ++j) { if (keep[j]) dg.a_keep += A[j]; else dg.a_del += A[j]; }
    dg.alpha = dg.a_del / (dg.a_keep + eps);

    /* O4: footnote to Eq. 7 - nothing deleted, or rank 0: plain eviction */
    if (N == 0 || rank <= 0) {
        dg.skipped = 1;
        if (diag) *diag = dg;
        free(keep); free(A);
        return k;
    }

    int *del = (int *)malloc((size_t)N * sizeof(int));
    { int n = 0; for (int j = 0; j < T; ++j) if (!keep[j]) del[n++] = j; }

    /* O6: Q = orth(V_keep^T), Eq. 2 (rows of Qb span the retained values) */
    double *Qb = (double *)malloc((size_t)(k < d ? k : d) * d * sizeof(double));
    int m = obf_oracle_span_basis(V_out, k, d, Qb);
    dg.span_rank = m;

    /* O7: R = V_del - (V_del Q) Q^T, Eq. 3 */
    double *R = (double *)malloc((size_t)N * d * sizeof(double));
    double *coef = (double *)malloc((size_t)(m > 0 ? m : 1) * sizeof(double));
    for (int n = 0; n < N; ++n) {
        const float *v = V + (size_t)del[n] * d;
        double *r = R + (size_t)n * d;
        for (int c = 0; c < d; ++c) { r[c] = (double)v[c]; dg.vdel_fro2 += r[c] * r[c]; }
        for (int i = 0; i < m; ++i) {
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += (double)v[c] * Qb[(size_t)i * d + c];
            coef[i] = dot;
        }
        for (int i = 0; i < m; ++i)
            for (int c = 0; c < d; ++c) r[c] -= coef[i] * Qb[(size_t)i * d + c];
        for (int c = 0; c < d; ++c) dg.r_fro2 += r[c] * r[c];
    }
    dg.rcr = dg.r_fro2 / (dg.vdel_fro2 + eps);
    {   /* PC (App. K.2): CosSim(sum_j V_del[j,:], sum_j V_par[j,:]) with V_par = V_del - R */
        double ss = 0.0, pp = 0.0, sp = 0.0;
        for (int c = 0; c < d; ++c) {
            double sv = 0.0, sr = 0.0;
            for (int n = 0; n < N; ++n) { sv += (double)V[(size_t)del[n] * d + c]; sr += R[(size_t)n * d + c]; }
            const double par = sv - sr;
            ss += sv * sv; pp += par * par; sp += sv * par;
        }
        dg.pc = (ss > 0.0 && pp > 0.0) ? sp / (sqrt(ss) * sqrt(pp)) : 0.0;
    }

    /* O8: residual of negligible Frobenius norm -> skip (footnote to Eq. 7) */
    if (dg.r_fro2 <= 1e-12 * dg.vdel_fro2) {
        dg.skipped = 1;
        if (diag) *diag = dg;
        free(coef); free(R); free(Qb); free(del); free(keep); free(A);
        return k;
    }

    /* O9: top right singular vectors of R = top eigenvectors of R^T R (no centring) */
    double *G = (double *)calloc((size_t)d * d, sizeof(double));
    for (int n = 0; n < N; ++n) {
        const double *r = R + (size_t)n * d;
        for (int a = 0; a < d; ++a) {
            double ra = r[a];
            for (int b = 0; b < d; ++b) G[(size_t)a * d + b] += ra * r[b];
        }
    }
    double *lam = (double *)malloc((size_t)d * sizeof(double));
    double *E = (double *)malloc((size_t)d * d * sizeof(double));
    obf_oracle_sym_eig(G, d, lam, E);
    if (eigvals_out) memcpy(eigvals_out, lam, (size_t)d * sizeof(double));
    int rankR = 0;
    for (int i = 0; i < d; ++i) if (lam[i] > (double)d * DBL_EPSILON * lam[0]) ++rankR;
    int rho = rank < rankR ? rank : rankR;          /* k = min(pca_rank, rank(R)) */
    dg.rho_eff = rho;
    dg.lam_1 = lam[0];
    dg.lam_rho = rho > 0 ? lam[rho - 1] : 0.0;
    dg.lam_next = rho < d ? lam[rho] : 0.0;
    { double kept = 0.0, all = 0.0;
      for (int i = 0; i < d; ++i) { all += lam[i]; if (i < rho) kept += lam[i]; }
      dg.revr = kept / (all + eps); }

    /*
     * App. H ("fast path"): instead of the eigenvectors, C_0 with orthonormal rows, then
     * C_{t+1} = orth(C_t G) for t = 0 .. fast_iters - 1 with G = R^T R.  The paper leaves C_0 open; here it is the
     * first rows of the identity.  orth() is Gram-Schmidt over the rows in order, twice, which spans what a thin QR
     * spans; a row that has nothing left after its predecessors were removed is dropped.
     */
    if (fast_iters > 0) {
        int rho_f = rank < d - m ? rank : d - m;          /* rank(R) <= d - m */
        double *Gc = (double *)calloc((size_t)d * d, sizeof(double));
        for (int n = 0; n < N; ++n) {
            const double *r = R + (size_t)n * d;
            for (int a = 0; a < d; ++a) { double ra = r[a]; for (int b = 0; b < d; ++b) Gc[(size_t)a * d + b] += ra * r[b]; }
        }
        double *C = (double *)calloc((size_t)(rho_f > 0 ? rho_f : 1) * d, sizeof(double));
        double *Y = (double *)calloc((size_t)(rho_f > 0 ? rho_f : 1) * d, sizeof(double));
        for (int i = 0; i < rho_f; ++i) C[(size_t)i * d + i] = 1.0;
        for (int t = 0; t < fast_iters; ++t) {
            for (int i = 0; i < rho_f; ++i)
                for (int b = 0; b < d; ++b) {
                    double acc = 0.0;
                    for (int a = 0; a < d; ++a) acc += C[(size_t)i * d + a] * Gc[(size_t)a * d + b];
                    Y[(size_t)i * d + b] = acc;
                }
            int kept = 0;
            for (int i = 0; i < rho_f; ++i) {
                double *y = Y + (size_t)i * d;
                double n0 = 0.0; for (int c = 0; c < d; ++c) n0 += y[c] * y[c];
                for (int pass = 0; pass < 2; ++pass)
                    for (int j = 0; j < kept; ++j) {
                        const double *q = C + (size_t)j * d;
                        double dot = 0.0; for (int c = 0; c < d; ++c) dot += y[c] * q[c];
                        for (int c = 0; c < d; ++c) y[c] -= dot * q[c];
                    }
                double n1 = 0.0; for (int c = 0; c < d; ++c) n1 += y[c] * y[c];
                if (n1 > 1e-24 * n0 && n1 > 0.0) {
                    double inv = 1.0 / sqrt(n1);
                    for (int c = 0; c < d; ++c) C[(size_t)kept * d + c] = y[c] * inv;
                    ++kept;
                }
            }
            rho_f = kept;
        }
        dg.rho_eff = rho_f;
        /* eigenvalue fields: Rayleigh quotients of the rows of C; REVR from them */
        double kept_sum = 0.0, tr = 0.0;
        for (int a = 0; a < d; ++a) tr += Gc[(size_t)a * d + a];
        dg.lam_1 = dg.lam_rho = dg.lam_next = 0.0;
        for (int i = 0; i < rho_f; ++i) {
            double rq = 0.0;
            for (int a = 0; a < d; ++a) { double acc = 0.0; for (int b = 0; b < d; ++b) acc += Gc[(size_t)a * d + b] * C[(size_t)i * d + b]; rq += C[(size_t)i * d + a] * acc; }
            kept_sum += rq;
            if (i == 0) dg.lam_1 = rq;
            if (i == rho_f - 1) dg.lam_rho = rq;
        }
        dg.revr = kept_sum / (tr + eps);
        for (int i = 0; i < rho_f; ++i) memcpy(E + (size_t)i * d, C + (size_t)i * d, (size_t)d * sizeof(double));
        rho = rho_f;
        free(Y); free(C); free(Gc);
    }

    /* O10: attention-weighted residual mean, Eq. 4 */
    double *rbar = (double *)calloc((size_t)d, sizeof(double));
    for (int n = 0; n < N; ++n) {
        double w = A[del[n]] / (dg.a_del + eps);
        const double *r = R + (size_t)n * d;
        for (int c = 0; c < d; ++c) rbar[c] += w * r[c];
    }
    { double s = 0.0; for (int c = 0; c < d; ++c) s += rbar[c] * rbar[c]; dg.rbar_norm = sqrt(s); }
    if (rbar_out) memcpy(rbar_out, rbar, (size_t)d * sizeof(double));

    /* O11: Delta = (rbar C^T) C, Eq. 5; delta = alpha * Delta, Eq. 6; V* = V + delta, Eq. 7 */
    double *Delta = (double *)calloc((size_t)d, sizeof(double));
    for (int i = 0; i < rho; ++i) {
        const double *c_i = E + (size_t)i * d;
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += rbar[c] * c_i[c];
        for (int c = 0; c < d; ++c) Delta[c] += dot * c_i[c];
    }
    if (Delta_out) memcpy(Delta_out, Delta, (size_t)d * sizeof(double));
    if (proj_out)
        for (int i = 0; i < rho; ++i)
            for (int a = 0; a < d; ++a)
                for (int b = 0; b < d; ++b)
                    proj_out[(size_t)a * d + b] += E[(size_t)i * d + a] * E[(size_t)i * d + b];
    double dn = 0.0;
    for (int c = 0; c < d; ++c) {
        double dl = dg.alpha * Delta[c];
        if (delta_out) delta_out[c] = dl;
        dn += dl * dl;
        for (int r = 0; r < k; ++r) V_out[(size_t)r * d + c] += dl;     /* keys untouched */
    }
    dg.delta_norm = sqrt(dn);
    if (diag) *diag = dg;

    free(Delta); free(rbar); free(E); free(lam); free(G);
    free(coef); free(R); free(Qb); free(del); free(keep); free(A);
    return k;
}

/* ------------------------------------------------------------------ */
/* A whole cache: every (layer, KV head) independently                  */
/* ------------------------------------------------------------------ */
/*
 * K, V : [layers, kv_heads, T, d];  Q : [layers, q_heads, n_obs, d] with
 * q head = kv_head * G + g, so the n_q = G * n_obs rows of one KV head are
 * contiguous.  Outputs are [layers, kv_heads, k_eff, ...].  delta_out (may be
 * NULL) is [layers, kv_heads, d].  Heads run in parallel when built with
 * OpenMP.  Returns k_eff.
 */
int obf_oracle_compress(const float *K, const float *V, const float *Q,
                        int layers, int kv_heads, int q_heads, int n_obs, int T, int d,
                        int budget, int rank, double eps,
                        int32_t *idx_out, double *K_out, double *V_out,
                        double *delta_out, obf_oracle_diag_t *diag_out, int n_sink)
{
    const int G = q_heads / kv_heads;
    const int n_q = G * n_obs;
    const int sink = n_sink < T ? (n_sink > 0 ? n_sink : 0) : T;
    const int k = sink + (budget < T - sink ? budget : T - sink);
    const int heads = layers * kv_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int lh = 0; lh < heads; ++lh) {
        const float *Kh = K + (size_t)lh * T * d;
        const float *Vh = V + (size_t)lh * T * d;
        const float *Qh = Q + (size_t)lh * n_q * d;
        obf_oracle_head_sink(Kh, Vh, Qh, T, d, n_q, budget, rank, eps,
                             idx_out + (size_t)lh * k,
                             K_out + (size_t)lh * k * d, V_out + (size_t)lh * k * d,
                             NULL, delta_out ? delta_out + (size_t)lh * d : NULL, NULL, NULL, NULL, NULL,
                             diag_out ? diag_out + lh : NULL, n_sink);
    }
    return k;
}

/* ------------------------------------------------------------------ */
/* Layerwise granularity (Algorithm 2, granularity L) + Algorithm 3     */
/* ------------------------------------------------------------------ */
/*
 * One layer: K, V [kv_heads, T, d]; Q [kv_heads, n_q, d].  The retained set is
 * TopK_B of the masses summed over the layer's KV heads (retention rule of
 * Section 3.2, second form) and is shared by all heads of the layer; the gather
 * and Orthogonal BackFill then run per head with that head's own masses
 * (Eq. 4 and Eq. 6 are written per (l, h)).  Outputs are [kv_heads, k_eff, ...];
 * S_out (may be NULL) receives the T summed masses, A_out (may be NULL) the
 * [kv_heads, T] per-head masses.  Returns k_eff.
 */
int obf_oracle_layer(const float *K, const float *V, const float *Q,
                     int kv_heads, int T, int d, int n_q, int budget, int rank, double eps,
                     int32_t *idx_out, double *K_out, double *V_out,
                     double *S_out, double *A_out, double *delta_out, obf_oracle_diag_t *diag_out, int n_sink)
{
    double *A = (double *)malloc((size_t)kv_heads * T * sizeof(double));
    double *S = (double *)calloc((size_t)T, sizeof(double));
    for (int h = 0; h < kv_heads; ++h) {
        obf_oracle_scores(K + (size_t)h * T * d, Q + (size_t)h * n_q * d, T, d, n_q, A + (size_t)h * T);
        for (int j = 0; j < T; ++j) S[j] += A[(size_t)h * T + j];
    }
    if (S_out) memcpy(S_out, S, (size_t)T * sizeof(double));
    if (A_out) memcpy(A_out, A, (size_t)kv_heads * T * sizeof(double));
    int32_t *idx = (int32_t *)malloc((size_t)T * sizeof(int32_t));
    double kth = 0.0, next = -1.0;
    const int k = obf_oracle_topk_sink(S, T, budget, n_sink, idx, &kth, &next);
    for (int h = 0; h < kv_heads; ++h) {
        memcpy(idx_out + (size_t)h * k, idx, (size_t)k * sizeof(int32_t));
        backfill_given_selection(K + (size_t)h * T * d, V + (size_t)h * T * d, A + (size_t)h * T, T, d, k, rank, eps,
                                 idx, kth, next, K_out + (size_t)h * k * d, V_out + (size_t)h * k * d,
                                 delta_out ? delta_out + (size_t)h * d : NULL, NULL, NULL, NULL, NULL,
                                 diag_out ? diag_out + h : NULL, 0);
    }
    free(idx); free(S); free(A);
    return k;
}

/* A whole cache with the layerwise selector; arrays as in obf_oracle_compress. */
int obf_oracle_compress_layerwise(const float *K, const float *V, const float *Q,
                                  int layers, int kv_heads, int q_heads, int n_obs, int T, int d,
                                  int budget, int rank, double eps,
                                  int32_t *idx_out, double *K_out, double *V_out,
                                  double *delta_out, obf_oracle_diag_t *diag_out, int n_sink)
{
    const int G = q_heads / kv_heads;
    const int n_q = G * n_obs;
    const int sink = n_sink < T ? (n_sink > 0 ? n_sink : 0) : T;
    const int k = sink + (budget < T - sink ? budget : T - sink);
#pragma omp parallel for schedule(dynamic, 1)
    for (int l = 0; l < layers; ++l) {
        const size_t lh = (size_t)l * kv_heads;
        obf_oracle_layer(K + lh * T * d, V + lh * T * d, Q + lh * n_q * d, kv_heads, T, d, n_q, budget, rank, eps,
                         idx_out + lh * k, K_out + lh * k * d, V_out + lh * k * d, NULL, NULL,
                         delta_out ? delta_out + lh * d : NULL, diag_out ? diag_out + lh : NULL, n_sink);
    }
    return k;
}

/*
 * Algorithm 3 for a retained set chosen elsewhere: masses A [T] and k ascending positions idx are given (the
 * last step of Algorithm 2 and everything after it).  For checking a result whose positions differ from this
 * oracle's inside the tie band: the back-fill is then compared on the positions that were actually retained.
 */
int obf_oracle_backfill(const float *K, const float *V, const double *A, int T, int d, int k, int rank, double eps,
                        const int32_t *idx, double *K_out, double *V_out, double *delta_out, obf_oracle_diag_t *diag)
{
    return backfill_given_selection(K, V, A, T, d, k, rank, eps, idx, 0.0, -1.0, K_out, V_out, delta_out,
                                    NULL, NULL, NULL, NULL, diag, 0);
}

/*
 * Attn-inject (App. D.2, alternative designs): the back-fill vector delta of Eq. 6 is not added uniformly but in
 * proportion to each retained position's attention mass,
 *   V*_t = V_t + B * w_t * delta,   w_t = A_t / (sum over retained s of A_s + eps),   B = number of retained positions,
 * so that the shares average one.  V [T, d], A [T], idx [k] ascending, delta [d] (the vector obf_oracle_head returns);
 * V_out [k, d].
 */
void obf_oracle_attn_inject(const float *V, const double *A, const int32_t *idx, int k, int d, const double *delta,
                            double eps, double *V_out)
{
    double a_keep = 0.0;
    for (int r = 0; r < k; ++r) a_keep += A[idx[r]];
    for (int r = 0; r < k; ++r) {
        const double w = (double)k * A[idx[r]] / (a_keep + eps);
        for (int c = 0; c < d; ++c) V_out[(size_t)r * d + c] = (double)V[(size_t)idx[r] * d + c] + w * delta[c];
    }
}

/* ------------------------------------------------------------------ */
/* Cache-merging baseline (App. E)                                      */
/* ------------------------------------------------------------------ */
/*
 * The comparison method of App. E on one (layer, KV head): (i) the same attention selector picks the retained
 * positions; (ii) every deleted position j is routed to the retained position whose key has the largest cosine
 * similarity with K_j (ties: the lowest position; a key of zero norm has similarity 0 with everything);
 * (iii) V*_t = V_t + sum over the j routed to t of A_j / (A_t + eps) * V_j; keys unchanged.
 * Outputs: idx [k], K_out, V_out [k, d], A_out [T] (may be NULL), assign [T] (slot 0..k-1 a deleted position is
 * routed to, -1 for retained positions; may be NULL), margin [T] (best minus second-best similarity of a deleted
 * position, +inf with a single retained position or for retained positions; may be NULL).  Returns k.
 */
int obf_oracle_merge_head(const float *K, const float *V, const float *Q, int T, int d, int n_q, int budget, double eps,
                          int n_sink, int32_t *idx, double *K_out, double *V_out, double *A_out, int32_t *assign,
                          double *margin)
{
    double *A = (double *)malloc((size_t)T * sizeof(double));
    obf_oracle_scores(K, Q, T, d, n_q, A);
    if (A_out) memcpy(A_out, A, (size_t)T * sizeof(double));
    double kth = 0.0, next = -1.0;
    const int k = obf_oracle_topk_sink(A, T, budget, n_sink, idx, &kth, &next);
    char *keep = (char *)calloc((size_t)T, 1);
    double *norm = (double *)malloc((size_t)T * sizeof(double));
    for (int j = 0; j < T; ++j) {
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += (double)K[(size_t)j * d + c] * (double)K[(size_t)j * d + c];
        norm[j] = sqrt(s);
    }
    for (int r = 0; r < k; ++r) {
        keep[idx[r]] = 1;
        for (int c = 0; c < d; ++c) {
            K_out[(size_t)r * d + c] = (double)K[(size_t)idx[r] * d + c];
            V_out[(size_t)r * d + c] = (double)V[(size_t)idx[r] * d + c];
        }
    }
    for (int j = 0; j < T; ++j) {
        if (assign) assign[j] = -1;
        if (margin) margin[j] = INFINITY;
        if (keep[j]) continue;
        int best_r = 0;
        double best = -INFINITY, second = -INFINITY;
        for (int r = 0; r < k; ++r) {
            const int t = idx[r];
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += (double)K[(size_t)j * d + c] * (double)K[(size_t)t * d + c];
            const double den = norm[j] * norm[t];
            const double cs = den > 0.0 ? dot / den : 0.0;
            if (cs > best) { second = best; best = cs; best_r = r; }
            else if (cs > second) second = cs;
        }
        if (assign) assign[j] = best_r;
        if (margin) margin[j] = k > 1 ? best - second : INFINITY;
        const double w = A[j] / (A[idx[best_r]] + eps);
        for (int c = 0; c < d; ++c) V_out[(size_t)best_r * d + c] += w * (double)V[(size_t)j * d + c];
    }
    free(norm); free(keep); free(A);
    return k;
}

/* Step (iii) alone for a given routing (assign as above): for checking a result whose routing differs from this
 * oracle's where two similarities are closer than the arithmetic can tell apart. */
void obf_oracle_merge_given(const float *V, const double *A, const int32_t *idx, int k, const int32_t *assign,
                            int T, int d, double eps, double *V_out)
{
    for (int r = 0; r < k; ++r)
        for (int c = 0; c < d; ++c) V_out[(size_t)r * d + c] = (double)V[(size_t)idx[r] * d + c];
    for (int j = 0; j < T; ++j) {
        if (assign[j] < 0) continue;
        const double w = A[j] / (A[idx[assign[j]]] + eps);
        for (int c = 0; c < d; ++c) V_out[(size_t)assign[j] * d + c] += w * (double)V[(size_t)j * d + c];
    }
}

/* ------------------------------------------------------------------ */
/* Post-hoc int8 quantisation of the compacted relay (App. E)          */
/* ------------------------------------------------------------------ */
/*
 * The paper stacks int8 quantisation on the compressed relay (App. E, Table 7) without fixing the quantiser.
 * Reading taken: symmetric, one fp32 scale per row (one retained position of one KV head),
 *   scale = max_c |x_c| / 127,   code_c = round-half-even(x_c / scale) in [-127, 127],   x_c ~ code_c * scale;
 * a row of zeros gets scale 0 and codes 0.  With head_dim 128 a row shrinks from 256 to 132 bytes, the factor
 * 1.94 by which Table 7's ratio grows from 4.6 to 9.0.  The decision of a code is taken in float32 (the
 * precision of the scale that is stored), on both sides.
 * X [rows, d] float32 (bf16 values up-cast exactly); codes [rows, d]; scales [rows].
 */
void obf_oracle_quantize_rows(const float *X, int rows, int d, int8_t *codes, float *scales)
{
    for (int r = 0; r < rows; ++r) {
        const float *x = X + (size_t)r * d;
        float amax = 0.0f;
        for (int c = 0; c < d; ++c) { const float a = fabsf(x[c]); if (a > amax) amax = a; }
        const float scale = amax / 127.0f;
        scales[r] = scale;
        for (int c = 0; c < d; ++c) {
            float q = scale > 0.0f ? rintf(x[c] / scale) : 0.0f;
            if (q > 127.0f) q = 127.0f;
            if (q < -127.0f) q = -127.0f;
            codes[(size_t)r * d + c] = (int8_t)q;
        }
    }
}

int obf_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
