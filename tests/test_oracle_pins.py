"""Pins for the CPU oracle: closed forms, invariants, brute force, library routines.

None of these tests needs a GPU.  Each pins one stage of the oracle to
something other than the oracle itself, so that a dropped term, a wrong sign or
index, or a transposed operand in ``oracle/obf_oracle.c`` fails at least one.
"""
import math
import os

import numpy as np
import pytest
import scipy.special

import oracle
from paper_2604_13349_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------
# independent statements built from library routines
# --------------------------------------------------------------------------
def lib_scores(K, Q):
    """Eq. 1 through scipy's softmax (fp64)."""
    K = K.astype(np.float64); Q = Q.astype(np.float64)
    S = Q @ K.T / math.sqrt(K.shape[1])
    return scipy.special.softmax(S, axis=1).sum(axis=0)


def brute_topk(A, k):
    order = sorted(range(len(A)), key=lambda j: (-A[j], j))
    return np.array(sorted(order[:min(k, len(A))]), dtype=np.int32)


def lib_obf(K, V, Q, budget, rank, eps=1e-12):
    """Algorithm 3 through LAPACK routines: pinv for the span projector, SVD of the explicit residual."""
    A = lib_scores(K, Q)
    T = K.shape[0]
    k = min(budget, T)
    idx = np.sort(np.argsort(-A, kind="stable")[:k]).astype(np.int32)
    keep = np.zeros(T, bool); keep[idx] = True
    Vd = V.astype(np.float64)
    Vk, Vdel = Vd[keep], Vd[~keep]
    out = {"idx": idx, "A": A, "delta": np.zeros(V.shape[1]), "V_out": Vk.copy()}
    if rank <= 0 or Vdel.shape[0] == 0:
        return out
    Pi = np.linalg.pinv(Vk) @ Vk                      # projector onto the row space of V_keep
    R = Vdel - Vdel @ Pi
    a_del, a_keep = A[~keep].sum(), A[keep].sum()
    out["rcr"] = (R ** 2).sum() / ((Vdel ** 2).sum() + eps)
    ssum = Vdel.sum(axis=0); psum = ssum @ Pi               # sum of the deleted values and of their projections
    out["pc"] = float(ssum @ psum / (np.linalg.norm(ssum) * np.linalg.norm(psum)))
    if (R ** 2).sum() <= 1e-12 * (Vdel ** 2).sum():
        return out
    _, s, Vt = np.linalg.svd(R, full_matrices=False)
    rho = min(rank, int((s ** 2 > V.shape[1] * np.finfo(float).eps * s[0] ** 2).sum()))
    C = Vt[:rho]
    w = A[~keep] / (a_del + eps)
    rbar = w @ R
    Delta = (rbar @ C.T) @ C
    delta = a_del / (a_keep + eps) * Delta
    out.update(delta=delta, rbar=rbar, Delta=Delta, proj=C.T @ C, V_out=Vk + delta, sing=s)
    return out


def rand_head(seed, T, d, n_q, heavy=0):
    g = np.random.default_rng(seed)
    K = g.standard_normal((T, d)).astype(np.float32)
    V = g.standard_normal((T, d)).astype(np.float32)
    Q = g.standard_normal((n_q, d)).astype(np.float32)
    if heavy:
        K[g.choice(T, heavy, replace=False)] *= 3.0
    return K, V, Q


# --------------------------------------------------------------------------
# scores (Eq. 1)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("T,d,n_q", [(1, 8, 3), (2, 4, 1), (37, 16, 5), (256, 64, 64), (300, 128, 7)])
def test_scores_sum_to_number_of_queries(T, d, n_q):
    K, _, Q = rand_head(T * 7 + d, T, d, n_q)
    A = oracle.scores(K, Q)
    assert A.shape == (T,)
    assert np.all(A >= 0)
    assert abs(A.sum() - n_q) < 1e-10 * n_q


def test_scores_equal_keys_are_uniform():
    g = np.random.default_rng(1)
    k = g.standard_normal(32).astype(np.float32)
    K = np.tile(k, (50, 1))
    Q = g.standard_normal((9, 32)).astype(np.float32)
    A = oracle.scores(K, Q)
    np.testing.assert_allclose(A, 9 / 50, rtol=1e-13)


def test_scores_two_keys_closed_form_sigmoid():
    # T = 2, one query: a_1 = sigmoid(s_1 - s_2) with s = q.k / sqrt(d); d = 16 so the scale is 1/4.
    q = np.zeros((1, 16), np.float32); q[0, :3] = [1.0, -2.0, 0.5]
    K = np.zeros((2, 16), np.float32); K[0, :3] = [3.0, 1.0, 2.0]; K[1, :3] = [-1.0, 0.5, 4.0]
    s1 = (1 * 3 - 2 * 1 + 0.5 * 2) / 4.0
    s2 = (-1 - 1 + 2) / 4.0
    a1 = 1.0 / (1.0 + math.exp(-(s1 - s2)))
    A = oracle.scores(K, q)
    np.testing.assert_allclose(A, [a1, 1 - a1], rtol=1e-14)


@pytest.mark.parametrize("seed", range(4))
def test_scores_match_library_softmax(seed):
    K, _, Q = rand_head(seed, 111, 24, 13, heavy=5)
    np.testing.assert_allclose(oracle.scores(K, Q), lib_scores(K, Q), rtol=1e-12, atol=1e-15)


def test_scores_large_logits_do_not_overflow():
    K, _, Q = rand_head(3, 40, 8, 4)
    K *= 400.0                                        # logits of order 1e3: exp overflows without the max shift
    A = oracle.scores(K, Q)
    assert np.all(np.isfinite(A))
    np.testing.assert_allclose(A, lib_scores(K, Q), rtol=1e-12, atol=1e-300)


def test_scores_permutation_equivariance():
    K, _, Q = rand_head(5, 64, 16, 6)
    g = np.random.default_rng(0)
    pk, pq = g.permutation(64), g.permutation(6)
    A = oracle.scores(K, Q)
    np.testing.assert_allclose(oracle.scores(K[pk], Q), A[pk], rtol=1e-13)
    np.testing.assert_allclose(oracle.scores(K, Q[pq]), A, rtol=1e-13)


# out-of-prompt softmax mass (Section 3.1: the attention weights are a softmax over the whole cache)
def test_scores_with_no_out_of_prompt_mass_are_the_plain_scores():
    K, _, Q = rand_head(7, 90, 16, 5)
    A = oracle.scores(K, Q)
    assert np.array_equal(oracle.scores(K, Q, np.full(5, -np.inf, np.float32)), A)
    np.testing.assert_allclose(oracle.scores(K, Q, np.full(5, -200.0, np.float32)), A, rtol=1e-13)


@pytest.mark.parametrize("seed", range(3))
def test_scores_with_out_of_prompt_mass_equal_an_appended_key_that_is_dropped(seed):
    # one more key behind the prompt, whose logit per query IS that query's out-of-prompt log-sum-exp
    K, _, Q = rand_head(seed, 70, 16, 6, heavy=3)
    extra = np.random.default_rng(seed).standard_normal(16).astype(np.float32) * 2
    lse = ((Q.astype(np.float64) @ extra.astype(np.float64)) / 4.0).astype(np.float32)     # 1 / sqrt(16)
    # the logits of the appended key as the oracle would see them: recompute from the float32 lse for equality
    full = oracle.scores(np.vstack([K, extra[None]]), Q)
    part = oracle.scores(K, Q, lse)
    np.testing.assert_allclose(part, full[:70], rtol=1e-6)          # lse is rounded to float32: 6e-8 in the logit
    assert part.sum() < 6.0
    np.testing.assert_allclose(part.sum() + full[70], 6.0, rtol=1e-6)


def test_scores_with_out_of_prompt_mass_match_library_logsumexp():
    from scipy.special import logsumexp
    K, _, Q = rand_head(11, 120, 32, 7, heavy=4)
    lse = np.linspace(-3.0, 9.0, 7).astype(np.float32)
    S = (Q.astype(np.float64) @ K.astype(np.float64).T) / math.sqrt(32)
    denom = logsumexp(np.concatenate([S, lse.astype(np.float64)[:, None]], axis=1), axis=1)
    ref = np.exp(S - denom[:, None]).sum(axis=0)
    np.testing.assert_allclose(oracle.scores(K, Q, lse), ref, rtol=1e-12)
    # and through the whole head: the selection runs on these masses
    _, V, _ = rand_head(12, 120, 32, 7)
    h = oracle.head(K, V, Q, 10, 1, lse_extra=lse)
    np.testing.assert_allclose(h["A"], ref, rtol=1e-12)
    assert np.array_equal(h["idx"], np.sort(np.argsort(-ref, kind="stable")[:10]))


# --------------------------------------------------------------------------
# top-k (Section 4.3.2, ties to the lowest index, ascending output)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(6))
def test_topk_matches_brute_force_and_stable_argsort(seed):
    g = np.random.default_rng(seed)
    T = int(g.integers(1, 60))
    A = g.random(T)
    A[g.integers(0, T, size=T // 3)] = A[0]           # plant exact ties
    for k in {1, T // 2 or 1, T, T + 5}:
        idx, kth, nxt = oracle.topk(A, k)
        np.testing.assert_array_equal(idx, brute_topk(A, k))
        np.testing.assert_array_equal(idx, np.sort(np.argsort(-A, kind="stable")[:min(k, T)]))
        srt = np.sort(A)[::-1]
        assert kth == srt[min(k, T) - 1]
        assert nxt == (srt[k] if k < T else -1.0)


def test_topk_all_equal_keeps_the_first_positions():
    idx, _, _ = oracle.topk(np.full(17, 0.25), 5)
    np.testing.assert_array_equal(idx, np.arange(5))


def test_topk_tie_at_the_boundary_goes_to_the_lower_index():
    A = np.array([0.1, 0.7, 0.3, 0.7, 0.3, 0.3, 0.05])
    idx, kth, nxt = oracle.topk(A, 3)                 # two 0.7s, then the first 0.3
    np.testing.assert_array_equal(idx, [1, 2, 3])
    assert kth == 0.3 and nxt == 0.3


# --------------------------------------------------------------------------
# span basis (Eq. 2)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("k,d,r", [(5, 16, 5), (16, 16, 16), (40, 16, 16), (12, 32, 7), (30, 8, 3), (1, 4, 1)])
def test_span_basis_is_orthonormal_and_spans_the_rows(k, d, r):
    g = np.random.default_rng(k * 100 + d)
    X = g.standard_normal((k, r)) @ g.standard_normal((r, d))       # rank r by construction
    Qb = oracle.span_basis(X)
    assert Qb.shape == (r, d)
    assert Qb.shape[0] == np.linalg.matrix_rank(X)
    np.testing.assert_allclose(Qb @ Qb.T, np.eye(r), atol=1e-12)
    np.testing.assert_allclose(X - (X @ Qb.T) @ Qb, 0, atol=1e-10)
    np.testing.assert_allclose(Qb.T @ Qb, np.linalg.pinv(X) @ X, atol=1e-10)


def test_span_basis_duplicates_zero_rows_and_zero_matrix():
    g = np.random.default_rng(9)
    x = g.standard_normal((3, 10))
    X = np.vstack([x, x[1:2], np.zeros((2, 10)), 2.0 * x[0:1]])
    assert oracle.span_basis(X).shape == (3, 10)
    assert oracle.span_basis(np.zeros((4, 6))).shape[0] == 0


# --------------------------------------------------------------------------
# symmetric eigen-solver (Gram form of the residual SVD, App. H)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("n,r", [(1, 1), (6, 6), (24, 24), (24, 5), (64, 40)])
def test_sym_eig_matches_lapack(n, r):
    g = np.random.default_rng(n + r)
    B = g.standard_normal((r + 3, r)) @ g.standard_normal((r, n))
    S = B.T @ B
    lam, E = oracle.sym_eig(S)
    ref = np.linalg.eigvalsh(S)[::-1]
    np.testing.assert_allclose(lam, ref, atol=1e-11 * max(ref[0], 1))
    np.testing.assert_allclose(E @ E.T, np.eye(n), atol=1e-12)
    np.testing.assert_allclose(E @ S @ E.T, np.diag(lam), atol=1e-10 * max(ref[0], 1))


def test_sym_eig_repeated_eigenvalues():
    g = np.random.default_rng(2)
    Qm, _ = np.linalg.qr(g.standard_normal((10, 10)))
    S = Qm @ np.diag([3, 3, 3, 1, 1, 0, 0, 0, 0, 0.0]) @ Qm.T
    lam, E = oracle.sym_eig(S)
    np.testing.assert_allclose(lam, [3, 3, 3, 1, 1, 0, 0, 0, 0, 0], atol=1e-12)
    P3 = E[:3].T @ E[:3]
    np.testing.assert_allclose(P3, Qm[:, :3] @ Qm[:, :3].T, atol=1e-12)


# --------------------------------------------------------------------------
# gather and the eviction-only special cases
# --------------------------------------------------------------------------
def test_gather_is_bitwise_and_rank0_is_plain_eviction():
    K, V, Q = rand_head(11, 90, 16, 8, heavy=6)
    r0 = oracle.head(K, V, Q, budget=12, rank=0)
    r2 = oracle.head(K, V, Q, budget=12, rank=2)
    idx = r0["idx"]
    np.testing.assert_array_equal(idx, brute_topk(lib_scores(K, Q), 12))
    np.testing.assert_array_equal(r2["idx"], idx)
    assert np.array_equal(r0["K_out"], K[idx].astype(np.float64))
    assert np.array_equal(r0["V_out"], V[idx].astype(np.float64))
    assert np.array_equal(r2["K_out"], K[idx].astype(np.float64))       # keys never change (Eq. 7)
    assert r0["diag"]["skipped"] == 1 and np.all(r0["delta"] == 0)
    assert np.linalg.norm(r2["delta"]) > 0


@pytest.mark.parametrize("budget", [50, 51, 1000])
def test_budget_at_least_T_is_the_identity(budget):
    K, V, Q = rand_head(12, 50, 8, 4)
    r = oracle.head(K, V, Q, budget=budget, rank=3)
    np.testing.assert_array_equal(r["idx"], np.arange(50))
    assert np.array_equal(r["K_out"], K.astype(np.float64))
    assert np.array_equal(r["V_out"], V.astype(np.float64))
    assert r["diag"]["skipped"] == 1 and r["diag"]["n_del"] == 0


# --------------------------------------------------------------------------
# OBF proper (Eq. 2-7)
# --------------------------------------------------------------------------
def _read_golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or ":" not in line:
                continue
            key, rest = line.split(":", 1)
            vals[key.strip()] = np.array([float(x) for x in rest.split()])
    return vals


@pytest.mark.parametrize("rank", [1, 2, 3])
def test_hand_worked_planted_example(rank):
    g = _read_golden("planted_obf_example.txt")
    T, d, budget = int(g["T"][0]), int(g["d"][0]), int(g["budget"][0])
    H = g["H"].reshape(d, d)
    K = np.zeros((T, d), np.float32); K[:, 0] = np.log(g["w"]).astype(np.float32)
    Q = g["q"].reshape(1, d).astype(np.float32)
    V = (g["U"].reshape(T, d) @ H).astype(np.float32)           # halves and integers: exact in float32
    r = oracle.head(K, V, Q, budget=budget, rank=rank)
    np.testing.assert_allclose(r["A"], g["A"], rtol=1e-6)
    np.testing.assert_array_equal(r["idx"], g["idx"].astype(np.int32))
    np.testing.assert_allclose(r["diag"]["a_keep"], g["a_keep"][0], rtol=1e-6)
    np.testing.assert_allclose(r["diag"]["a_del"], g["a_del"][0], rtol=1e-6)
    np.testing.assert_allclose(r["diag"]["alpha"], g["alpha"][0], rtol=1e-6)
    np.testing.assert_allclose(r["rbar"], g["rbar_U"] @ H, atol=1e-6)
    exp_delta = (g["delta_U_rank1"] if rank == 1 else g["delta_U_rank2"]) @ H
    np.testing.assert_allclose(r["delta"], exp_delta, atol=1e-6)
    np.testing.assert_allclose(r["eigvals"][:2], g["eig_top2"], rtol=1e-12)
    np.testing.assert_allclose(r["V_out"], V[:2].astype(np.float64) + exp_delta, atol=1e-6)
    assert r["diag"]["span_rank"] == 2
    assert r["diag"]["rho_eff"] == min(rank, 2)


@pytest.mark.parametrize("seed,T,d,n_q,budget,rank", [
    (0, 80, 16, 6, 5, 1), (1, 80, 16, 6, 5, 3), (2, 200, 32, 12, 20, 2),
    (3, 64, 24, 4, 23, 4), (4, 300, 64, 16, 32, 2), (5, 40, 8, 3, 3, 8)])
def test_obf_matches_lapack_pipeline(seed, T, d, n_q, budget, rank):
    K, V, Q = rand_head(seed, T, d, n_q, heavy=3)
    r = oracle.head(K, V, Q, budget=budget, rank=rank)
    ref = lib_obf(K, V, Q, budget, rank)
    np.testing.assert_array_equal(r["idx"], ref["idx"])
    np.testing.assert_allclose(r["A"], ref["A"], rtol=1e-12)
    np.testing.assert_allclose(r["rbar"], ref["rbar"], atol=1e-11)
    np.testing.assert_allclose(r["eigvals"][:len(ref["sing"])], ref["sing"] ** 2,
                               atol=1e-9 * ref["sing"][0] ** 2)
    # diagnostics of App. K.2: kept share of the squared singular values (REVR), residual content ratio (RCR)
    rho = r["diag"]["rho_eff"]
    assert r["diag"]["revr"] == pytest.approx((ref["sing"][:rho] ** 2).sum() / (ref["sing"] ** 2).sum(), rel=1e-9)
    assert r["diag"]["rcr"] == pytest.approx(ref["rcr"], rel=1e-9)
    assert r["diag"]["pc"] == pytest.approx(ref["pc"], abs=1e-10)             # projection cosine (PC)
    np.testing.assert_allclose(r["proj"], ref["proj"], atol=1e-8)      # sign/rotation free comparison
    np.testing.assert_allclose(r["Delta"], ref["Delta"], atol=1e-9)
    np.testing.assert_allclose(r["delta"], ref["delta"], atol=1e-9)
    np.testing.assert_allclose(r["V_out"], ref["V_out"], atol=1e-9)
    np.testing.assert_allclose(r["diag"]["rcr"], ref["rcr"], rtol=1e-10)


@pytest.mark.parametrize("seed", range(3))
def test_full_rank_cap_gives_rbar(seed):
    # "Max-P": once rank >= d - m every residual direction is kept, so Delta = r_bar (App. D.1).
    K, V, Q = rand_head(20 + seed, 120, 16, 5)
    r = oracle.head(K, V, Q, budget=6, rank=16)
    assert r["diag"]["span_rank"] == 6 and r["diag"]["rho_eff"] == 10
    np.testing.assert_allclose(r["Delta"], r["rbar"], atol=1e-11)
    np.testing.assert_allclose(r["delta"], r["diag"]["alpha"] * r["rbar"], atol=1e-11)


@pytest.mark.parametrize("rank", [1, 2, 5])
def test_codimension_one_residual(rank):
    # budget = d - 1 generic rows: the residual has rank one, C is the unit normal of the
    # retained span and Delta = r_bar for any rank >= 1.
    d = 12
    K, V, Q = rand_head(31, 90, d, 4)
    r = oracle.head(K, V, Q, budget=d - 1, rank=rank)
    Vk = V[r["idx"]].astype(np.float64)
    normal = np.linalg.svd(Vk)[2][-1]
    assert r["diag"]["rho_eff"] == 1
    np.testing.assert_allclose(r["proj"], np.outer(normal, normal), atol=1e-9)
    np.testing.assert_allclose(r["Delta"], r["rbar"], atol=1e-10)
    assert abs(abs(r["rbar"] @ normal) - np.linalg.norm(r["rbar"])) < 1e-10


def test_single_query_identity_from_the_error_bound_setup():
    # One query (App. L.1): A_j = alpha_j, A_keep + A_del = 1, and Eq. 4-6 give
    # delta * A_keep = Pi_C (I - Pi_keep) sum_{del} alpha_j v_j   (up to eps = 1e-12).
    K, V, Q = rand_head(41, 70, 16, 1, heavy=4)
    r = oracle.head(K, V, Q, budget=6, rank=2)
    a = scipy.special.softmax(Q[0].astype(np.float64) @ K.T.astype(np.float64) / 4.0)
    keep = np.zeros(70, bool); keep[r["idx"]] = True
    assert abs(r["diag"]["a_keep"] + r["diag"]["a_del"] - 1.0) < 1e-12
    Vd = V.astype(np.float64)
    Pk = np.linalg.pinv(Vd[keep]) @ Vd[keep]
    Rm = Vd[~keep] @ (np.eye(16) - Pk)
    C = np.linalg.svd(Rm)[2][:2]
    rhs = (C.T @ C) @ (np.eye(16) - Pk) @ (a[~keep] @ Vd[~keep])
    np.testing.assert_allclose(r["delta"] * r["diag"]["a_keep"], rhs, atol=1e-10)


@pytest.mark.parametrize("seed", range(4))
def test_injection_is_orthogonal_to_the_retained_span(seed):
    K, V, Q = rand_head(50 + seed, 150, 32, 8, heavy=5)
    r = oracle.head(K, V, Q, budget=10, rank=3)
    Vk = V[r["idx"]].astype(np.float64)
    dl = r["delta"]
    assert np.linalg.norm(dl) > 0
    assert np.abs(Vk @ dl).max() / (np.linalg.norm(Vk, 2) * np.linalg.norm(dl)) <= 1e-5
    assert np.linalg.norm(r["Delta"]) <= np.linalg.norm(r["rbar"]) * (1 + 1e-12)
    assert r["diag"]["rcr"] <= 1.0 + 1e-12


def test_budget_above_head_dim_with_full_rank_values_injects_nothing():
    # rank(V_keep) = d: the retained span is everything, the residual vanishes, OBF is a no-op.
    K, V, Q = rand_head(60, 200, 16, 6)
    r = oracle.head(K, V, Q, budget=40, rank=2)
    assert r["diag"]["span_rank"] == 16 and r["diag"]["skipped"] == 1
    assert np.all(r["delta"] == 0)
    assert np.array_equal(r["V_out"], V[r["idx"]].astype(np.float64))


def test_rank_deficient_values_with_budget_above_head_dim_still_inject():
    # All values live in a 10-dim coordinate subspace of R^16 except a few tokens whose keys make
    # them unselectable; budget >= d, yet the residual is not zero and OBF must act.
    g = np.random.default_rng(61)
    T, d = 160, 16
    K, V, Q = rand_head(61, T, d, 6)
    V[:, 10:] = 0.0
    qm = Q.mean(axis=0)
    odd = g.choice(T, 12, replace=False)
    K[odd] = (-6.0 * qm / np.linalg.norm(qm) * np.linalg.norm(K[odd], axis=1, keepdims=True)).astype(np.float32)
    V[odd, 10:] = g.standard_normal((12, 6)).astype(np.float32)
    r = oracle.head(K, V, Q, budget=30, rank=2)
    assert not set(odd) & set(r["idx"])
    assert r["diag"]["span_rank"] == 10 and r["diag"]["skipped"] == 0
    assert np.linalg.norm(r["delta"]) > 1e-6
    assert np.abs(r["delta"][:10]).max() < 1e-12
    ref = lib_obf(K, V, Q, 30, 2)
    np.testing.assert_allclose(r["delta"], ref["delta"], atol=1e-10)


# --------------------------------------------------------------------------
# the tiny benchmark configuration end to end, whole-cache entry point
# --------------------------------------------------------------------------
def test_c1_whole_cache_matches_lapack_pipeline_per_head():
    w = synth.workload("c1")
    arr = synth.gen_cache(w, 0)
    res = oracle.compress(arr["K"], arr["V"], arr["Q"], w.q_heads, w.n_obs,
                          w.caches[0].budget, w.rank)
    Qv = arr["Q"].reshape(w.layers, w.kv_heads, w.n_q, w.head.head_dim)
    for h in range(w.kv_heads):
        ref = lib_obf(arr["K"][0, h], arr["V"][0, h], Qv[0, h], w.caches[0].budget, w.rank)
        np.testing.assert_array_equal(res["idx"][0, h], ref["idx"])
        np.testing.assert_allclose(res["V_out"][0, h], ref["V_out"], atol=1e-9)
        np.testing.assert_allclose(res["delta"][0, h], ref["delta"], atol=1e-9)
        assert np.array_equal(res["K_out"][0, h], arr["K"][0, h][ref["idx"]].astype(np.float64))
        assert res["diag"][h]["span_rank"] == 32 and res["diag"][h]["skipped"] == 0
        # the planted heavy hitters must be among the retained positions
        k1, _, _ = synth.gen_head(w, 0, 0, h)
        assert np.array_equal(k1, arr["K"][0, h])


# --------------------------------------------------------------------------
# layerwise selector (retention rule, second form; Algorithm 2 with granularity L)
# --------------------------------------------------------------------------
def lib_obf_given_idx(V, A, idx, rank, eps=1e-12):
    """Algorithm 3 through LAPACK routines for a retained set chosen elsewhere."""
    T = V.shape[0]
    keep = np.zeros(T, bool); keep[idx] = True
    Vd = V.astype(np.float64)
    Vk, Vdel = Vd[keep], Vd[~keep]
    if rank <= 0 or Vdel.shape[0] == 0:
        return np.zeros(V.shape[1]), Vk
    R = Vdel - Vdel @ (np.linalg.pinv(Vk) @ Vk)
    if (R ** 2).sum() <= 1e-12 * (Vdel ** 2).sum():
        return np.zeros(V.shape[1]), Vk
    _, s, Vt = np.linalg.svd(R, full_matrices=False)
    rho = min(rank, int((s ** 2 > V.shape[1] * np.finfo(float).eps * s[0] ** 2).sum()))
    C = Vt[:rho]
    a_del, a_keep = A[~keep].sum(), A[keep].sum()
    rbar = (A[~keep] / (a_del + eps)) @ R
    delta = a_del / (a_keep + eps) * ((rbar @ C.T) @ C)
    return delta, Vk + delta


def rand_layer(seed, H, T, d, n_q):
    g = np.random.default_rng(seed)
    K = g.standard_normal((H, T, d)).astype(np.float32)
    V = g.standard_normal((H, T, d)).astype(np.float32)
    Q = g.standard_normal((H, n_q, d)).astype(np.float32)
    K[:, g.choice(T, 3, replace=False)] *= 3.0
    return K, V, Q


@pytest.mark.parametrize("seed,H,T,d,n_q,budget,rank", [(0, 2, 48, 16, 4, 6, 1), (1, 4, 96, 32, 8, 12, 2),
                                                         (2, 3, 40, 8, 4, 40, 2), (3, 8, 64, 16, 8, 5, 4)])
def test_layerwise_selects_on_summed_masses_and_backfills_per_head(seed, H, T, d, n_q, budget, rank):
    K, V, Q = rand_layer(seed, H, T, d, n_q)
    out = oracle.layer(K, V, Q, budget, rank)
    A = np.stack([lib_scores(K[h], Q[h]) for h in range(H)])
    S = A.sum(axis=0)
    np.testing.assert_allclose(out["S"], S, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(out["A"], A, rtol=1e-12, atol=1e-15)
    want = brute_topk(S, budget)                                # brute force over the summed masses
    assert np.array_equal(want, np.sort(np.argsort(-S, kind="stable")[:min(budget, T)]))
    for h in range(H):
        assert np.array_equal(out["idx"][h], want)              # one set, shared by the heads of the layer
        assert np.array_equal(out["K_out"][h], K[h][want].astype(np.float64))
        delta, v_out = lib_obf_given_idx(V[h], A[h], want, rank)
        scale = max(1.0, np.abs(delta).max())
        np.testing.assert_allclose(out["delta"][h], delta, atol=1e-9 * scale)
        np.testing.assert_allclose(out["V_out"][h], v_out, atol=1e-9 * scale)
        dg = out["diag"][h]
        keep = np.zeros(T, bool); keep[want] = True
        assert dg["a_keep"] == pytest.approx(A[h][keep].sum(), rel=1e-12)     # the head's own masses (Eq. 6)
        assert dg["a_del"] == pytest.approx(A[h][~keep].sum(), rel=1e-12, abs=1e-300)


def test_layerwise_with_one_kv_head_is_the_headwise_result():
    K, V, Q = rand_layer(7, 1, 80, 16, 6)
    lay = oracle.layer(K, V, Q, 9, 2)
    hd = oracle.head(K[0], V[0], Q[0], 9, 2)
    assert np.array_equal(lay["idx"][0], hd["idx"])
    assert np.array_equal(lay["V_out"][0], hd["V_out"])
    assert np.array_equal(lay["delta"][0], hd["delta"])


def test_layerwise_with_identical_heads_is_the_headwise_result():
    K1, V1, Q1 = rand_layer(8, 1, 72, 16, 6)
    K, V, Q = np.repeat(K1, 4, 0), np.repeat(V1, 4, 0), np.repeat(Q1, 4, 0)
    lay = oracle.layer(K, V, Q, 10, 1)
    hd = oracle.head(K1[0], V1[0], Q1[0], 10, 1)
    for h in range(4):
        assert np.array_equal(lay["idx"][h], hd["idx"])          # summing equal masses keeps their order
        np.testing.assert_allclose(lay["V_out"][h], hd["V_out"], atol=1e-12)


def test_layerwise_differs_from_headwise_when_heads_disagree():
    # two heads whose heavy keys sit at different positions: headwise keeps each head's own, layerwise the union's top
    g = np.random.default_rng(11)
    H, T, d = 2, 32, 8
    K = 0.01 * g.standard_normal((H, T, d)).astype(np.float32)
    V = g.standard_normal((H, T, d)).astype(np.float32)
    Q = np.ones((H, 2, d), np.float32)
    K[0, 3] = 4.0; K[1, 20] = 4.0; K[0, 9] = 2.0; K[1, 9] = 2.0
    lay = oracle.layer(K, V, Q, 2, 0)
    assert oracle.head(K[0], V[0], Q[0], 2, 0)["idx"].tolist() == [3, 9]
    assert oracle.head(K[1], V[1], Q[1], 2, 0)["idx"].tolist() == [9, 20]
    assert lay["idx"][0].tolist() == lay["idx"][1].tolist() == [3, 20]       # 3 and 20 each carry one head's top mass


def test_layerwise_whole_cache_matches_per_layer_calls():
    w = synth.workload("c1")
    a = synth.gen_cache(w, 0)
    d, n_q = w.head.head_dim, w.n_q
    out = oracle.compress(a["K"], a["V"], a["Q"], w.q_heads, w.n_obs, w.caches[0].budget, w.rank, layerwise=True)
    Qv = a["Q"].reshape(w.layers, w.kv_heads, n_q, d)
    for l in range(w.layers):
        lay = oracle.layer(a["K"][l], a["V"][l], Qv[l], w.caches[0].budget, w.rank)
        assert np.array_equal(out["idx"][l], lay["idx"])
        assert np.array_equal(out["V_out"][l], lay["V_out"])


# --------------------------------------------------------------------------
# protected sink prefix (the first s positions are retained besides the budget and are no candidates)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("seed,T,budget,n_sink", [(0, 50, 7, 4), (1, 50, 7, 0), (2, 12, 20, 4), (3, 9, 3, 9), (4, 6, 2, 10)])
def test_sink_prefix_is_retained_besides_the_budget(seed, T, budget, n_sink):
    g = np.random.default_rng(seed)
    A = g.random(T)
    A[:2] = 0.0                                            # protected even when nothing attends to them
    idx, kth, nxt = oracle.topk(A, budget, n_sink)
    s = min(n_sink, T)
    rest = np.arange(s, T)
    want_rest = rest[np.argsort(-A[rest], kind="stable")[:min(budget, T - s)]]      # library sort of the candidates
    want = np.sort(np.concatenate([np.arange(s), want_rest])).astype(np.int32)
    assert np.array_equal(idx, want)
    assert len(idx) == oracle.k_eff(T, budget, n_sink) == s + min(budget, T - s)
    if len(want_rest):
        assert kth == A[want_rest].min()
    deleted = np.setdiff1d(rest, want_rest)
    assert nxt == (A[deleted].max() if len(deleted) else -1.0)


def test_sink_prefix_head_backfill_uses_the_union_as_retained_set():
    K, V, Q = rand_head(12, 90, 16, 6, heavy=3)
    out = oracle.head(K, V, Q, budget=6, rank=2, n_sink=4)
    A = lib_scores(K, Q)
    assert out["idx"][:4].tolist() == [0, 1, 2, 3] and len(out["idx"]) == 10
    delta, v_out = lib_obf_given_idx(V, A, out["idx"], 2)
    np.testing.assert_allclose(out["delta"], delta, atol=1e-9)
    np.testing.assert_allclose(out["V_out"], v_out, atol=1e-9)
    keep = np.zeros(90, bool); keep[out["idx"]] = True
    assert out["diag"]["a_keep"] == pytest.approx(A[keep].sum(), rel=1e-12)       # sink masses count as retained demand
    plain = oracle.head(K, V, Q, budget=6, rank=2)
    assert np.array_equal(oracle.head(K, V, Q, budget=6, rank=2, n_sink=0)["idx"], plain["idx"])


def test_sink_prefix_with_the_layerwise_selector():
    K, V, Q = rand_layer(13, 3, 70, 16, 5)
    lay = oracle.layer(K, V, Q, 8, 1, n_sink=4)
    S = sum(lib_scores(K[h], Q[h]) for h in range(3))
    rest = np.arange(4, 70)
    want = np.sort(np.concatenate([np.arange(4), rest[np.argsort(-S[rest], kind="stable")[:8]]]))
    for h in range(3):
        assert np.array_equal(lay["idx"][h], want)


# --------------------------------------------------------------------------
# fixed-iteration Gram subspace path (App. H)
# --------------------------------------------------------------------------
def lib_fast_path(K, V, Q, budget, rank, iters, eps=1e-12):
    """The same iteration through numpy's thin QR (a library orth), from the first rows of the identity."""
    A = lib_scores(K, Q)
    T, d = V.shape
    idx = np.sort(np.argsort(-A, kind="stable")[:min(budget, T)])
    keep = np.zeros(T, bool); keep[idx] = True
    Vd = V.astype(np.float64)
    Vk, Vdel = Vd[keep], Vd[~keep]
    Pi = np.linalg.pinv(Vk) @ Vk
    R = Vdel - Vdel @ Pi
    G = R.T @ R
    m = np.linalg.matrix_rank(Vk)
    rho = min(rank, d - m)
    C = np.eye(d)[:rho]
    for _ in range(iters):
        Qm, _ = np.linalg.qr((C @ G).T)                    # thin QR: columns of Qm span the rows of C G
        C = Qm.T
    a_del, a_keep = A[~keep].sum(), A[keep].sum()
    rbar = (A[~keep] / (a_del + eps)) @ R
    Delta = (rbar @ C.T) @ C
    return {"proj": C.T @ C, "Delta": Delta, "delta": a_del / (a_keep + eps) * Delta, "G": G, "rho": rho}


@pytest.mark.parametrize("seed,T,d,n_q,budget,rank,iters", [(0, 120, 16, 6, 5, 2, 3), (1, 200, 32, 8, 12, 4, 3),
                                                            (2, 90, 16, 4, 6, 1, 1), (3, 150, 24, 6, 20, 8, 3)])
def test_fast_path_matches_the_same_iteration_through_library_qr(seed, T, d, n_q, budget, rank, iters):
    K, V, Q = rand_head(seed, T, d, n_q, heavy=3)
    r = oracle.head(K, V, Q, budget, rank, fast_iters=iters)
    ref = lib_fast_path(K, V, Q, budget, rank, iters)
    assert r["diag"]["rho_eff"] == ref["rho"]
    np.testing.assert_allclose(r["Delta"], ref["Delta"], atol=1e-9 * max(1.0, np.abs(ref["Delta"]).max()))
    np.testing.assert_allclose(r["delta"], ref["delta"], atol=1e-9 * max(1.0, np.abs(ref["delta"]).max()))
    Vk = V[r["idx"]].astype(np.float64)
    assert np.abs(Vk @ r["delta"]).max() <= 1e-9 * np.linalg.norm(Vk, 2) * max(np.linalg.norm(r["delta"]), 1e-300)


def test_fast_path_reaches_the_exact_subspace_when_the_spectrum_has_a_gap():
    # a residual with two dominant directions (planted, 30 times the rest of the values)
    g = np.random.default_rng(5)
    T, d = 160, 16
    K = g.standard_normal((T, d)).astype(np.float32); Q = g.standard_normal((5, d)).astype(np.float32)
    V = g.standard_normal((T, d)).astype(np.float32)
    V[:, 8] *= 30.0; V[:, 9] *= 30.0
    V[oracle.topk(oracle.scores(K, Q), 4)[0], 8:10] = 0.0   # the retained values stay out of the planted plane
    exact = oracle.head(K, V, Q, 4, 2)
    fast = oracle.head(K, V, Q, 4, 2, fast_iters=3)
    # one iteration contracts the error by about lambda_3 / lambda_2 ~ 1/580: three leave ~1e-6, five ~1e-11
    np.testing.assert_allclose(fast["delta"], exact["delta"], atol=1e-5 * np.abs(exact["delta"]).max())
    np.testing.assert_allclose(oracle.head(K, V, Q, 4, 2, fast_iters=5)["delta"], exact["delta"],
                               atol=1e-9 * np.abs(exact["delta"]).max())
    assert np.linalg.norm(oracle.head(K, V, Q, 4, 2, fast_iters=1)["delta"] - exact["delta"]) > \
        np.linalg.norm(fast["delta"] - exact["delta"])


# --------------------------------------------------------------------------
# post-hoc int8 quantisation of the compacted relay (App. E)
# --------------------------------------------------------------------------
def test_int8_rows_round_trip_within_half_a_step_and_use_the_full_range():
    g = np.random.default_rng(3)
    X = (g.standard_normal((37, 128)) * g.uniform(0.01, 30, (37, 1))).astype(np.float32)
    codes, scales = oracle.quantize_rows(X)
    assert codes.dtype == np.int8 and scales.dtype == np.float32
    back = codes.astype(np.float64) * scales.astype(np.float64)[:, None]
    # x / scale is rounded to fp32 before the rounding to a code: 127 * 2^-24 of a step on top of half a step
    assert np.all(np.abs(back - X) <= 0.5 * scales[:, None] * (1 + 2.0 ** -15))
    assert np.all(np.abs(codes).max(axis=1) == 127)                      # the largest element of a row sits at the end of the range
    assert np.all(np.sign(codes[np.arange(37), np.abs(X).argmax(axis=1)]) == np.sign(X[np.arange(37), np.abs(X).argmax(axis=1)]))
    np.testing.assert_allclose(scales, np.abs(X).max(axis=1) / 127.0, rtol=1e-6)


def test_int8_rows_match_a_library_statement_and_handle_zero_rows():
    g = np.random.default_rng(4)
    X = g.standard_normal((5, 3, 64)).astype(np.float32)
    X[2, 1] = 0.0
    X[0, 0, :4] = [0.5, 1.5, 2.5, -2.5]                                   # halves: the rounding rule shows
    X[0, 0, 4:] = 0.0
    X[0, 0, 5] = 127.0                                                    # scale exactly 1
    codes, scales = oracle.quantize_rows(X)
    sc = (np.abs(X).max(axis=-1) / np.float32(127.0)).astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        ref = np.where(sc[..., None] > 0, np.rint((X / sc[..., None]).astype(np.float32)), 0.0)
    assert np.array_equal(codes, np.clip(ref, -127, 127).astype(np.int8))
    assert np.array_equal(scales, sc)
    assert scales[2, 1] == 0 and not codes[2, 1].any()
    assert codes[0, 0, :4].tolist() == [0, 2, 2, -2]                      # ties go to the even code


def test_backfill_for_given_positions_is_the_head_result_on_its_own_positions():
    K, V, Q = rand_head(21, 90, 32, 6, heavy=3)
    h = oracle.head(K, V, Q, 12, 2)
    b = oracle.backfill(K, V, h["A"], h["idx"], 2)
    np.testing.assert_array_equal(b["V_out"], h["V_out"])
    np.testing.assert_array_equal(b["delta"], h["delta"])
    # another retained set: the last position swapped for a deleted one; the gather follows it
    idx2 = np.sort(np.append(h["idx"][:-1], np.setdiff1d(np.arange(90), h["idx"])[0])).astype(np.int32)
    b2 = oracle.backfill(K, V, h["A"], idx2, 2)
    np.testing.assert_array_equal(b2["K_out"], K[idx2].astype(np.float64))
    Vk = V[idx2].astype(np.float64)
    assert np.abs(Vk @ b2["delta"]).max() <= 1e-10 * np.linalg.norm(Vk, 2) * max(np.linalg.norm(b2["delta"]), 1e-300)


# --------------------------------------------------------------------------
# Attn-inject (App. D.2): the back-fill shared out by attention mass
# --------------------------------------------------------------------------
def test_attn_inject_shares_add_up_and_equal_masses_give_the_uniform_injection():
    g = np.random.default_rng(6)
    V = g.standard_normal((40, 16)).astype(np.float32)
    delta = g.standard_normal(16)
    idx = np.array([1, 5, 6, 20, 33], np.int32)
    A = g.uniform(0.1, 2.0, 40)
    out = oracle.attn_inject(V, A, idx, delta)
    ref = V[idx].astype(np.float64) + (5 * A[idx] / (A[idx].sum() + 1e-12))[:, None] * delta[None, :]
    np.testing.assert_allclose(out, ref, rtol=1e-14, atol=1e-15)
    # the shares average one: the mean injected vector is delta
    np.testing.assert_allclose((out - V[idx]).mean(axis=0), delta, rtol=1e-10)
    A[idx] = 0.7
    np.testing.assert_allclose(oracle.attn_inject(V, A, idx, delta), V[idx] + delta[None, :], rtol=1e-11, atol=1e-12)


# --------------------------------------------------------------------------
# cache-merging baseline (App. E)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(3))
def test_merge_matches_a_library_statement(seed):
    K, V, Q = rand_head(30 + seed, 120, 32, 6, heavy=3)
    m = oracle.merge_head(K, V, Q, 9)
    A = oracle.scores(K, Q)
    idx = oracle.topk(A, 9)[0]
    assert np.array_equal(m["idx"], idx)
    Kd = K.astype(np.float64)
    Kn = Kd / np.linalg.norm(Kd, axis=1, keepdims=True)
    cos = Kn @ Kn[idx].T                                              # [T, k]
    route = cos.argmax(axis=1)
    dele = np.setdiff1d(np.arange(120), idx)
    assert np.array_equal(m["assign"][dele], route[dele]) and np.all(m["assign"][idx] == -1)
    srt = np.sort(cos[dele], axis=1)
    np.testing.assert_allclose(m["margin"][dele], srt[:, -1] - srt[:, -2], atol=1e-14)
    ref = V[idx].astype(np.float64).copy()
    for j in dele:
        ref[route[j]] += A[j] / (A[idx[route[j]]] + 1e-12) * V[j].astype(np.float64)
    np.testing.assert_allclose(m["V_out"], ref, rtol=1e-12, atol=1e-13)
    assert np.array_equal(m["K_out"], K[idx].astype(np.float64))
    np.testing.assert_allclose(oracle.merge_given(V, A, idx, m["assign"]), m["V_out"], rtol=1e-13, atol=1e-14)


def test_merge_conserves_the_mass_weighted_values_and_routes_a_duplicate_to_its_twin():
    K, V, Q = rand_head(41, 80, 16, 5, heavy=2)
    m0 = oracle.merge_head(K, V, Q, 7)
    j = int(np.setdiff1d(np.arange(80), m0["idx"])[3])
    t = int(m0["idx"][2])
    K[j] = 3.0 * K[t]                                                # same direction as a retained key
    m = oracle.merge_head(K, V, Q, 7)
    if j not in m["idx"] and t in m["idx"]:
        assert m["idx"][m["assign"][j]] == t
    # sum over retained t of A_t V*_t = sum over all positions of A_j V_j (eps aside): nothing is dropped
    A, idx = m["A"], m["idx"]
    lhs = (A[idx][:, None] * m["V_out"]).sum(axis=0)
    rhs = (A[:, None] * V.astype(np.float64)).sum(axis=0)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-9, atol=1e-9)
    # budget >= T: nothing to merge
    full = oracle.merge_head(K, V, Q, 80)
    assert np.array_equal(full["V_out"], V.astype(np.float64)) and np.all(full["assign"] == -1)
