"""ctypes front end of the CPU oracle (``obf_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle is the slow fp64 restatement of the
paper's Eq. 1-7 / Algorithms 2-3 that the CUDA path is checked against.  Only
the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the product package never does.

``build()`` compiles the C file with gcc (OpenMP over heads) into
``oracle/_build/libobf_oracle.so``; the library is rebuilt when the source is
newer than the binary.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "obf_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_OUT_DIR, "libobf_oracle.so")
_lib = None


class Diag(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in (
        "a_keep", "a_del", "alpha", "vdel_fro2", "r_fro2", "rcr", "rbar_norm",
        "delta_norm", "kth_score", "next_score", "lam_rho", "lam_next", "lam_1")] + [
        (n, ctypes.c_int32) for n in ("span_rank", "rho_eff", "n_del", "skipped")] + [("revr", ctypes.c_double), ("pc", ctypes.c_double)]

    def asdict(self) -> Dict[str, float]:
        return {n: getattr(self, n) for n, _ in self._fields_}


def build(force: bool = False) -> str:
    os.makedirs(_OUT_DIR, exist_ok=True)
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    tmp = _LIB_PATH + ".tmp%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        fp = ctypes.POINTER(ctypes.c_float)
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        ci = ctypes.c_int
        _lib.obf_oracle_scores.argtypes = [fp, fp, ci, ci, ci, dp]
        _lib.obf_oracle_scores.restype = None
        _lib.obf_oracle_scores_ext.argtypes = [fp, fp, fp, ci, ci, ci, dp]
        _lib.obf_oracle_scores_ext.restype = None
        _lib.obf_oracle_topk.argtypes = [dp, ci, ci, ip, dp, dp]
        _lib.obf_oracle_topk.restype = ci
        _lib.obf_oracle_topk_sink.argtypes = [dp, ci, ci, ci, ip, dp, dp]
        _lib.obf_oracle_topk_sink.restype = ci
        _lib.obf_oracle_span_basis.argtypes = [dp, ci, ci, dp]
        _lib.obf_oracle_span_basis.restype = ci
        _lib.obf_oracle_sym_eig.argtypes = [dp, ci, dp, dp]
        _lib.obf_oracle_sym_eig.restype = None
        _lib.obf_oracle_head.argtypes = [fp, fp, fp, ci, ci, ci, ci, ci, ctypes.c_double,
                                         ip, dp, dp, dp, dp, dp, dp, dp, dp, ctypes.POINTER(Diag)]
        _lib.obf_oracle_head.restype = ci
        _lib.obf_oracle_head_sink.argtypes = _lib.obf_oracle_head.argtypes + [ci]
        _lib.obf_oracle_head_sink.restype = ci
        _lib.obf_oracle_head_ex.argtypes = _lib.obf_oracle_head.argtypes + [ci, ci]
        _lib.obf_oracle_head_ex.restype = ci
        _lib.obf_oracle_head_lse.argtypes = [fp, fp, fp, fp] + _lib.obf_oracle_head.argtypes[3:] + [ci, ci]
        _lib.obf_oracle_head_lse.restype = ci
        _lib.obf_oracle_compress.argtypes = [fp, fp, fp, ci, ci, ci, ci, ci, ci, ci, ci,
                                             ctypes.c_double, ip, dp, dp, dp, ctypes.POINTER(Diag), ci]
        _lib.obf_oracle_compress.restype = ci
        _lib.obf_oracle_layer.argtypes = [fp, fp, fp, ci, ci, ci, ci, ci, ci, ctypes.c_double,
                                          ip, dp, dp, dp, dp, dp, ctypes.POINTER(Diag), ci]
        _lib.obf_oracle_layer.restype = ci
        _lib.obf_oracle_compress_layerwise.argtypes = _lib.obf_oracle_compress.argtypes
        _lib.obf_oracle_compress_layerwise.restype = ci
        _lib.obf_oracle_backfill.argtypes = [fp, fp, dp, ci, ci, ci, ci, ctypes.c_double, ip, dp, dp, dp, ctypes.POINTER(Diag)]
        _lib.obf_oracle_backfill.restype = ci
        _lib.obf_oracle_merge_head.argtypes = [fp, fp, fp, ci, ci, ci, ci, ctypes.c_double, ci, ip, dp, dp, dp, ip, dp]
        _lib.obf_oracle_merge_head.restype = ci
        _lib.obf_oracle_merge_given.argtypes = [fp, dp, ip, ci, ip, ci, ci, ctypes.c_double, dp]
        _lib.obf_oracle_merge_given.restype = None
        _lib.obf_oracle_attn_inject.argtypes = [fp, dp, ip, ci, ci, dp, ctypes.c_double, dp]
        _lib.obf_oracle_attn_inject.restype = None
        _lib.obf_oracle_quantize_rows.argtypes = [fp, ci, ci, ctypes.POINTER(ctypes.c_int8), fp]
        _lib.obf_oracle_quantize_rows.restype = None
        _lib.obf_oracle_num_threads.argtypes = []
        _lib.obf_oracle_num_threads.restype = ci
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def num_threads() -> int:
    return int(lib().obf_oracle_num_threads())


def scores(K, Q, lse_extra=None) -> np.ndarray:
    """Attention mass A[T] of one KV head (Eq. 1); K [T,d], Q [n_q,d].

    lse_extra [n_q] (optional): log-sum-exp of each query row's logits over the keys outside the prompt; they
    take their share of the softmax normaliser."""
    K, Q = _f32(K), _f32(Q)
    T, d = K.shape
    A = np.empty(T, dtype=np.float64)
    if lse_extra is None:
        lib().obf_oracle_scores(_p(K, ctypes.c_float), _p(Q, ctypes.c_float), T, d, Q.shape[0],
                                _p(A, ctypes.c_double))
    else:
        le = _f32(lse_extra)
        assert le.shape == (Q.shape[0],)
        lib().obf_oracle_scores_ext(_p(K, ctypes.c_float), _p(Q, ctypes.c_float), _p(le, ctypes.c_float), T, d,
                                    Q.shape[0], _p(A, ctypes.c_double))
    return A


def k_eff(T: int, budget: int, n_sink: int = 0) -> int:
    """Retained positions: the protected prefix plus at most `budget` of the others."""
    s = max(0, min(n_sink, T))
    return s + min(budget, T - s)


def topk(A, budget: int, n_sink: int = 0):
    """Ascending retained positions, plus the smallest retained and largest deleted mass among the candidates.

    n_sink: the first n_sink positions are protected: retained besides the budget, no candidates."""
    A = _f64(A)
    T = A.shape[0]
    idx = np.empty(max(T, 1), dtype=np.int32)
    kth, nxt = ctypes.c_double(), ctypes.c_double()
    k2 = lib().obf_oracle_topk_sink(_p(A, ctypes.c_double), T, budget, n_sink, _p(idx, ctypes.c_int32),
                                    ctypes.byref(kth), ctypes.byref(nxt))
    assert k2 == k_eff(T, budget, n_sink)
    return idx[:k2].copy(), kth.value, nxt.value


def span_basis(X) -> np.ndarray:
    """Orthonormal rows spanning the row space of X [k,d] (Eq. 2)."""
    X = _f64(X)
    k, d = X.shape
    Qb = np.zeros((max(min(k, d), 1), d), dtype=np.float64)
    m = lib().obf_oracle_span_basis(_p(X, ctypes.c_double), k, d, _p(Qb, ctypes.c_double))
    return Qb[:m].copy()


def sym_eig(S):
    """Eigenvalues (descending) and eigenvectors (rows) of a symmetric matrix."""
    S = _f64(S).copy()
    n = S.shape[0]
    lam = np.empty(n, dtype=np.float64)
    E = np.empty((n, n), dtype=np.float64)
    lib().obf_oracle_sym_eig(_p(S, ctypes.c_double), n, _p(lam, ctypes.c_double), _p(E, ctypes.c_double))
    return lam, E


def head(K, V, Q, budget: int, rank: int, eps: float = 1e-12, n_sink: int = 0,
         fast_iters: int = 0, lse_extra=None) -> Dict[str, object]:
    """Algorithm 2 (headwise) + Algorithm 3 on one (layer, KV head).

    K, V [T,d]; Q [n_q,d] (float32 values; bf16 inputs up-cast exactly).
    fast_iters > 0: the subspace comes from that many Gram subspace iterations (App. H) started at the first
    rows of the identity, instead of the exact eigenvectors.
    lse_extra [n_q] (optional): out-of-prompt softmax mass per query row, see scores().
    Returns idx, K_out, V_out (float64), A, delta, rbar, Delta, eigvals, proj, diag.
    """
    K, V, Q = _f32(K), _f32(V), _f32(Q)
    T, d = K.shape
    k = k_eff(T, budget, n_sink)
    idx = np.empty(max(k, 1), dtype=np.int32)
    K_out = np.zeros((max(k, 1), d), dtype=np.float64)
    V_out = np.zeros((max(k, 1), d), dtype=np.float64)
    A = np.empty(T, dtype=np.float64)
    delta = np.empty(d); rbar = np.empty(d); Delta = np.empty(d); eig = np.empty(d)
    proj = np.empty((d, d))
    dg = Diag()
    cd = ctypes.c_double
    le = None if lse_extra is None else _f32(lse_extra)
    assert le is None or le.shape == (Q.shape[0],)
    k2 = lib().obf_oracle_head_lse(
        _p(K, ctypes.c_float), _p(V, ctypes.c_float), _p(Q, ctypes.c_float), _p(le, ctypes.c_float),
        T, d, Q.shape[0], budget, rank, eps,
        _p(idx, ctypes.c_int32), _p(K_out, cd), _p(V_out, cd), _p(A, cd), _p(delta, cd),
        _p(rbar, cd), _p(Delta, cd), _p(eig, cd), _p(proj, cd), ctypes.byref(dg), n_sink, fast_iters)
    assert k2 == k
    return {"idx": idx[:k].copy(), "K_out": K_out[:k], "V_out": V_out[:k], "A": A, "delta": delta,
            "rbar": rbar, "Delta": Delta, "eigvals": eig, "proj": proj, "diag": dg.asdict()}


def layer(K, V, Q, budget: int, rank: int, eps: float = 1e-12, n_sink: int = 0) -> Dict[str, object]:
    """Layerwise selector (Algorithm 2, granularity L) + Algorithm 3 on one layer.

    K, V [kv_heads,T,d]; Q [kv_heads,n_q,d].  The retained positions are TopK_B of the masses summed over
    the KV heads and are shared by the heads; the back-fill runs per head with the head's own masses.
    Returns idx [kv_heads,k], K_out, V_out (float64), S (summed masses), A [kv_heads,T], delta, diag (per head).
    """
    K, V, Q = _f32(K), _f32(V), _f32(Q)
    H, T, d = K.shape
    k = k_eff(T, budget, n_sink)
    idx = np.empty((H, max(k, 1)), dtype=np.int32)
    K_out = np.zeros((H, max(k, 1), d), dtype=np.float64)
    V_out = np.zeros((H, max(k, 1), d), dtype=np.float64)
    S = np.empty(T, dtype=np.float64)
    A = np.empty((H, T), dtype=np.float64)
    delta = np.zeros((H, d), dtype=np.float64)
    diags = (Diag * H)()
    cd = ctypes.c_double
    k2 = lib().obf_oracle_layer(
        _p(K, ctypes.c_float), _p(V, ctypes.c_float), _p(Q, ctypes.c_float),
        H, T, d, Q.shape[1], budget, rank, eps,
        _p(idx, ctypes.c_int32), _p(K_out, cd), _p(V_out, cd), _p(S, cd), _p(A, cd), _p(delta, cd), diags, n_sink)
    assert k2 == k
    return {"idx": idx[:, :k].copy(), "K_out": K_out[:, :k], "V_out": V_out[:, :k], "S": S, "A": A,
            "delta": delta, "diag": [diags[h].asdict() for h in range(H)]}


def backfill(K, V, A, idx, rank: int, eps: float = 1e-12) -> Dict[str, object]:
    """Algorithm 3 on one (layer, KV head) for given masses A [T] and given ascending retained positions idx."""
    K, V, A = _f32(K), _f32(V), _f64(A)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    T, d = K.shape
    k = idx.shape[0]
    K_out = np.zeros((max(k, 1), d)); V_out = np.zeros((max(k, 1), d)); delta = np.zeros(d)
    dg = Diag()
    cd = ctypes.c_double
    lib().obf_oracle_backfill(_p(K, ctypes.c_float), _p(V, ctypes.c_float), _p(A, cd), T, d, k, rank, eps,
                              _p(idx, ctypes.c_int32), _p(K_out, cd), _p(V_out, cd), _p(delta, cd), ctypes.byref(dg))
    return {"idx": idx, "K_out": K_out[:k], "V_out": V_out[:k], "A": A, "delta": delta, "diag": dg.asdict()}


def merge_head(K, V, Q, budget: int, eps: float = 1e-12, n_sink: int = 0) -> Dict[str, object]:
    """Cache-merging baseline (App. E) on one (layer, KV head): select, route every deleted position to the
    retained position with the most similar key (cosine), add its value in, weighted by A_j / (A_t + eps).
    Returns idx, K_out, V_out, A, assign [T] (-1 for retained positions), margin [T]."""
    K, V, Q = _f32(K), _f32(V), _f32(Q)
    T, d = K.shape
    k = k_eff(T, budget, n_sink)
    idx = np.empty(max(k, 1), dtype=np.int32)
    K_out = np.zeros((max(k, 1), d)); V_out = np.zeros((max(k, 1), d))
    A = np.empty(T); assign = np.empty(T, dtype=np.int32); margin = np.empty(T)
    cd = ctypes.c_double
    k2 = lib().obf_oracle_merge_head(_p(K, ctypes.c_float), _p(V, ctypes.c_float), _p(Q, ctypes.c_float), T, d, Q.shape[0],
                                     budget, eps, n_sink, _p(idx, ctypes.c_int32), _p(K_out, cd), _p(V_out, cd), _p(A, cd),
                                     _p(assign, ctypes.c_int32), _p(margin, cd))
    assert k2 == k
    return {"idx": idx[:k].copy(), "K_out": K_out[:k], "V_out": V_out[:k], "A": A, "assign": assign, "margin": margin}


def merge_given(V, A, idx, assign, eps: float = 1e-12) -> np.ndarray:
    """Step (iii) of the cache-merging baseline for a given routing."""
    V, A = _f32(V), _f64(A)
    idx = np.ascontiguousarray(idx, dtype=np.int32); assign = np.ascontiguousarray(assign, dtype=np.int32)
    T, d = V.shape
    out = np.zeros((max(len(idx), 1), d))
    lib().obf_oracle_merge_given(_p(V, ctypes.c_float), _p(A, ctypes.c_double), _p(idx, ctypes.c_int32), len(idx),
                                 _p(assign, ctypes.c_int32), T, d, eps, _p(out, ctypes.c_double))
    return out[:len(idx)]


def attn_inject(V, A, idx, delta, eps: float = 1e-12) -> np.ndarray:
    """Attn-inject (App. D.2): V_out [k, d] = V[idx] + k * A[idx] / (sum A[idx] + eps) * delta."""
    V, A, delta = _f32(V), _f64(A), _f64(delta)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    k, d = idx.shape[0], V.shape[1]
    out = np.zeros((max(k, 1), d))
    lib().obf_oracle_attn_inject(_p(V, ctypes.c_float), _p(A, ctypes.c_double), _p(idx, ctypes.c_int32), k, d,
                                 _p(delta, ctypes.c_double), eps, _p(out, ctypes.c_double))
    return out[:k]


def quantize_rows(X):
    """Post-hoc int8 quantisation of compacted rows (App. E): X [..., d] float32 -> (codes int8 [..., d], scales
    float32 [...]), one symmetric absmax scale per row."""
    X = _f32(X)
    d = X.shape[-1]
    rows = X.size // d
    codes = np.empty(X.shape, dtype=np.int8)
    scales = np.empty(X.shape[:-1], dtype=np.float32)
    lib().obf_oracle_quantize_rows(_p(X, ctypes.c_float), rows, d, _p(codes, ctypes.c_int8), _p(scales, ctypes.c_float))
    return codes, scales


def compress(K, V, Q, q_heads: int, n_obs: int, budget: int, rank: int,
             eps: float = 1e-12, layerwise: bool = False, n_sink: int = 0) -> Dict[str, object]:
    """A whole cache: K, V [layers, kv_heads, T, d]; Q [layers, q_heads, n_obs, d].

    layerwise: one retained set per layer (masses summed over its KV heads) instead of one per head."""
    K, V, Q = _f32(K), _f32(V), _f32(Q)
    layers, kv_heads, T, d = K.shape
    k = k_eff(T, budget, n_sink)
    heads = layers * kv_heads
    idx = np.empty((layers, kv_heads, k), dtype=np.int32)
    K_out = np.zeros((layers, kv_heads, k, d), dtype=np.float64)
    V_out = np.zeros((layers, kv_heads, k, d), dtype=np.float64)
    delta = np.zeros((layers, kv_heads, d), dtype=np.float64)
    diags = (Diag * heads)()
    cd = ctypes.c_double
    fn = lib().obf_oracle_compress_layerwise if layerwise else lib().obf_oracle_compress
    fn(
        _p(K, ctypes.c_float), _p(V, ctypes.c_float), _p(Q, ctypes.c_float),
        layers, kv_heads, q_heads, n_obs, T, d, budget, rank, eps,
        _p(idx, ctypes.c_int32), _p(K_out, cd), _p(V_out, cd), _p(delta, cd), diags, n_sink)
    return {"idx": idx, "K_out": K_out, "V_out": V_out, "delta": delta,
            "diag": [diags[i].asdict() for i in range(heads)]}
