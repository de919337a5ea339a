"""Seeded synthetic prompt-KV caches for the relay-compression path.

This module only *draws inputs*. It holds none of the method's arithmetic (no
scores, no selection, no OBF), so both the CPU oracle's tests and the CUDA
path's tests and benchmark may import it.

The paper measures on Qwen3 caches produced by LatentMAS prompts over public
benchmarks; neither the weights nor the prompts are available offline, so the
seeded arrays below take the shapes of those model scales and stand in for
them.

Layout (row-major, C order):

    K, V    [layers, kv_heads, T, head_dim]
    Q_obs   [layers, q_heads, n_obs, head_dim]      q head = kv_head * G + g

so the ``n_q = G * n_obs`` observation-query rows pooled into one KV head are
one contiguous ``[n_q, head_dim]`` block.

Every (cache, layer, kv head) has its own counter-based stream,
``PCG64(SeedSequence([seed, cache, layer, head]))``, so any single head of a
large configuration can be regenerated alone (the parity tests at full size
sample heads this way).  Draw order inside a head, fixed forever:

    1. K  ~ N(0,1)  [T, d] float32
    2. V  ~ N(0,1)  [T, d] float32
    3. Q  ~ N(0,1)  [n_q, d] float32
    4. outlier channels (if any): ``n_out`` channel ids for K, then for V,
       without replacement; those channels are multiplied by ``outlier_scale``
    5. sink prefix (if any): positions 0..n_sink-1 get
       ``K_j <- sink_scale * ||K_j|| * q_hat``
    6. heavy hitters (if any): ``n_heavy`` positions drawn without replacement
       from the non-sink positions get ``K_j <- heavy_scale * ||K_j|| * q_hat``

``q_hat`` is the unit vector along the mean of the head's n_q query rows
(computed in float64, stored back as float32).  For bf16 configurations the
float32 arrays are rounded to nearest-even bf16 at the very end; the oracle
up-casts those bf16 values exactly, so both sides see the same numbers.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, List, Optional, Tuple

import numpy as np

__all__ = [
    "HeadSpec", "CacheSpec", "Workload", "WORKLOADS", "workload",
    "gen_head", "gen_cache", "to_bf16_bits", "bf16_bits_to_f32", "k_eff",
]


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact up-cast of bfloat16 bit patterns (uint16) to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def k_eff(budget: int, T: int) -> int:
    """Number of retained positions: the budget, capped by the prompt length."""
    return min(int(budget), int(T))


@dataclasses.dataclass(frozen=True)
class HeadSpec:
    """Value recipe shared by all heads of a workload."""
    head_dim: int
    n_q: int                      # G * n_obs query rows pooled into one KV head
    n_outlier: int = 0            # channels scaled by outlier_scale (independently for K and V)
    outlier_scale: float = 8.0
    heavy_frac: float = 0.0       # fraction of T made heavy hitters (count = round(frac*T)) ...
    heavy_count: int = 0          # ... or an absolute count (used when heavy_frac == 0)
    heavy_scale: float = 4.0
    n_sink: int = 0
    sink_scale: float = 8.0


@dataclasses.dataclass(frozen=True)
class CacheSpec:
    T: int
    budget: int


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    layers: int
    kv_heads: int
    q_heads: int
    n_obs: int
    rank: int
    dtype: str                    # "f32" or "bf16"
    head: HeadSpec
    caches: Tuple[CacheSpec, ...]
    layerwise: bool = False       # layerwise selector: one retained set per layer
    fast_path: bool = False       # three Gram subspace iterations instead of the exact eigenvectors
    int8_out: bool = False        # the relay leaves as int8 codes with one fp32 scale per row (App. E)
    merge: bool = False           # cache-merging baseline instead of Orthogonal BackFill (App. E)
    early_out: bool = False       # span test first; the pass over V skips heads whose retained values span R^d

    @property
    def G(self) -> int:
        return self.q_heads // self.kv_heads

    @property
    def n_q(self) -> int:
        return self.G * self.n_obs

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def algorithmic_bytes(self) -> int:
        """K, V and queries read once; compacted K, V and the index list written once (with int8_out the relay
        that leaves is the int8 codes and their scales: d + 4 bytes per row instead of d * elem_bytes)."""
        d, e = self.head.head_dim, self.elem_bytes
        row = (d + 4) if self.int8_out else d * e
        total = 0
        for c in self.caches:
            ke = k_eff(c.budget, c.T)
            heads = self.layers * self.kv_heads
            total += heads * (2 * c.T * d * e + self.n_q * d * e + 2 * ke * row + 4 * ke)
        return total

    def tokens(self) -> int:
        return sum(c.T for c in self.caches)


def _rng(seed: int, cache: int, layer: int, head: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, cache, layer, head])))


def gen_head(w: Workload, cache: int, layer: int, head: int,
             T: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """One (cache, layer, kv head): returns float32 ``K[T,d], V[T,d], Q[n_q,d]``.

    For bf16 workloads the returned float32 values are exactly representable in
    bf16 (already rounded).
    """
    hs = w.head
    T = w.caches[cache].T if T is None else T
    d, n_q = hs.head_dim, w.n_q
    g = _rng(w.seed, cache, layer, head)
    K = g.standard_normal((T, d), dtype=np.float32)
    V = g.standard_normal((T, d), dtype=np.float32)
    Q = g.standard_normal((n_q, d), dtype=np.float32)
    if hs.n_outlier > 0:
        ck = g.choice(d, size=hs.n_outlier, replace=False)
        cv = g.choice(d, size=hs.n_outlier, replace=False)
        K[:, ck] *= np.float32(hs.outlier_scale)
        V[:, cv] *= np.float32(hs.outlier_scale)
    n_heavy = int(round(hs.heavy_frac * T)) if hs.heavy_frac > 0 else hs.heavy_count
    if hs.n_sink > 0 or n_heavy > 0:
        qm = Q.astype(np.float64).mean(axis=0)
        q_hat = qm / np.linalg.norm(qm)
        n_sink = min(hs.n_sink, T)
        for j in range(n_sink):
            nrm = np.linalg.norm(K[j].astype(np.float64))
            K[j] = (hs.sink_scale * nrm * q_hat).astype(np.float32)
        n_heavy = min(n_heavy, T - n_sink)
        if n_heavy > 0:
            pos = n_sink + g.choice(T - n_sink, size=n_heavy, replace=False)
            for j in pos:
                nrm = np.linalg.norm(K[j].astype(np.float64))
                K[j] = (hs.heavy_scale * nrm * q_hat).astype(np.float32)
    if w.dtype == "bf16":
        K = bf16_bits_to_f32(to_bf16_bits(K))
        V = bf16_bits_to_f32(to_bf16_bits(V))
        Q = bf16_bits_to_f32(to_bf16_bits(Q))
    return K, V, Q


def gen_cache(w: Workload, cache: int, threads: int = 8) -> Dict[str, np.ndarray]:
    """All heads of one cache.

    Returns float32 arrays for "f32" workloads and uint16 bf16 bit patterns for
    "bf16" workloads: ``K, V [layers, kv_heads, T, d]`` and
    ``Q [layers, q_heads, n_obs, d]``.
    """
    T = w.caches[cache].T
    d = w.head.head_dim
    dt = np.float32 if w.dtype == "f32" else np.uint16
    K = np.empty((w.layers, w.kv_heads, T, d), dtype=dt)
    V = np.empty((w.layers, w.kv_heads, T, d), dtype=dt)
    Q = np.empty((w.layers, w.q_heads, w.n_obs, d), dtype=dt)
    Qv = Q.reshape(w.layers, w.kv_heads, w.n_q, d)

    def one(lh):
        l, h = lh
        k, v, q = gen_head(w, cache, l, h)
        if w.dtype == "bf16":
            K[l, h], V[l, h], Qv[l, h] = to_bf16_bits(k), to_bf16_bits(v), to_bf16_bits(q)
        else:
            K[l, h], V[l, h], Qv[l, h] = k, v, q

    items = [(l, h) for l in range(w.layers) for h in range(w.kv_heads)]
    if threads > 1 and len(items) > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(one, items))
    else:
        for it in items:
            one(it)
    return {"K": K, "V": V, "Q": Q}


def _ragged_T(seed: int, n: int) -> List[int]:
    g = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 0xC5])))
    return [int(t) for t in g.choice([1024, 2048, 4096, 8192], size=n, replace=True)]


def _budget(frac: float, T: int) -> int:
    return int(round(frac * T))


def _make_workloads() -> Dict[str, Workload]:
    out: Dict[str, Workload] = {}
    out["c1"] = Workload(
        name="c1", seed=0, layers=1, kv_heads=2, q_heads=8, n_obs=16, rank=1, dtype="f32",
        head=HeadSpec(head_dim=64, n_q=64, heavy_count=4, heavy_scale=4.0),
        caches=(CacheSpec(T=256, budget=32),))
    hs_outl = HeadSpec(head_dim=128, n_q=128, n_outlier=3, outlier_scale=8.0)
    out["c2"] = Workload(
        name="c2", seed=1, layers=1, kv_heads=8, q_heads=32, n_obs=32, rank=1, dtype="bf16",
        head=hs_outl, caches=(CacheSpec(T=2048, budget=205),))
    hs_full = HeadSpec(head_dim=128, n_q=128, n_outlier=3, outlier_scale=8.0,
                       heavy_frac=0.01, heavy_scale=4.0, n_sink=4, sink_scale=8.0)
    out["c3"] = Workload(
        name="c3", seed=2, layers=36, kv_heads=8, q_heads=32, n_obs=32, rank=1, dtype="bf16",
        head=hs_full, caches=(CacheSpec(T=4096, budget=819),))
    out["c4"] = Workload(
        name="c4", seed=3, layers=40, kv_heads=8, q_heads=32, n_obs=32, rank=4, dtype="bf16",
        head=hs_full, caches=(CacheSpec(T=8192, budget=811),))
    out["c4_evict"] = dataclasses.replace(out["c4"], name="c4_evict", rank=0)
    # the layerwise selector with the rank the paper pairs it with (L-OBF, pca_rank 4)
    out["c4_layer"] = dataclasses.replace(out["c4"], name="c4_layer", layerwise=True)
    # L-OBF + int8 (App. E, Table 7): the layerwise relay leaves as int8 codes
    out["c4_int8"] = dataclasses.replace(out["c4"], name="c4_int8", layerwise=True, int8_out=True)
    Ts = _ragged_T(4, 4)
    out["c5"] = Workload(
        name="c5", seed=4, layers=36, kv_heads=8, q_heads=32, n_obs=32, rank=2, dtype="bf16",
        head=hs_full, caches=tuple(CacheSpec(T=t, budget=_budget(0.15, t)) for t in Ts))
    # Paper regime (kv_budget = 32 < head_dim, 40 latent steps): the only large
    # shapes where OBF's dense algebra actually runs for every head.
    hs_paper = dataclasses.replace(hs_full, n_q=160)
    out["pa"] = Workload(
        name="pa", seed=5, layers=36, kv_heads=8, q_heads=32, n_obs=40, rank=2, dtype="bf16",
        head=hs_paper, caches=(CacheSpec(T=1024, budget=32),))
    out["pb"] = Workload(
        name="pb", seed=6, layers=36, kv_heads=8, q_heads=32, n_obs=40, rank=4, dtype="bf16",
        head=hs_paper, caches=(CacheSpec(T=2048, budget=32),))
    # the paper's own approximation of the subspace (App. H), on the paper-regime shape
    out["pa_fast"] = dataclasses.replace(out["pa"], name="pa_fast", fast_path=True)
    # the cache-merging comparison method on the paper-regime shape
    out["pa_merge"] = dataclasses.replace(out["pa"], name="pa_merge", merge=True)
    out["c4_early"] = dataclasses.replace(out["c4"], name="c4_early", early_out=True)
    return out


WORKLOADS: Dict[str, Workload] = _make_workloads()


def workload(name: str) -> Workload:
    return WORKLOADS[name]
