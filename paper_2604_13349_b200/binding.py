"""Thin ctypes binding of the C ABI in ``include/obf.h``.

Argument marshalling only: every step of the compression runs in the CUDA
kernels of ``libobf_b200.so``.  PyTorch appears here for device memory and
streams, nothing else.  There is no CPU fallback: if the library has not been
built (``python -m paper_2604_13349_b200.build``) loading it raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence

import torch

from . import build as _build

OBF_OK = 0
OBF_ERR_INVALID_ARG = 1
OBF_ERR_UNSUPPORTED = 2
OBF_ERR_WORKSPACE = 3
OBF_ERR_CUDA = 4
OBF_ERR_DEVICE_STATUS = 5

OBF_F32 = 0
OBF_BF16 = 1

OBF_DEV_NONFINITE = 0x1
OBF_DEV_NO_CONVERGE = 0x2
OBF_DEV_TIMEOUT = 0x4
OBF_DEV_INTERNAL = 0x8
OBF_DEV_SKIPPED = 0x100
OBF_DEV_SPAN_FULL = 0x200

OBF_FLAG_GENERIC_PATH = 0x1
OBF_FLAG_LAYERWISE = 0x2        # one retained set per layer (masses summed over its KV heads)
OBF_FLAG_FAST_PATH = 0x4        # three Gram subspace iterations instead of the exact eigenvectors
OBF_FLAG_ATTN_INJECT = 0x8      # the back-fill shared out by attention mass instead of uniformly (App. D.2)
OBF_FLAG_EARLY_OUT = 0x20       # span test first; the pass over V skips heads whose retained values span R^d
OBF_FLAG_MERGE = 0x10           # cache-merging baseline instead of Orthogonal BackFill (App. E)
OBF_FLAG_TEST_WAIT_EXPIRES = 0x10000   # test hook: the score kernel's wait for a head's normalisers runs out


def OBF_FLAG_SINK(n: int) -> int:
    """Protected sink prefix: the first n <= 255 positions are retained besides the budget."""
    return (int(n) & 0xFF) << 8


def k_eff(T: int, budget: int, flags: int = 0) -> int:
    """Rows of K_out / V_out / idx per head for a cache of T positions."""
    s = min((flags >> 8) & 0xFF, T)
    return s + min(int(budget), T - s)
OBF_MAX_CACHES = 32

EXPORTS = ("obf_workspace_bytes", "obf_compress", "evict_only", "obf_host_arena_bytes",
           "obf_compress_host", "obf_last_device_status", "obf_status_string",
           "obf_last_launch_count", "obf_compress_profiled", "obf_phase_name",
           "evict_only_static", "obf_static_scratch_status")
OBF_STATIC_SCRATCH_BYTES = 8 << 20
OBF_MAX_PHASES = 16


class ObfParams(ctypes.Structure):
    _fields_ = [("layers", ctypes.c_int32), ("kv_heads", ctypes.c_int32), ("q_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("n_obs", ctypes.c_int32), ("rank", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("eps", ctypes.c_float), ("flags", ctypes.c_uint32)]


class ObfDiag(ctypes.Structure):
    _fields_ = [(n, ctypes.c_float) for n in (
        "a_keep", "a_del", "alpha", "rcr", "delta_norm", "kth_score", "next_score",
        "lam_1", "lam_rho", "lam_next")] + [
        ("span_rank", ctypes.c_int32), ("rho_eff", ctypes.c_int32), ("status", ctypes.c_uint32),
        ("revr", ctypes.c_float), ("pc", ctypes.c_float)]


DIAG_BYTES = ctypes.sizeof(ObfDiag)
DIAG_FLOAT_FIELDS = [n for n, t in ObfDiag._fields_ if t is ctypes.c_float]


class ObfCache(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("q_obs", ctypes.c_void_p),
                ("T", ctypes.c_int32), ("budget", ctypes.c_int32),
                ("k_out", ctypes.c_void_p), ("v_out", ctypes.c_void_p), ("idx_out", ctypes.c_void_p),
                ("diag_out", ctypes.c_void_p), ("scores_out", ctypes.c_void_p), ("delta_out", ctypes.c_void_p),
                ("lse_extra", ctypes.c_void_p), ("k_q8_out", ctypes.c_void_p), ("v_q8_out", ctypes.c_void_p),
                ("k_scale_out", ctypes.c_void_p), ("v_scale_out", ctypes.c_void_p), ("assign_out", ctypes.c_void_p)]


class ObfError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (status %d)" % (where, obf_status_string(code), code))


_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def load() -> ctypes.CDLL:
    """Loads ``libobf_b200.so``; raises if it has not been built."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(
                "CUDA extension %s is missing; build it with `python -m paper_2604_13349_b200.build` "
                "(there is no CPU fallback)" % path)
        lib = ctypes.CDLL(path)
        pp, pc = ctypes.POINTER(ObfParams), ctypes.POINTER(ObfCache)
        lib.obf_workspace_bytes.argtypes = [pp, pc, ctypes.c_int32, ctypes.POINTER(ctypes.c_size_t)]
        lib.obf_workspace_bytes.restype = ctypes.c_int
        lib.obf_host_arena_bytes.argtypes = [pp, pc, ctypes.c_int32, ctypes.POINTER(ctypes.c_size_t)]
        lib.obf_host_arena_bytes.restype = ctypes.c_int
        for name in ("obf_compress", "evict_only", "obf_compress_host"):
            fn = getattr(lib, name)
            fn.argtypes = [pp, pc, ctypes.c_int32, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
            fn.restype = ctypes.c_int
        lib.obf_last_device_status.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_uint32)]
        lib.obf_last_device_status.restype = ctypes.c_int
        lib.obf_status_string.argtypes = [ctypes.c_int]
        lib.obf_status_string.restype = ctypes.c_char_p
        lib.obf_compress_profiled.argtypes = [pp, pc, ctypes.c_int32, ctypes.c_void_p, ctypes.c_size_t,
                                              ctypes.c_void_p, ctypes.POINTER(ctypes.c_float),
                                              ctypes.POINTER(ctypes.c_int32)]
        lib.obf_compress_profiled.restype = ctypes.c_int
        lib.obf_phase_name.argtypes = [ctypes.c_int32]
        lib.obf_phase_name.restype = ctypes.c_char_p
        lib.evict_only_static.argtypes = [pp, pc, ctypes.c_int32, ctypes.c_void_p]
        lib.evict_only_static.restype = ctypes.c_int
        lib.obf_static_scratch_status.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_uint32)]
        lib.obf_static_scratch_status.restype = ctypes.c_int
        lib.obf_last_launch_count.argtypes = []
        lib.obf_last_launch_count.restype = ctypes.c_int32
        _lib = lib
    return _lib


def obf_status_string(code: int) -> str:
    return load().obf_status_string(int(code)).decode()


def make_params(layers: int, kv_heads: int, q_heads: int, head_dim: int, n_obs: int, rank: int,
                dtype: int, eps: float = 1e-12, flags: int = 0) -> ObfParams:
    return ObfParams(layers, kv_heads, q_heads, head_dim, n_obs, rank, dtype, eps, flags)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def make_cache(k, v, q_obs, T: int, budget: int, k_out, v_out, idx_out, diag_out=None,
               scores_out=None, delta_out=None, lse_extra=None, q8=None, assign_out=None) -> ObfCache:
    """Tensors (device or, for the host entry point, pinned/pageable CPU) or raw addresses.
    q8: (k_q8_out, v_q8_out, k_scale_out, v_scale_out) for the int8 copy of the relay, or None."""
    q8 = q8 or (None, None, None, None)
    return ObfCache(_ptr(k), _ptr(v), _ptr(q_obs), int(T), int(budget), _ptr(k_out), _ptr(v_out),
                    _ptr(idx_out), _ptr(diag_out), _ptr(scores_out), _ptr(delta_out), _ptr(lse_extra),
                    _ptr(q8[0]), _ptr(q8[1]), _ptr(q8[2]), _ptr(q8[3]), _ptr(assign_out))


def _carray(caches: Sequence[ObfCache]):
    arr = (ObfCache * len(caches))(*caches)
    return arr


def _stream_handle(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def obf_workspace_bytes(params: ObfParams, caches: Sequence[ObfCache]) -> int:
    out = ctypes.c_size_t(0)
    rc = load().obf_workspace_bytes(ctypes.byref(params), _carray(caches), len(caches), ctypes.byref(out))
    if rc != OBF_OK:
        raise ObfError(rc, "obf_workspace_bytes")
    return int(out.value)


def obf_host_arena_bytes(params: ObfParams, caches: Sequence[ObfCache]) -> int:
    out = ctypes.c_size_t(0)
    rc = load().obf_host_arena_bytes(ctypes.byref(params), _carray(caches), len(caches), ctypes.byref(out))
    if rc != OBF_OK:
        raise ObfError(rc, "obf_host_arena_bytes")
    return int(out.value)


def _call(name: str, params, caches, buf, buf_bytes, stream, check=True) -> int:
    rc = getattr(load(), name)(ctypes.byref(params), _carray(caches), len(caches),
                               _ptr(buf), int(buf_bytes), _stream_handle(stream))
    if check and rc != OBF_OK:
        raise ObfError(rc, name)
    return rc


def obf_compress(params, caches, workspace, workspace_bytes=None, stream=None, check=True) -> int:
    nb = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
    return _call("obf_compress", params, caches, workspace, nb, stream, check)


def evict_only(params, caches, workspace, workspace_bytes=None, stream=None, check=True) -> int:
    nb = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
    return _call("evict_only", params, caches, workspace, nb, stream, check)


def evict_only_static(params, caches, stream=None, check=True) -> int:
    """evict_only on the library's built-in scratch array, for callers that cannot allocate a
    workspace (see include/obf.h).  Inputs and outputs are device tensors as for evict_only; the
    call shape must fit OBF_STATIC_SCRATCH_BYTES; calls that overlap on the GPU race on the array."""
    rc = load().evict_only_static(ctypes.byref(params), _carray(caches), len(caches), _stream_handle(stream))
    if check and rc != OBF_OK:
        raise ObfError(rc, "evict_only_static")
    return rc


def obf_static_scratch_status(stream=None) -> int:
    """Status word left by the last evict_only_static call on the current device."""
    out = ctypes.c_uint32(0)
    rc = load().obf_static_scratch_status(_stream_handle(stream), ctypes.byref(out))
    if rc not in (OBF_OK, OBF_ERR_DEVICE_STATUS):
        raise ObfError(rc, "obf_static_scratch_status")
    return int(out.value)


def obf_compress_host(params, caches, device_arena, arena_bytes=None, stream=None, check=True) -> int:
    nb = device_arena.numel() * device_arena.element_size() if arena_bytes is None else arena_bytes
    return _call("obf_compress_host", params, caches, device_arena, nb, stream, check)


def obf_compress_profiled(params, caches, workspace, workspace_bytes=None, stream=None):
    """Runs the call with an event after every launch; returns [(kernel name, milliseconds), ...]."""
    nb = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
    ms = (ctypes.c_float * OBF_MAX_PHASES)()
    n = ctypes.c_int32(0)
    rc = load().obf_compress_profiled(ctypes.byref(params), _carray(caches), len(caches), _ptr(workspace),
                                      int(nb), _stream_handle(stream), ms, ctypes.byref(n))
    if rc != OBF_OK:
        raise ObfError(rc, "obf_compress_profiled")
    return [(load().obf_phase_name(i).decode(), float(ms[i])) for i in range(n.value)]


def obf_last_device_status(workspace, stream=None) -> int:
    out = ctypes.c_uint32(0)
    rc = load().obf_last_device_status(_ptr(workspace), _stream_handle(stream), ctypes.byref(out))
    if rc not in (OBF_OK, OBF_ERR_DEVICE_STATUS):
        raise ObfError(rc, "obf_last_device_status")
    return int(out.value)


def obf_last_launch_count() -> int:
    return int(load().obf_last_launch_count())


# ---------------------------------------------------------------------------
# convenience: allocate outputs with torch and call the C ABI once
# ---------------------------------------------------------------------------
def _torch_dtype(dtype: int):
    return torch.float32 if dtype == OBF_F32 else torch.bfloat16


def parse_diag(diag_bytes: torch.Tensor) -> List[Dict[str, float]]:
    """uint8 tensor [heads, sizeof(obf_diag_t)] (any device) -> list of dicts."""
    raw = diag_bytes.detach().cpu().contiguous().numpy().tobytes()
    n = len(raw) // DIAG_BYTES
    arr = (ObfDiag * n).from_buffer_copy(raw)
    return [{name: getattr(arr[i], name) for name, _ in ObfDiag._fields_} for i in range(n)]


def compress_caches(params: ObfParams, caches_in: Sequence[Dict[str, object]], *, evict: bool = False,
                    want_scores: bool = False, want_delta: bool = True, want_diag: bool = True,
                    want_int8: bool = False, want_assign: bool = False,
                    stream=None, workspace: Optional[torch.Tensor] = None) -> List[Dict[str, object]]:
    """Compress a batch of device caches.

    ``caches_in``: dicts with device tensors ``K, V [layers, kv_heads, T, d]``,
    ``Q [layers, q_heads, n_obs, d]``, an int ``budget`` and optionally ``lse_extra [layers, q_heads, n_obs]``
    (fp32, the out-of-prompt softmax mass per observation query).  Returns one dict per
    cache with ``K_out, V_out, idx`` (and ``scores``, ``delta``, ``diag`` bytes when asked).
    """
    dt = _torch_dtype(params.dtype)
    hpc = params.layers * params.kv_heads
    outs, cs = [], []
    for ci in caches_in:
        K, V, Q = ci["K"], ci["V"], ci["Q"]
        assert K.is_cuda and K.is_contiguous() and V.is_contiguous() and Q.is_contiguous()
        assert K.dtype == dt and V.dtype == dt and Q.dtype == dt
        T = K.shape[2]
        ke = k_eff(T, ci["budget"], params.flags)
        dev = K.device
        o = {
            "K_out": torch.empty((params.layers, params.kv_heads, ke, params.head_dim), dtype=dt, device=dev),
            "V_out": torch.empty((params.layers, params.kv_heads, ke, params.head_dim), dtype=dt, device=dev),
            "idx": torch.empty((params.layers, params.kv_heads, ke), dtype=torch.int32, device=dev),
            "diag": torch.zeros((hpc, DIAG_BYTES), dtype=torch.uint8, device=dev) if want_diag else None,
            "scores": torch.empty((params.layers, params.kv_heads, T), dtype=torch.float32, device=dev)
            if want_scores else None,
            "delta": torch.zeros((params.layers, params.kv_heads, params.head_dim), dtype=torch.float32,
                                 device=dev) if want_delta else None,
        }
        q8 = None
        if want_int8:
            o["K_q8"] = torch.empty((params.layers, params.kv_heads, ke, params.head_dim), dtype=torch.int8, device=dev)
            o["V_q8"] = torch.empty_like(o["K_q8"])
            o["K_scale"] = torch.empty((params.layers, params.kv_heads, ke), dtype=torch.float32, device=dev)
            o["V_scale"] = torch.empty_like(o["K_scale"])
            q8 = (o["K_q8"], o["V_q8"], o["K_scale"], o["V_scale"])
        o["assign"] = torch.empty((params.layers, params.kv_heads, T), dtype=torch.int32, device=dev) if want_assign else None
        outs.append(o)
        cs.append(make_cache(K, V, Q, T, ci["budget"], o["K_out"], o["V_out"], o["idx"], o["diag"],
                             o["scores"], o["delta"], ci.get("lse_extra"), q8, o["assign"]))
    nb = obf_workspace_bytes(params, cs)
    if workspace is None or workspace.numel() * workspace.element_size() < nb:
        workspace = torch.empty(nb, dtype=torch.uint8, device=caches_in[0]["K"].device)
    (evict_only if evict else obf_compress)(params, cs, workspace, stream=stream)
    for o in outs:
        o["workspace"] = workspace
        o["cache_structs"] = cs                 # for a repeated call on the same buffers (profiling)
    return outs
