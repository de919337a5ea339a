"""The C-ABI library: it loads, exports every symbol the header declares, and
rejects bad arguments on the host before touching a device (no GPU needed)."""
import ctypes
import os
import re

import pytest

import paper_2604_13349_b200 as P
from paper_2604_13349_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "obf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"^\s*#.*$", "", text, flags=re.M)            # preprocessor lines declare nothing
    return sorted(set(re.findall(r"\b(\w+)\s*\([^;{}]*\)\s*;", text)))


def test_header_functions_are_all_exported(lib):
    names = declared_functions()
    assert set(binding.EXPORTS) == set(names)
    for n in names:
        assert getattr(lib, n) is not None


def test_struct_sizes_match_the_header():
    assert ctypes.sizeof(binding.ObfParams) == 36
    assert ctypes.sizeof(binding.ObfDiag) == 60
    assert ctypes.sizeof(binding.ObfCache) == 128


def test_status_strings(lib):
    seen = {P.obf_status_string(c) for c in range(6)}
    assert len(seen) == 6 and "ok" in seen
    assert P.obf_status_string(99) == "unknown status"


def _params(**kw):
    base = dict(layers=1, kv_heads=2, q_heads=8, head_dim=64, n_obs=16, rank=1, dtype=P.OBF_F32)
    base.update(kw)
    return P.make_params(**base)


def _cache(T=256, budget=32, ptr=0x1000):
    return P.make_cache(ptr, ptr, ptr, T, budget, ptr, ptr, ptr)


def test_workspace_size_grows_with_the_problem(lib):
    a = P.obf_workspace_bytes(_params(), [_cache()])
    b = P.obf_workspace_bytes(_params(), [_cache(T=512)])
    c = P.obf_workspace_bytes(_params(rank=0), [_cache()])
    d = P.obf_workspace_bytes(_params(), [_cache(), _cache(T=100, budget=7)])
    assert b > a > c > 0 and d > a
    assert a % 256 == 0


@pytest.mark.parametrize("kw,code", [
    (dict(head_dim=96), binding.OBF_ERR_UNSUPPORTED),
    (dict(dtype=7), binding.OBF_ERR_UNSUPPORTED),
    (dict(q_heads=7), binding.OBF_ERR_INVALID_ARG),
    (dict(rank=-1), binding.OBF_ERR_INVALID_ARG),
    (dict(rank=65), binding.OBF_ERR_INVALID_ARG),
    (dict(layers=0), binding.OBF_ERR_INVALID_ARG),
    (dict(n_obs=0), binding.OBF_ERR_INVALID_ARG),
    (dict(eps=-1.0), binding.OBF_ERR_INVALID_ARG),
])
def test_bad_params_are_rejected_on_the_host(lib, kw, code):
    with pytest.raises(P.ObfError) as e:
        P.obf_workspace_bytes(_params(**kw), [_cache()])
    assert e.value.code == code


@pytest.mark.parametrize("cache,code", [
    (dict(T=0), binding.OBF_ERR_INVALID_ARG),
    (dict(budget=0), binding.OBF_ERR_INVALID_ARG),
    (dict(T=(1 << 20) + 1), binding.OBF_ERR_INVALID_ARG),
])
def test_bad_cache_shapes_are_rejected_on_the_host(lib, cache, code):
    with pytest.raises(P.ObfError) as e:
        P.obf_workspace_bytes(_params(), [_cache(**cache)])
    assert e.value.code == code


def test_compress_rejects_before_any_launch(lib):
    # None of these calls reaches the CUDA runtime: validation comes first.
    p = _params()
    pp, arr = ctypes.byref(p), (binding.ObfCache * 1)(_cache())
    assert lib.obf_compress(pp, arr, 0, 0x100, 1 << 30, None) == binding.OBF_ERR_INVALID_ARG
    assert lib.obf_compress(pp, arr, 33, 0x100, 1 << 30, None) == binding.OBF_ERR_UNSUPPORTED
    assert lib.obf_compress(None, arr, 1, 0x100, 1 << 30, None) == binding.OBF_ERR_INVALID_ARG
    assert lib.obf_compress(pp, arr, 1, None, 1 << 30, None) == binding.OBF_ERR_WORKSPACE
    assert lib.obf_compress(pp, arr, 1, 0x101, 1 << 30, None) == binding.OBF_ERR_WORKSPACE     # misaligned
    assert lib.obf_compress(pp, arr, 1, 0x100, 16, None) == binding.OBF_ERR_WORKSPACE          # too small
    null_k = (binding.ObfCache * 1)(P.make_cache(None, 0x1000, 0x1000, 256, 32, 0x1000, 0x1000, 0x1000))
    assert lib.obf_compress(pp, null_k, 1, 0x100, 1 << 30, None) == binding.OBF_ERR_INVALID_ARG
    odd = (binding.ObfCache * 1)(P.make_cache(0x1004, 0x1000, 0x1000, 256, 32, 0x1000, 0x1000, 0x1000))
    assert lib.evict_only(pp, odd, 1, 0x100, 1 << 30, None) == binding.OBF_ERR_INVALID_ARG
    assert lib.obf_compress_host(pp, arr, 1, None, 0, None) == binding.OBF_ERR_WORKSPACE
    assert lib.obf_last_launch_count() == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(build, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load()
