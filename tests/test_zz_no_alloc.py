"""evict_only_static: the entry point for callers that cannot allocate a workspace.

Such callers (a server that gave all device memory to its own pool, a plug-in
that must not allocate behind its host framework's back, a loop that cannot
afford an allocation's device-wide synchronisation) pass only inputs and
outputs; the scratch is a fixed array inside the library.  The test calls it
through the C ABI twice in a row, on different inputs, and requires the very
same outputs as evict_only with a caller-provided workspace: retained positions
and compacted K/V bit for bit (the parity tests' bar for eviction-only results),
and holds them against the CPU oracle's eviction-only result as well.
The second call finds the first call's leftovers in the shared array and must
not be affected by them.  Runs last so that a failure here cannot hide another
test's result.
"""
import ctypes

import pytest
import torch

import paper_2604_13349_b200 as P
from paper_2604_13349_b200 import binding, synth
from tests import _parity as par

pytestmark = pytest.mark.gpu


def _device_caches(w, arrays):
    dev, outs, caches = [], [], []
    tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    for ci, a in enumerate(arrays):
        K, V, Q = (par.to_device(a[n], w.dtype) for n in ("K", "V", "Q"))
        T, budget = w.caches[ci].T, w.caches[ci].budget
        ke = min(budget, T)
        o = {"K_out": torch.zeros((w.layers, w.kv_heads, ke, w.head.head_dim), dtype=tdt, device="cuda"),
             "V_out": torch.zeros((w.layers, w.kv_heads, ke, w.head.head_dim), dtype=tdt, device="cuda"),
             "idx": torch.full((w.layers, w.kv_heads, ke), -1, dtype=torch.int32, device="cuda")}
        dev.append((K, V, Q)); outs.append(o)
        caches.append(P.make_cache(K, V, Q, T, budget, o["K_out"], o["V_out"], o["idx"]))
    return dev, outs, caches


def _reference(w, arrays):
    outs, _, st = par.run_gpu(w, arrays, evict=True, want_scores=False)
    assert st & 0xFF == 0
    return outs


@pytest.mark.parametrize("names", [("c1", "c2"), ("c2", "c1")])
def test_static_scratch_entry_point_matches_evict_only_on_two_calls_in_a_row(names):
    for name in names:                                    # two calls in a row share the built-in array
        w = synth.workload(name)
        arrays = [synth.gen_cache(w, 0)]
        ref = _reference(w, arrays)
        dev, outs, caches = _device_caches(w, arrays)
        params = par.params_for(w)
        P.evict_only_static(params, caches)                # the first call on a device resolves the array's address
        torch.cuda.synchronize()
        for o in outs:
            o["idx"].fill_(-1); o["K_out"].zero_(); o["V_out"].zero_()
        torch.cuda.synchronize()
        before, before_free = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        P.evict_only_static(params, caches)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before     # nothing was allocated through torch
        assert torch.cuda.mem_get_info()[0] == before_free  # nor behind its back: the driver's free memory is unchanged
        assert P.obf_static_scratch_status() & 0xFF == 0
        for o, r in zip(outs, ref):
            assert torch.equal(o["idx"], r["idx"])
            assert torch.equal(o["K_out"], r["K_out"])
            assert torch.equal(o["V_out"], r["V_out"])
        # and against the oracle's eviction-only result: retained positions (bit-exact outside the tie band) and
        # bit-exact copies of the retained rows, every head
        stats = par.check_cache_whole(w, 0, arrays[0], outs[0], rank=0, name="static " + name)
        assert stats["heads"] == w.layers * w.kv_heads


def test_static_scratch_entry_point_rejects_shapes_beyond_its_array(capfd):
    w = synth.workload("c2")
    params = P.make_params(64, w.kv_heads, w.q_heads, 128, w.n_obs, 0, P.OBF_BF16)
    big = P.make_cache(0x1000, 0x1000, 0x1000, 8192, 100, 0x1000, 0x1000, 0x1000)
    need = P.obf_workspace_bytes(params, [big])
    assert need > binding.OBF_STATIC_SCRATCH_BYTES
    rc = P.evict_only_static(params, [big], check=False)   # refused on the host: nothing is enqueued
    assert rc == binding.OBF_ERR_WORKSPACE
    err = capfd.readouterr().err
    assert str(need) in err and str(binding.OBF_STATIC_SCRATCH_BYTES) in err
