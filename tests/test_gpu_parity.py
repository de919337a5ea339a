"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle.

Bar: retained positions bit-exact outside a 1e-6 tie band on the attention
mass; K_out a bit-exact gather; V_out bit-exact where no injection happens,
within 1e-4 (fp32) / 2e-2 relative (bf16) otherwise; delta compared with an
eigen-gap-aware tolerance (the principal subspace is only determined up to the
gap between the last kept and first dropped eigenvalue).
"""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
import paper_2604_13349_b200 as P
from paper_2604_13349_b200 import synth
from tests import _parity as par

pytestmark = pytest.mark.gpu


def small(name, *, seed=7, layers=1, kv_heads=2, G=2, n_obs=5, d=64, dtype="f32", rank=2,
          caches=((100, 10),), heavy=3, n_outlier=0, n_sink=0):
    hs = synth.HeadSpec(head_dim=d, n_q=G * n_obs, n_outlier=n_outlier, heavy_count=heavy, n_sink=n_sink)
    return synth.Workload(name=name, seed=seed, layers=layers, kv_heads=kv_heads, q_heads=kv_heads * G,
                          n_obs=n_obs, rank=rank, dtype=dtype, head=hs,
                          caches=tuple(synth.CacheSpec(T=t, budget=b) for t, b in caches))


def all_heads(w):
    return [(l, h) for l in range(w.layers) for h in range(w.kv_heads)]


def run_and_check(w, rank=None, evict=False, heads=None, arrays=None, flags=0):
    arrays = arrays or [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
    outs, _, st = par.run_gpu(w, arrays, rank=rank, evict=evict, flags=flags)
    assert st & 0xFF == 0, "device status %#x" % st
    eff_rank = 0 if evict else (w.rank if rank is None else rank)
    reps = []
    for ci in range(len(w.caches)):
        reps += par.check_cache(w, ci, arrays[ci], outs[ci], heads or all_heads(w), rank=eff_rank)
    print("\n[%s] %s" % (w.name, par.summarize(reps)))
    return outs, reps, arrays


# ---------------------------------------------------------------------------
# benchmark configurations that the oracle finishes whole
# ---------------------------------------------------------------------------
def test_c1_tiny_fp32_whole():
    outs, reps, _ = run_and_check(synth.workload("c1"))
    assert all(not r.oracle_skipped for r in reps)          # budget 32 < head_dim 64: OBF is active
    assert all(not r.band_mismatch for r in reps)


def test_c1_rank0_and_evict_only_agree():
    w = synth.workload("c1")
    a, _, arrays = run_and_check(w, rank=0)
    b, _, _ = run_and_check(w, evict=True, arrays=arrays)
    for x, y in zip(a, b):
        assert torch.equal(x["idx"], y["idx"]) and torch.equal(x["K_out"], y["K_out"])
        assert torch.equal(x["V_out"], y["V_out"])


def test_c2_bf16_whole():
    outs, reps, _ = run_and_check(synth.workload("c2"))
    assert all(r.oracle_skipped for r in reps)              # budget 205 > head_dim: span is full, delta = 0
    diags = P.parse_diag(outs[0]["diag"])
    assert all(dg["status"] & P.binding.OBF_DEV_SPAN_FULL for dg in diags)
    assert all(dg["span_rank"] == 128 for dg in diags)


# ---------------------------------------------------------------------------
# shapes: ragged tiles, tiny T, every dtype / head_dim, multi-layer, ragged batch
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("T,budget", [(1, 1), (2, 1), (63, 9), (65, 64), (129, 17), (1000, 31), (1025, 100)])
def test_ragged_shapes(dtype, d, T, budget):
    w = small("ragged", d=d, dtype=dtype, caches=((T, budget),), heavy=min(3, T), seed=T * 3 + d)
    run_and_check(w)


@pytest.mark.parametrize("G,n_obs", [(1, 1), (1, 5), (3, 7), (4, 16), (4, 40), (5, 32)])
def test_query_counts(G, n_obs):
    w = small("queries", G=G, n_obs=n_obs, d=128, dtype="bf16", caches=((300, 20),), n_outlier=3, seed=G * 10 + n_obs)
    run_and_check(w)


def test_multi_layer_ragged_batch_in_one_call():
    w = small("batch", layers=3, kv_heads=2, d=128, dtype="bf16", rank=2, n_sink=4,
              caches=((130, 13), (64, 64), (777, 100), (40, 3), (1, 1)))
    outs, reps, _ = run_and_check(w)
    assert len(reps) == 5 * 6


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_budget_at_least_T_is_the_identity(dtype):
    w = small("identity", d=64, dtype=dtype, caches=((50, 50), (50, 80)))
    outs, _, arrays = run_and_check(w)
    for ci in range(2):
        assert torch.equal(outs[ci]["idx"][0, 0].cpu(), torch.arange(50, dtype=torch.int32))
        assert np.array_equal(par.out_bits(outs[ci]["K_out"]), arrays[ci]["K"].view(
            np.int16 if dtype == "bf16" else np.int32))
        assert np.array_equal(par.out_bits(outs[ci]["V_out"]), arrays[ci]["V"].view(
            np.int16 if dtype == "bf16" else np.int32))


@pytest.mark.parametrize("rank", [1, 3, 64])
def test_rank_sweep_including_full_rank_cap(rank):
    w = small("ranks", d=64, dtype="f32", rank=rank, caches=((200, 12),))
    outs, reps, _ = run_and_check(w)
    assert all(not r.oracle_skipped for r in reps)


def test_codimension_one():
    w = small("codim1", d=64, dtype="f32", rank=2, caches=((150, 63),))
    outs, reps, _ = run_and_check(w)
    diags = P.parse_diag(outs[0]["diag"])
    assert all(dg["span_rank"] == 63 and dg["rho_eff"] == 1 for dg in diags)


def test_budget_above_head_dim_full_rank_is_bit_exact_eviction():
    w = small("full", d=64, dtype="bf16", rank=3, caches=((400, 90),))
    outs, reps, _ = run_and_check(w)
    assert all(r.oracle_skipped for r in reps)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_rank_deficient_values_with_budget_above_head_dim(dtype):
    # every value lives in the first 40 channels except a few tokens the keys make unselectable:
    # budget >= head_dim, span(V_keep) has dimension 40, the residual is not zero.
    w = small("rd", d=64, dtype=dtype, rank=2, caches=((300, 80),), heavy=0, kv_heads=2, seed=21)
    arrays = [synth.gen_cache(w, 0)]
    a = arrays[0]
    K = par.f32_view(a["K"], dtype).copy(); V = par.f32_view(a["V"], dtype).copy()
    Qv = par.f32_view(a["Q"], dtype).reshape(1, 2, w.n_q, 64)
    g = np.random.default_rng(5)
    V[..., 40:] = 0.0
    for h in range(2):
        qm = Qv[0, h].mean(axis=0)
        odd = g.choice(300, 15, replace=False)
        K[0, h, odd] = -1.5 * qm / np.linalg.norm(qm) * np.linalg.norm(K[0, h, odd], axis=1, keepdims=True)
        V[0, h, odd, 40:] = g.standard_normal((15, 24)).astype(np.float32)
    if dtype == "bf16":
        a["K"], a["V"] = synth.to_bf16_bits(K), synth.to_bf16_bits(V)
    else:
        a["K"], a["V"] = K, V
    outs, reps, _ = run_and_check(w, arrays=arrays)
    diags = P.parse_diag(outs[0]["diag"])
    assert all(dg["span_rank"] == 40 for dg in diags)
    assert all(not r.oracle_skipped for r in reps)
    assert torch.all(outs[0]["delta"][..., :40].abs() < 1e-5)
    assert torch.all(outs[0]["delta"].norm(dim=-1) > 1e-6)


# ---------------------------------------------------------------------------
# tuned bf16 / head_dim 128 path (tensor cores) against the oracle and against the shape-generic path
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("caches", [((128, 16),), ((300, 20), (130, 129), (777, 100)), ((1000, 200), (257, 31)),
                                    ((4096, 64),)])
def test_tuned_path_ragged_batches_match_oracle_and_generic_path(caches):
    w = small("tuned", layers=2, kv_heads=3, G=2, n_obs=9, d=128, dtype="bf16", rank=2, caches=caches,
              n_outlier=3, n_sink=2, seed=len(caches) * 31 + caches[0][0])
    a, reps, arrays = run_and_check(w)
    b, _, _ = run_and_check(w, arrays=arrays, flags=P.binding.OBF_FLAG_GENERIC_PATH)
    for x, y in zip(a, b):
        assert torch.equal(x["K_out"], y["K_out"])
        same = torch.equal(x["idx"], y["idx"])
        if same:
            assert torch.allclose(x["delta"], y["delta"], atol=2e-4, rtol=1e-3)
    assert any(not r.oracle_skipped for r in reps) or all(c[1] >= 128 for c in caches)


def test_tuned_path_with_many_caches_of_different_lengths():
    # twelve caches in one call: every role of the score kernel walks the per-cache table
    Ts = [128, 131, 200, 256, 300, 511, 512, 513, 640, 777, 900, 1025]
    w = small("many", layers=1, kv_heads=2, G=2, n_obs=8, d=128, dtype="bf16", rank=2,
              caches=tuple((t, 16 + (t % 7)) for t in Ts), n_outlier=3, n_sink=2, seed=5)
    a, reps, arrays = run_and_check(w)
    assert all(not r.oracle_skipped for r in reps)
    b, _, _ = run_and_check(w, arrays=arrays, flags=P.binding.OBF_FLAG_GENERIC_PATH)
    for x, y in zip(a, b):
        assert torch.equal(x["K_out"], y["K_out"])


def test_tuned_path_rank_deficient_values_with_budget_above_head_dim():
    # head_dim 128, budget 160 >= head_dim, but every selectable value lives in the first 90 channels
    w = small("rd128", d=128, dtype="bf16", rank=3, caches=((700, 160),), heavy=0, kv_heads=2, seed=23)
    arrays = [synth.gen_cache(w, 0)]
    a = arrays[0]
    K = par.f32_view(a["K"], "bf16").copy(); V = par.f32_view(a["V"], "bf16").copy()
    Qv = par.f32_view(a["Q"], "bf16").reshape(1, 2, w.n_q, 128)
    g = np.random.default_rng(6)
    V[..., 90:] = 0.0
    for h in range(2):
        qm = Qv[0, h].mean(axis=0)
        odd = g.choice(700, 40, replace=False)
        K[0, h, odd] = -1.5 * qm / np.linalg.norm(qm) * np.linalg.norm(K[0, h, odd], axis=1, keepdims=True)
        V[0, h, odd, 90:] = g.standard_normal((40, 38)).astype(np.float32)
    a["K"], a["V"] = synth.to_bf16_bits(K), synth.to_bf16_bits(V)
    outs, reps, _ = run_and_check(w, arrays=arrays)
    diags = P.parse_diag(outs[0]["diag"])
    assert all(dg["span_rank"] == 90 for dg in diags)
    assert all(not r.oracle_skipped for r in reps)
    assert torch.all(outs[0]["delta"][..., :90].abs() < 1e-4)
    assert torch.all(outs[0]["delta"].norm(dim=-1) > 1e-6)


def _subspace_case(full_later: bool):
    """T = 2000, budget 400 >= head_dim.  Positions below 1500 hold values confined to the first 100 channels, so
    the first 256 retained rows (the subset the span test factorises) have rank 100.  full_later: the values at
    positions >= 1500 fill all 128 channels, else they are confined too and only a few unselectable tokens carry
    the other channels."""
    w = small("subspace", d=128, dtype="bf16", rank=3, caches=((2000, 400),), heavy=0, kv_heads=2, seed=29)
    arrays = [synth.gen_cache(w, 0)]
    a = arrays[0]
    K = par.f32_view(a["K"], "bf16").copy(); V = par.f32_view(a["V"], "bf16").copy()
    Qv = par.f32_view(a["Q"], "bf16").reshape(1, 2, w.n_q, 128)
    g = np.random.default_rng(8)
    V[:, :, :1500, 100:] = 0.0
    if not full_later:
        V[:, :, 1500:, 100:] = 0.0
        for h in range(2):
            qm = Qv[0, h].mean(axis=0)
            odd = g.choice(2000, 60, replace=False)
            K[0, h, odd] = -1.5 * qm / np.linalg.norm(qm) * np.linalg.norm(K[0, h, odd], axis=1, keepdims=True)
            V[0, h, odd, 100:] = g.standard_normal((60, 28)).astype(np.float32)
    a["K"], a["V"] = synth.to_bf16_bits(K), synth.to_bf16_bits(V)
    outs, reps, _ = run_and_check(w, arrays=arrays)
    idx = outs[0]["idx"].cpu().numpy()
    for h in range(2):
        assert (idx[0, h] < 1500).sum() >= 256 and (idx[0, h] >= 1500).sum() >= 40    # the construction holds
    return outs, reps


def test_span_subset_deficient_but_all_retained_rows_span_everything():
    # the Cholesky test on the first 256 retained rows fails; Gram-Schmidt over all 400 must reach rank 128: delta = 0
    outs, reps = _subspace_case(full_later=True)
    diags = P.parse_diag(outs[0]["diag"])
    assert all(dg["span_rank"] == 128 for dg in diags)
    assert all(r.oracle_skipped for r in reps)               # run_and_check has compared V_out bit for bit
    assert torch.all(outs[0]["delta"] == 0)


def test_span_subset_deficient_and_all_retained_rows_deficient_too():
    outs, reps = _subspace_case(full_later=False)
    diags = P.parse_diag(outs[0]["diag"])
    assert all(dg["span_rank"] == 100 for dg in diags)
    assert all(not r.oracle_skipped for r in reps)
    assert torch.all(outs[0]["delta"][..., :100].abs() < 1e-4)
    assert torch.all(outs[0]["delta"].norm(dim=-1) > 1e-6)


def test_retained_rows_with_a_dominant_common_component():
    # budget 24 < head_dim: every value is a common vector plus 3 % of noise, so after the first retained row every
    # further row loses nearly all of its norm to the basis in the first Gram-Schmidt pass and the kernel has to go
    # round a second time for it (a row that keeps more than half of its squared norm is orthogonalised once);
    # the basis, delta and V_out must still agree with the oracle, which always orthogonalises twice
    w = small("common", d=128, dtype="bf16", rank=2, caches=((900, 24),), heavy=4, kv_heads=2, seed=41)
    arrays = [synth.gen_cache(w, 0)]
    a = arrays[0]
    V = par.f32_view(a["V"], "bf16").copy()
    g = np.random.default_rng(5)
    common = g.standard_normal(128).astype(np.float32)
    V[:] = common + 0.03 * V
    a["V"] = synth.to_bf16_bits(V)
    outs, reps, _ = run_and_check(w, arrays=arrays)
    diags = P.parse_diag(outs[0]["diag"])
    assert all(dg["span_rank"] == 24 for dg in diags)
    assert all(not r.oracle_skipped for r in reps)
    assert torch.all(outs[0]["delta"].norm(dim=-1) > 0)


@pytest.mark.parametrize("T,budget", [(20000, 300), (70000, 250), (80000, 200)])
def test_long_prompts_take_the_fallback_kernels(T, budget):
    # 20000 keys: more than the select kernel keeps in shared memory; 70000 keys: one head's team is 137 blocks,
    # nearly the whole grid of the persistent score kernel; 80000 keys: more chunks than that kernel has blocks,
    # so the shape-generic score kernels run (the Gram pass stays tuned)
    w = small("long", layers=1, kv_heads=1, G=4, n_obs=8, d=128, dtype="bf16", rank=1, caches=((T, budget),),
              n_outlier=3, n_sink=4, heavy=8, seed=T % 97)
    outs, reps, _ = run_and_check(w)
    assert all(r.oracle_skipped for r in reps)              # budget >= head_dim with generic values: delta = 0


@pytest.mark.parametrize("G,n_obs,caches", [(5, 32, ((640, 24),)),          # 160 rows: two query tiles per head
                                            (4, 40, ((1024, 32), (300, 20), (2048, 32))),   # the paper's 40 latent steps
                                            (8, 32, ((700, 40),)),          # 256 rows: two full tiles
                                            (2, 65, ((513, 30),))])         # 130 rows: second tile nearly empty
def test_between_129_and_256_query_rows_take_two_query_tiles_per_head(G, n_obs, caches):
    w = small("wideq", layers=2, kv_heads=3, G=G, n_obs=n_obs, d=128, dtype="bf16", rank=2, caches=caches,
              n_outlier=3, seed=77 + G)
    a, reps, arrays = run_and_check(w)
    assert all(not r.oracle_skipped for r in reps)
    names = [n for n, _ in P.obf_compress_profiled(par.params_for(w), a[0]["cache_structs"], a[0]["workspace"])]
    assert "k_score_tc" in names and "k_score_join" in names
    b, _, _ = run_and_check(w, arrays=arrays, flags=P.binding.OBF_FLAG_GENERIC_PATH)
    for x, y in zip(a, b):
        assert torch.equal(x["K_out"], y["K_out"])


def test_more_than_256_query_rows_use_the_generic_score_kernels_and_the_tuned_gram_pass():
    w = small("widerq", layers=1, kv_heads=2, G=9, n_obs=32, d=128, dtype="bf16", rank=2, caches=((640, 24),),
              n_outlier=3, seed=78)
    outs, reps, arrays = run_and_check(w)
    assert all(not r.oracle_skipped for r in reps)
    names = [n for n, _ in P.obf_compress_profiled(par.params_for(w), outs[0]["cache_structs"], outs[0]["workspace"])]
    assert "k_score_stats" in names and "k_gram_tc" in names


def test_exact_ties_go_to_the_lowest_position():
    # duplicated keys give bit-identical masses on the GPU as well; ties must resolve to lower positions
    w = small("ties", d=64, dtype="f32", rank=0, caches=((96, 20),), heavy=0, kv_heads=1)
    arrays = [synth.gen_cache(w, 0)]
    K = arrays[0]["K"]
    K[0, 0, 48:] = K[0, 0, :48]                          # position j+48 duplicates position j
    outs, _, st = par.run_gpu(w, arrays, rank=0)
    idx = outs[0]["idx"][0, 0].cpu().numpy()
    sc = outs[0]["scores"][0, 0].cpu().numpy()
    assert np.array_equal(sc[:48], sc[48:])
    ref = oracle.topk(sc.astype(np.float64), 20)[0]      # the oracle's rule applied to the GPU's own masses
    assert np.array_equal(idx, ref)
    assert all((j - 48) in idx for j in idx if j >= 48)     # a kept duplicate implies its lower twin is kept
    all_equal = small("alleq", d=64, dtype="bf16", rank=0, caches=((77, 11),), heavy=0, kv_heads=1)
    arr2 = [synth.gen_cache(all_equal, 0)]
    arr2[0]["K"][0, 0, :] = arr2[0]["K"][0, 0, 0]
    o2, _, _ = par.run_gpu(all_equal, arr2, rank=0)
    assert np.array_equal(o2[0]["idx"][0, 0].cpu().numpy(), np.arange(11))


def test_runs_are_deterministic():
    w = synth.workload("c1")
    arrays = [synth.gen_cache(w, 0)]
    a, _, _ = par.run_gpu(w, arrays)
    b, _, _ = par.run_gpu(w, arrays)
    for key in ("idx", "K_out", "V_out", "scores", "delta"):
        assert torch.equal(a[0][key], b[0][key]), key


def test_non_finite_inputs_set_the_status_word_and_stay_in_bounds():
    w = small("nan", d=64, dtype="f32", rank=1, caches=((120, 10),), kv_heads=1)
    arrays = [synth.gen_cache(w, 0)]
    arrays[0]["K"][0, 0, 5, 3] = np.nan
    outs, _, st = par.run_gpu(w, arrays)
    assert st & P.binding.OBF_DEV_NONFINITE
    idx = outs[0]["idx"][0, 0].cpu().numpy()
    assert len(set(idx.tolist())) == 10 and idx.min() >= 0 and idx.max() < 120


def test_a_device_side_wait_that_runs_out_reports_a_timeout_and_the_kernels_return():
    # nothing publishes the head's softmax normalisers and the wait limit is 20 ms: the score kernel's wait runs out
    w = small("expire", layers=1, kv_heads=2, G=2, n_obs=8, d=128, dtype="bf16", rank=2, caches=((700, 40),), seed=13)
    arrays = [synth.gen_cache(w, 0)]
    outs, dev, st = par.run_gpu(w, arrays, flags=P.binding.OBF_FLAG_TEST_WAIT_EXPIRES)
    assert st & P.binding.OBF_DEV_TIMEOUT
    idx = outs[0]["idx"].cpu().numpy()
    assert idx.min() >= 0 and idx.max() < 700               # whatever was selected lies inside the cache
    assert np.all(np.diff(idx, axis=-1) > 0)
    # the workspace, the streams and the device are as usable as before
    ws = outs[0]["workspace"]
    good = P.compress_caches(par.params_for(w), dev, want_scores=True, workspace=ws)
    torch.cuda.synchronize()
    assert P.obf_last_device_status(ws) & 0xFF == 0
    reps = par.check_cache(w, 0, arrays[0], good[0], all_heads(w))
    assert all(not r.oracle_skipped for r in reps)
    # the hook is refused outside its small shapes
    big = small("expire_big", layers=3, kv_heads=2, G=2, n_obs=8, d=128, dtype="bf16", caches=((700, 40),))
    with pytest.raises(Exception):
        par.run_gpu(big, [synth.gen_cache(big, 0)], flags=P.binding.OBF_FLAG_TEST_WAIT_EXPIRES)


def test_host_entry_point_matches_the_device_entry_point():
    w = synth.workload("c1")
    arrays = [synth.gen_cache(w, 0)]
    outs, _, _ = par.run_gpu(w, arrays)
    params = par.params_for(w)
    k = w.caches[0].budget
    hK = torch.from_numpy(arrays[0]["K"]).pin_memory(); hV = torch.from_numpy(arrays[0]["V"]).pin_memory()
    hQ = torch.from_numpy(arrays[0]["Q"]).pin_memory()
    oK = torch.empty((1, 2, k, 64)).pin_memory(); oV = torch.empty((1, 2, k, 64)).pin_memory()
    oI = torch.empty((1, 2, k), dtype=torch.int32).pin_memory()
    oD = torch.empty((1, 2, 64)).pin_memory()
    c = P.make_cache(hK, hV, hQ, 256, k, oK, oV, oI, None, None, oD)
    arena = torch.empty(P.obf_host_arena_bytes(params, [c]), dtype=torch.uint8, device="cuda")
    P.obf_compress_host(params, [c], arena)
    assert torch.equal(oI, outs[0]["idx"].cpu())
    assert torch.equal(oK, outs[0]["K_out"].cpu()) and torch.equal(oV, outs[0]["V_out"].cpu())
    assert torch.equal(oD, outs[0]["delta"].cpu())


@pytest.mark.parametrize("layers", [1, 5, 9])
def test_host_entry_point_pipelines_slabs_of_layers_for_ragged_batches(layers):
    # layer counts that the slabs do not divide evenly, two caches of different lengths, bf16 on the tuned path
    w = small("host", layers=layers, kv_heads=2, G=2, n_obs=8, d=128, dtype="bf16", rank=2,
              caches=((300, 20), (700, 140)), n_outlier=3, seed=19 + layers)
    arrays = [synth.gen_cache(w, ci) for ci in range(2)]
    outs, _, st = par.run_gpu(w, arrays)
    assert st & 0xFF == 0
    params = par.params_for(w)
    host, cs = [], []
    for ci, (T, b) in enumerate(((300, 20), (700, 140))):
        a = arrays[ci]
        h = {n: torch.from_numpy(a[n].view(np.int16)).view(torch.bfloat16).pin_memory() for n in ("K", "V", "Q")}
        h["oK"] = torch.empty((layers, 2, b, 128), dtype=torch.bfloat16).pin_memory()
        h["oV"] = torch.empty((layers, 2, b, 128), dtype=torch.bfloat16).pin_memory()
        h["oI"] = torch.empty((layers, 2, b), dtype=torch.int32).pin_memory()
        h["oS"] = torch.empty((layers, 2, T), dtype=torch.float32).pin_memory()
        h["oD"] = torch.empty((layers, 2, 128), dtype=torch.float32).pin_memory()
        host.append(h)
        cs.append(P.make_cache(h["K"], h["V"], h["Q"], T, b, h["oK"], h["oV"], h["oI"], None, h["oS"], h["oD"]))
    arena = torch.empty(P.obf_host_arena_bytes(params, cs), dtype=torch.uint8, device="cuda")
    for _ in range(2):                                      # twice: the second call reuses the arena and the streams
        P.obf_compress_host(params, cs, arena)
    for ci in range(2):
        h = host[ci]
        assert torch.equal(h["oI"], outs[ci]["idx"].cpu())
        assert torch.equal(h["oK"].view(torch.int16), outs[ci]["K_out"].cpu().view(torch.int16))
        assert torch.allclose(h["oV"].float(), outs[ci]["V_out"].cpu().float(), rtol=1e-2, atol=1e-5)
        assert torch.equal(h["oS"], outs[ci]["scores"].cpu())
        # the streaming pass cuts its tile sequence by the size of the call, so a slab adds its partial sums
        # up in another order than the whole call: delta agrees to fp32 rounding of the largest terms of those
        # sums (2^-22 of a value row's norm, about 15 here), not bit for bit
        assert torch.allclose(h["oD"], outs[ci]["delta"].cpu(), rtol=1e-4, atol=4e-6)


# ---------------------------------------------------------------------------
# benchmark configurations at full size: every head of every cache against one oracle run per cache, and the
# call shape the benchmark times (no optional outputs) bit for bit against the call with all outputs
# ---------------------------------------------------------------------------
@pytest.fixture(scope="module")
def c4_arrays():
    return [synth.gen_cache(synth.workload("c4"), 0)]


def run_whole(wname, arrays=None, evict=False, flags=0, layerwise=False):
    w = synth.workload(wname)
    arrays = arrays or [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
    outs, dev, st = par.run_gpu(w, arrays, evict=evict, flags=flags)
    assert st & 0xFF == 0, "device status %#x" % st
    # what the benchmark times: the same call without diagnostics, masses and delta
    bare, _, st2 = par.run_gpu(w, arrays, evict=evict, flags=flags, want_scores=False, dev=dev,
                               want_delta=False, want_diag=False)
    assert st2 & 0xFF == 0
    for x, y in zip(outs, bare):
        assert torch.equal(x["idx"], y["idx"]), "retained positions depend on the optional outputs"
        assert torch.equal(x["K_out"].view(torch.int16), y["K_out"].view(torch.int16))
        assert torch.equal(x["V_out"].view(torch.int16), y["V_out"].view(torch.int16))
    del bare
    total = {}
    for ci in range(len(w.caches)):
        st_ci = par.check_cache_whole(w, ci, arrays[ci], outs[ci], rank=0 if evict else None, layerwise=layerwise)
        for k, v in st_ci.items():
            total[k] = total.get(k, 0) + v
    print("\n[%s whole] %s" % (wname, total))
    assert total["heads"] == len(w.caches) * w.layers * w.kv_heads
    return total


def test_c3_full_size_every_head():
    run_whole("c3")


def test_c4_full_size_rank4_every_head(c4_arrays):
    run_whole("c4", arrays=c4_arrays)


def test_c4_full_size_evict_only_every_head(c4_arrays):
    run_whole("c4_evict", arrays=c4_arrays, evict=True)


def test_c4_full_size_layerwise_every_layer(c4_arrays):
    run_whole("c4_layer", arrays=c4_arrays, flags=P.binding.OBF_FLAG_LAYERWISE, layerwise=True)


def test_c5_ragged_relay_batch_every_head_of_every_cache():
    run_whole("c5")


def test_paper_regime_budget_32_every_head():
    # kv_budget = 32 < head_dim with 40 latent steps: OBF's dense algebra runs for every head
    total = run_whole("pa")
    assert total["backfilled"] == total["heads"]


# ---------------------------------------------------------------------------
# layerwise selector: one retained set per layer, back-fill per head
# ---------------------------------------------------------------------------
def run_and_check_layerwise(w, arrays=None, flags=0, evict=False):
    arrays = arrays or [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
    outs, _, st = par.run_gpu(w, arrays, evict=evict, flags=flags | P.binding.OBF_FLAG_LAYERWISE)
    assert st & 0xFF == 0, "device status %#x" % st
    reps = []
    for ci in range(len(w.caches)):
        reps += par.check_cache_layerwise(w, ci, arrays[ci], outs[ci], range(w.layers), rank=0 if evict else None)
    print("\n[%s layerwise] %s" % (w.name, par.summarize(reps)))
    return outs, reps, arrays


@pytest.mark.parametrize("dtype,d", [("f32", 64), ("bf16", 64), ("f32", 128)])
def test_layerwise_small_budgets_backfill_every_head(dtype, d):
    w = small("lw", layers=3, kv_heads=4, G=2, n_obs=5, d=d, dtype=dtype, rank=2, caches=((220, 14), (97, 9)), seed=33)
    outs, reps, _ = run_and_check_layerwise(w)
    assert all(not r.oracle_skipped for r in reps)              # budget < head_dim: OBF is active everywhere


def test_layerwise_c1_and_its_eviction_only_form():
    w = synth.workload("c1")
    a, reps, arrays = run_and_check_layerwise(w)
    assert all(not r.oracle_skipped for r in reps)
    b, _, _ = run_and_check_layerwise(w, arrays=arrays, evict=True)
    for x, y in zip(a, b):
        assert torch.equal(x["idx"], y["idx"]) and torch.equal(x["K_out"], y["K_out"])


@pytest.mark.parametrize("caches", [((300, 20), (130, 129), (777, 100)), ((2048, 205),)])
def test_layerwise_on_the_tensor_core_path(caches):
    w = small("lw_tuned", layers=2, kv_heads=3, G=2, n_obs=9, d=128, dtype="bf16", rank=4, caches=caches,
              n_outlier=3, n_sink=2, seed=51 + len(caches))
    a, reps, arrays = run_and_check_layerwise(w)
    b, _, _ = run_and_check_layerwise(w, arrays=arrays, flags=P.binding.OBF_FLAG_GENERIC_PATH)
    for x, y in zip(a, b):
        assert torch.equal(x["K_out"], y["K_out"])


def test_layerwise_with_one_kv_head_equals_headwise():
    w = small("lw1", layers=2, kv_heads=1, G=4, n_obs=4, d=64, dtype="f32", rank=1, caches=((150, 11),), seed=3)
    a, _, arrays = run_and_check_layerwise(w)
    b, _, _ = run_and_check(w, arrays=arrays)
    assert torch.equal(a[0]["idx"], b[0]["idx"]) and torch.equal(a[0]["V_out"], b[0]["V_out"])


def test_layerwise_rejects_prompts_that_do_not_fit_shared_memory():
    w = small("lw_long", layers=1, kv_heads=2, d=64, dtype="f32", rank=0, caches=((20000, 8),))
    arrays = [synth.gen_cache(w, 0)]
    with pytest.raises(Exception):
        par.run_gpu(w, arrays, flags=P.binding.OBF_FLAG_LAYERWISE)


# ---------------------------------------------------------------------------
# eigen-solve of the small-rank path: a residual spectrum with a tie at the top
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("rank", [1, 2, 3])
def test_residual_with_two_equal_leading_singular_values(rank):
    # The retained values live in the first 10 channels; every deleted value adds a component along channel 20
    # or channel 21, with the same energy on both and no correlation between them: the residual has two equal
    # leading singular values and nothing else.  Rank 2 and 3 have a unique answer (Delta = r_bar); rank 1 does
    # not (any direction of that plane is a leading singular vector), so only the invariants are checked for it.
    w = small("tie", d=64, dtype="f32", rank=rank, caches=((240, 12),), heavy=0, kv_heads=2, seed=77)
    arrays = [synth.gen_cache(w, 0)]
    a = arrays[0]
    Qv = a["Q"].reshape(1, 2, w.n_q, 64)
    g = np.random.default_rng(9)
    V = np.zeros_like(a["V"])
    for h in range(2):
        A = oracle.scores(a["K"][0, h], Qv[0, h])
        keep = np.zeros(240, bool); keep[oracle.topk(A, 12)[0]] = True
        V[0, h, :, :10] = g.standard_normal((240, 10)).astype(np.float32)
        dele = np.flatnonzero(~keep)
        half = len(dele) // 2
        V[0, h, dele[:half], 20] = 0.5                       # same count, same magnitude, disjoint supports
        V[0, h, dele[half:2 * half], 21] = 0.5
    a["V"] = V
    outs, reps, _ = run_and_check(w, arrays=arrays)
    assert all(not r.oracle_skipped for r in reps)
    d = outs[0]["delta"].cpu().numpy()
    assert np.all(np.abs(d[..., :10]) < 1e-5) and np.all(np.abs(d[..., 22:]) < 1e-5)
    if rank >= 2:
        assert all(r.gap_rel > 0.5 for r in reps)            # the plane itself is well separated from the rest
        assert np.all(np.linalg.norm(d, axis=-1) > 1e-4)


# ---------------------------------------------------------------------------
# protected sink prefix: the first s positions are retained besides the budget
# ---------------------------------------------------------------------------
def check_sink(w, n_sink, outs, arrays, layerwise=False, rank=None):
    rank = w.rank if rank is None else rank
    d, n_q, H = w.head.head_dim, w.n_q, w.kv_heads
    bits = np.int16 if w.dtype == "bf16" else np.int32
    reps = []
    for ci in range(len(w.caches)):
        a, out = arrays[ci], outs[ci]
        budget = w.caches[ci].budget
        Qv = a["Q"].reshape(w.layers, H, n_q, d)
        diags = P.parse_diag(out["diag"])
        for l in range(w.layers):
            K, V, Q = par.f32_view(a["K"][l], w.dtype), par.f32_view(a["V"][l], w.dtype), par.f32_view(Qv[l], w.dtype)
            lay = oracle.layer(K, V, Q, budget, rank, n_sink=n_sink) if layerwise else None
            for h in range(H):
                if layerwise:
                    ref = {"A": lay["A"][h], "idx": lay["idx"][h], "delta": lay["delta"][h], "V_out": lay["V_out"][h],
                           "diag": lay["diag"][h]}
                    sel, band = lay["S"].copy(), par.TIE_BAND * H
                else:
                    ref = oracle.head(K[h], V[h], Q[h], budget, rank, n_sink=n_sink)
                    sel, band = ref["A"].copy(), par.TIE_BAND
                sel[:n_sink] = np.inf                               # protected positions are never in the tie band
                g_idx = out["idx"][l, h].cpu().numpy()
                assert g_idx[:min(n_sink, K.shape[1])].tolist() == list(range(min(n_sink, K.shape[1])))
                reps.append(par.check_head(
                    w.dtype, K[h], V[h], Q[h], budget, rank, g_idx, par.out_bits(out["K_out"][l, h]),
                    par.out_bits(out["V_out"][l, h]), par.out_to_f32(out["V_out"][l, h]),
                    out["scores"][l, h].cpu().numpy(), out["delta"][l, h].cpu().numpy(), diags[l * H + h],
                    a["K"][l, h].view(bits), a["V"][l, h].view(bits), name="sink cache %d layer %d head %d" % (ci, l, h),
                    ref=ref, sel_scores=sel, tie_band=band, k_expected=oracle.k_eff(K.shape[1], budget, n_sink)))
    return reps


@pytest.mark.parametrize("dtype,d,caches,layerwise", [
    ("f32", 64, ((200, 12), (90, 9)), False), ("bf16", 128, ((300, 20), (777, 100), (130, 129)), False),
    ("f32", 64, ((200, 12),), True), ("bf16", 128, ((512, 28),), True)])
def test_sink_prefix_is_retained_besides_the_budget(dtype, d, caches, layerwise):
    w = small("sink", layers=2, kv_heads=3, G=2, n_obs=6, d=d, dtype=dtype, rank=2, caches=caches, seed=91, n_sink=0)
    arrays = [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
    flags = P.binding.OBF_FLAG_SINK(4) | (P.binding.OBF_FLAG_LAYERWISE if layerwise else 0)
    outs, _, st = par.run_gpu(w, arrays, flags=flags)
    assert st & 0xFF == 0
    for ci, (T, b) in enumerate(caches):
        assert outs[ci]["idx"].shape[-1] == min(4, T) + min(b, T - min(4, T))
    reps = check_sink(w, 4, outs, arrays, layerwise=layerwise)
    print("\n[sink] %s" % par.summarize(reps))


# ---------------------------------------------------------------------------
# out-of-prompt softmax mass: the keys outside the prompt take their share of every row's normaliser
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,d,G,n_obs,caches,flags", [
    ("f32", 64, 2, 5, ((200, 12), (90, 9)), 0),
    ("bf16", 128, 2, 9, ((300, 20), (777, 100), (1100, 32)), 0),                 # tuned score kernel, several chunks per head
    ("bf16", 128, 5, 32, ((640, 24),), 0),                                       # two query tiles per head
    ("bf16", 128, 2, 9, ((300, 20),), P.binding.OBF_FLAG_GENERIC_PATH)])
def test_out_of_prompt_softmax_mass(dtype, d, G, n_obs, caches, flags):
    w = small("lse", layers=2, kv_heads=2, G=G, n_obs=n_obs, d=d, dtype=dtype, rank=2, caches=caches, seed=71 + G)
    arrays = [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
    g = np.random.default_rng(17)
    params = par.params_for(w, flags=flags)
    dev, lses = [], []
    from scipy.special import logsumexp
    for ci, a in enumerate(arrays):
        # around each row's own log-sum-exp over the prompt: between "nearly nothing outside the prompt" and
        # "most of the mass outside it"; one row without any
        Kf = par.f32_view(a["K"], dtype).astype(np.float64)
        Qf = par.f32_view(a["Q"], dtype).astype(np.float64).reshape(w.layers, w.kv_heads, w.n_q, d)
        own = logsumexp(np.einsum("lhqd,lhtd->lhqt", Qf, Kf) / np.sqrt(d), axis=-1)
        le = (own + g.standard_normal(own.shape) * 3).astype(np.float32).reshape(w.layers, w.q_heads, w.n_obs)
        le[0, 0, 0] = -np.inf
        lses.append(le)
        dev.append({"K": par.to_device(a["K"], dtype), "V": par.to_device(a["V"], dtype), "Q": par.to_device(a["Q"], dtype),
                    "budget": w.caches[ci].budget, "lse_extra": torch.from_numpy(le).cuda()})
    outs = P.compress_caches(params, dev, want_scores=True)
    torch.cuda.synchronize()
    assert P.obf_last_device_status(outs[0]["workspace"]) & 0xFF == 0
    bits = np.int16 if dtype == "bf16" else np.int32
    reps = []
    for ci, a in enumerate(arrays):
        Qv = par.f32_view(a["Q"], dtype).reshape(w.layers, w.kv_heads, w.n_q, d)
        le = lses[ci].reshape(w.layers, w.kv_heads, w.n_q)
        diags = P.parse_diag(outs[ci]["diag"])
        for l, h in all_heads(w):
            K, V = par.f32_view(a["K"][l, h], dtype), par.f32_view(a["V"][l, h], dtype)
            ref = oracle.head(K, V, Qv[l, h], w.caches[ci].budget, w.rank, lse_extra=le[l, h])
            assert ref["A"].sum() < w.n_q * 0.999                   # the outside keys did take mass
            out = outs[ci]
            reps.append(par.check_head(
                dtype, K, V, Qv[l, h], w.caches[ci].budget, w.rank, out["idx"][l, h].cpu().numpy(),
                par.out_bits(out["K_out"][l, h]), par.out_bits(out["V_out"][l, h]), par.out_to_f32(out["V_out"][l, h]),
                out["scores"][l, h].cpu().numpy(), out["delta"][l, h].cpu().numpy(), diags[l * w.kv_heads + h],
                a["K"][l, h].view(bits), a["V"][l, h].view(bits), name="lse cache %d layer %d head %d" % (ci, l, h), ref=ref))
    print("\n[lse_extra] %s" % par.summarize(reps))


# ---------------------------------------------------------------------------
# Attn-inject (App. D.2): the back-fill shared out by attention mass
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,d,caches", [("f32", 64, ((200, 12), (90, 9))), ("bf16", 128, ((300, 20), (1024, 32)))])
def test_attn_inject_shares_the_backfill_by_attention_mass(dtype, d, caches):
    w = small("attn", layers=2, kv_heads=2, G=2, n_obs=6, d=d, dtype=dtype, rank=2, caches=caches, seed=97)
    arrays = [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
    outs, _, st = par.run_gpu(w, arrays, flags=P.binding.OBF_FLAG_ATTN_INJECT)
    assert st & 0xFF == 0
    plain, _, _ = par.run_gpu(w, arrays)
    checked = 0
    for ci, a in enumerate(arrays):
        o = outs[ci]
        # selection, keys and delta itself are those of the uniform injection
        assert torch.equal(o["idx"], plain[ci]["idx"]) and torch.equal(o["K_out"], plain[ci]["K_out"])
        assert torch.equal(o["delta"], plain[ci]["delta"])
        Qv = par.f32_view(a["Q"], dtype).reshape(w.layers, w.kv_heads, w.n_q, d)
        for l, h in all_heads(w):
            K, V = par.f32_view(a["K"][l, h], dtype), par.f32_view(a["V"][l, h], dtype)
            ref = oracle.head(K, V, Qv[l, h], w.caches[ci].budget, w.rank)
            idx = o["idx"][l, h].cpu().numpy()
            if not np.array_equal(idx, ref["idx"]) or ref["diag"]["skipped"]:
                continue
            dg = ref["diag"]
            gap = (dg["lam_rho"] - dg["lam_next"]) / dg["lam_1"]
            if gap < 1e-3:
                continue
            expect = oracle.attn_inject(V, ref["A"], idx, ref["delta"])
            share = len(idx) * ref["A"][idx] / (ref["A"][idx].sum() + 1e-12)
            dtol = max(2e-5 if dtype == "f32" else 2e-4, 200.0 * par.U32 / gap * dg["alpha"] * dg["rbar_norm"])
            # the tolerance on delta times the row's share (plus the share's own error: masses to 1e-5), and half a
            # bf16 ulp of the result on the bf16 path
            bound = share[:, None] * (dtol + 2e-5 * np.abs(ref["delta"])[None, :]) + 1e-6
            if dtype == "bf16":
                bound = bound + 2.0 ** -8 * 1.01 * np.abs(expect)
            err = np.abs(par.out_to_f32(o["V_out"][l, h]).astype(np.float64) - expect)
            assert np.all(err <= bound), "cache %d layer %d head %d: max err %.3g" % (ci, l, h, err.max())
            assert not np.allclose(share, 1.0)                      # the shares do differ from the uniform ones
            checked += 1
    assert checked >= 4


# ---------------------------------------------------------------------------
def test_early_out_skips_the_value_pass_of_full_heads_and_changes_nothing():
    # two caches: budget 200 >= head_dim (generic values: every head's retained values span R^d) and budget 40 < head_dim
    # (every head is back-filled).  With OBF_FLAG_EARLY_OUT the span test runs first and the pass over V skips the heads
    # of the first cache: every output must be the same bit for bit, and the back-filled heads must still be back-filled
    w = small("early", layers=2, kv_heads=2, G=4, n_obs=8, d=128, dtype="bf16", rank=2, caches=((1300, 200), (900, 40)),
              seed=53)
    arrays = [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
    plain, _, st0 = par.run_gpu(w, arrays)
    early, _, st1 = par.run_gpu(w, arrays, flags=P.binding.OBF_FLAG_EARLY_OUT)
    assert st0 & 0xFF == 0 and st1 & 0xFF == 0
    for a, b in zip(plain, early):
        for key in ("idx", "K_out", "V_out", "delta", "scores"):
            assert torch.equal(a[key], b[key]), key
    assert torch.all(early[0]["delta"] == 0) and torch.all(early[1]["delta"].norm(dim=-1) > 0)
    d0, d1 = P.parse_diag(early[0]["diag"]), P.parse_diag(early[1]["diag"])
    assert all(dg["span_rank"] == 128 for dg in d0) and all(dg["span_rank"] == 40 for dg in d1)


# cache-merging baseline (App. E): deleted values merged into the retained position with the most similar key
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,d,caches,flags", [
    ("f32", 64, ((200, 12), (90, 9), (70, 70)), 0),
    ("bf16", 128, ((300, 20), (1024, 32), (700, 150)), 0),
    ("bf16", 128, ((512, 28),), P.binding.OBF_FLAG_LAYERWISE)])
def test_cache_merging_baseline(dtype, d, caches, flags):
    w = small("merge", layers=2, kv_heads=2, G=2, n_obs=6, d=d, dtype=dtype, rank=2, caches=caches, seed=101)
    arrays = [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
    outs, _, st = par.run_gpu(w, arrays, flags=flags | P.binding.OBF_FLAG_MERGE, want_assign=True)
    assert st & 0xFF == 0
    ev, _, _ = par.run_gpu(w, arrays, evict=True, flags=flags)
    bits = np.int16 if dtype == "bf16" else np.int32
    near_ties = flips = 0
    for ci, a in enumerate(arrays):
        o = outs[ci]
        assert torch.equal(o["idx"], ev[ci]["idx"]) and torch.equal(o["K_out"], ev[ci]["K_out"])    # selection and keys: plain eviction
        assert torch.all(o["delta"] == 0)
        Qv = par.f32_view(a["Q"], dtype).reshape(w.layers, w.kv_heads, w.n_q, d)
        for l in range(w.layers):
            lay = None
            if flags & P.binding.OBF_FLAG_LAYERWISE:
                lay = oracle.layer(par.f32_view(a["K"][l], dtype), par.f32_view(a["V"][l], dtype), Qv[l], w.caches[ci].budget, 0)
            for h in range(w.kv_heads):
                K, V = par.f32_view(a["K"][l, h], dtype), par.f32_view(a["V"][l, h], dtype)
                ref = oracle.merge_head(K, V, Qv[l, h], w.caches[ci].budget)
                idx = o["idx"][l, h].cpu().numpy()
                g_assign = o["assign"][l, h].cpu().numpy()
                if lay is not None:
                    assert np.array_equal(idx, lay["idx"][h])
                elif not np.array_equal(idx, ref["idx"]):
                    continue                                        # a tie inside the selection band
                T = K.shape[0]
                keep = np.zeros(T, bool); keep[idx] = True
                assert np.all(g_assign[keep] == -1) and np.all((g_assign[~keep] >= 0) & (g_assign[~keep] < len(idx)))
                A = lay["A"][h] if lay is not None else ref["A"]
                if lay is None:
                    # routing: equal to the oracle's wherever the two best similarities are further apart than fp32
                    # can blur (1e-5); elsewhere the GPU's choice must be one of the near-best
                    clear = ref["margin"] > 1e-5
                    assert np.array_equal(g_assign[clear & ~keep], ref["assign"][clear & ~keep])
                    near_ties += int((~clear & ~keep).sum())
                    flips += int((g_assign != ref["assign"]).sum())
                    Kd = K.astype(np.float64); Kn = Kd / np.maximum(np.linalg.norm(Kd, axis=1, keepdims=True), 1e-300)
                    for j in np.flatnonzero(g_assign != ref["assign"]):
                        cs = Kn[idx] @ Kn[j]
                        assert cs[g_assign[j]] >= cs.max() - 1e-5
                # merged values: the oracle's step (iii) on the routing the GPU took
                expect = oracle.merge_given(V, A, idx, g_assign)
                absum = np.abs(V[idx].astype(np.float64))
                for j in np.flatnonzero(~keep):
                    absum[g_assign[j]] += A[j] / (A[idx[g_assign[j]]] + 1e-12) * np.abs(V[j].astype(np.float64))
                # fp32 accumulation of the weighted sum (weights carry the masses' 1e-5) and one rounding of the result
                bound = 4e-5 * absum + 1e-6
                if dtype == "bf16":
                    bound = bound + 2.0 ** -8 * 1.01 * np.abs(expect)
                err = np.abs(par.out_to_f32(o["V_out"][l, h]).astype(np.float64) - expect)
                assert np.all(err <= bound), "cache %d layer %d head %d: merged values off by %.3g" % (ci, l, h, err.max())
                assert np.array_equal(par.out_bits(o["K_out"][l, h]), a["K"][l, h].view(bits)[idx])
    print("\n[merge] near-tie routings %d, of which the GPU chose another near-best slot %d" % (near_ties, flips))


# ---------------------------------------------------------------------------
# int8 copy of the compacted relay (post-hoc quantisation stacked on the compression, App. E)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,d,caches,flags", [
    ("f32", 64, ((200, 12), (90, 90)), 0),
    ("bf16", 128, ((300, 20), (777, 140)), 0),
    ("bf16", 128, ((512, 28),), P.binding.OBF_FLAG_LAYERWISE)])
def test_int8_copy_of_the_relay(dtype, d, caches, flags):
    w = small("q8", layers=2, kv_heads=2, G=2, n_obs=6, d=d, dtype=dtype, rank=2, caches=caches, seed=83)
    arrays = [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
    outs, _, st = par.run_gpu(w, arrays, flags=flags, want_int8=True)
    assert st & 0xFF == 0
    plain, _, _ = par.run_gpu(w, arrays, flags=flags)
    injected = 0
    for ci, a in enumerate(arrays):
        o = outs[ci]
        # the usual outputs do not depend on the int8 copy being asked for
        for key in ("idx", "K_out", "V_out"):
            assert torch.equal(o[key], plain[ci][key]), key
        Kf, Vf = o["K_out"].float().cpu().numpy(), o["V_out"].float().cpu().numpy()
        for name, X in (("K", Kf), ("V", Vf)):
            codes, scales = oracle.quantize_rows(X)                     # the oracle's quantiser on the relay as it left
            assert np.array_equal(o[name + "_q8"].cpu().numpy(), codes), "%s codes differ" % name
            assert np.array_equal(o[name + "_scale"].cpu().numpy(), scales), "%s scales differ" % name
            back = codes.astype(np.float64) * scales.astype(np.float64)[..., None]
            # x / scale is rounded to fp32 before the rounding to a code: 127 * 2^-24 of a step on top of half a step
            assert np.all(np.abs(back - X) <= 0.5 * scales[..., None] * (1 + 2.0 ** -15))
        # the keys are exact copies of the inputs: their codes are those of the oracle's own gather
        idx = o["idx"].cpu().numpy()
        Kin = par.f32_view(a["K"], dtype)
        for l, h in all_heads(w):
            assert np.array_equal(o["K_q8"][l, h].cpu().numpy(), oracle.quantize_rows(Kin[l, h][idx[l, h]])[0])
        injected += int((o["delta"].abs().sum(dim=-1) > 0).sum())
    assert injected > 0                                                 # some values were quantised after an injection


def test_sink_prefix_longer_than_the_prompt_keeps_everything():
    w = small("sink_all", d=64, dtype="f32", rank=1, caches=((6, 3),), heavy=0)
    arrays = [synth.gen_cache(w, 0)]
    outs, _, st = par.run_gpu(w, arrays, flags=P.binding.OBF_FLAG_SINK(10))
    assert st & 0xFF == 0
    assert outs[0]["idx"].shape[-1] == 6
    assert torch.equal(outs[0]["idx"][0, 0].cpu(), torch.arange(6, dtype=torch.int32))


# ---------------------------------------------------------------------------
# fixed three-iteration Gram subspace path (an approximation: compared with the oracle's same iteration)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,d,rank,caches", [("f32", 64, 2, ((200, 12), (90, 9))), ("f32", 128, 4, ((300, 20),)),
                                                 ("bf16", 128, 4, ((1024, 32), (300, 20))), ("f32", 64, 8, ((150, 10),))])
def test_fast_path_matches_the_oracles_same_iteration(dtype, d, rank, caches):
    w = small("fast", layers=2, kv_heads=2, G=2, n_obs=6, d=d, dtype=dtype, rank=rank, caches=caches, seed=61)
    arrays = [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
    outs, _, st = par.run_gpu(w, arrays, flags=P.binding.OBF_FLAG_FAST_PATH)
    assert st & 0xFF == 0
    worst = 0.0
    for ci in range(len(w.caches)):
        a, out = arrays[ci], outs[ci]
        Qv = a["Q"].reshape(w.layers, w.kv_heads, w.n_q, d)
        diags = P.parse_diag(out["diag"])
        for l in range(w.layers):
            for h in range(w.kv_heads):
                K, V, Q = par.f32_view(a["K"][l, h], dtype), par.f32_view(a["V"][l, h], dtype), par.f32_view(Qv[l, h], dtype)
                ref = oracle.head(K, V, Q, w.caches[ci].budget, rank, fast_iters=3)
                g_idx = out["idx"][l, h].cpu().numpy()
                if not np.array_equal(g_idx, ref["idx"]):
                    continue                                        # a tie inside the band: another valid retained set
                gd = out["delta"][l, h].cpu().numpy().astype(np.float64)
                scale = ref["diag"]["alpha"] * ref["diag"]["rbar_norm"]
                err = np.linalg.norm(gd - ref["delta"])
                worst = max(worst, err / scale)
                # three multiplications by an fp32 Gram matrix whose eigenvalues are within a small factor of each
                # other: the error stays near fp32 rounding (measured: 4e-7 of the scale)
                assert err <= 1e-4 * scale + 1e-6, "delta off by %.3g (scale %.3g)" % (err, scale)
                Vk = V[g_idx].astype(np.float64)
                assert np.abs(Vk @ gd).max() <= 1e-4 * np.linalg.norm(Vk, 2) * np.linalg.norm(gd)
                assert np.linalg.norm(gd) <= scale * (1 + 1e-3)
                dg = diags[l * w.kv_heads + h]
                assert dg["rho_eff"] == ref["diag"]["rho_eff"]
                assert abs(dg["revr"] - ref["diag"]["revr"]) <= 1e-3
                gv = par.out_to_f32(out["V_out"][l, h]).astype(np.float64)
                tol = (2e-3 * scale + 1e-4) if dtype == "f32" else (2e-2 * np.abs(ref["V_out"]) + 2e-3 * scale + 1e-3)
                assert np.all(np.abs(gv - ref["V_out"]) <= tol)
    print("\n[fast path] worst relative delta error %.3g" % worst)
