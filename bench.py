#!/usr/bin/env python
"""Benchmark of the relay-boundary prompt-KV compression path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl ours|reference]

One step = one pass of the whole hot path (score, select, gather, OBF) over one
batch of seeded synthetic caches.  Metric: prompt-KV GB/s compressed, i.e. the
algorithmic bytes (K, V and queries read once; compacted K, V and the index list
written once) over the device time of the step.  With N > 1 every rank runs an
independent replica of the workload on its own GPU (the path has no exchange
step) and the aggregate is reported.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "prompt_kv_gbs_compressed"
UNIT = "GB/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        return float(pk["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        inside = [r for t, r in self.rows if t0 - 0.05 <= t <= t1 + 0.15] or [r for _, r in self.rows]
        sm, mx, reasons = [], [], set()
        for r in inside:
            p = [x.strip() for x in r.split(",")]
            if len(p) < 7:
                continue
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def cpu_baseline(w, arrays0, seconds_target: float = 15.0):
    """The oracle as it stands, on the host cores, on a bounded sample of layers of cache 0."""
    import oracle
    from paper_2604_13349_b200 import synth
    K, V, Q = arrays0["K"], arrays0["V"], arrays0["Q"]
    conv = (lambda a: synth.bf16_bits_to_f32(a)) if w.dtype == "bf16" else (lambda a: a)
    T = w.caches[0].T
    per_layer_bytes = w.kv_heads * (2 * T * w.head.head_dim * w.elem_bytes + w.n_q * w.head.head_dim * w.elem_bytes
                                    + 2 * min(w.caches[0].budget, T) * w.head.head_dim * w.elem_bytes
                                    + 4 * min(w.caches[0].budget, T))
    layers_done, t_total = 0, 0.0
    while layers_done < w.layers and (layers_done == 0 or t_total * (layers_done + 1) / layers_done < seconds_target):
        l = layers_done
        k, v, q = conv(K[l:l + 1]), conv(V[l:l + 1]), conv(Q[l:l + 1])
        t0 = time.perf_counter()
        oracle.compress(k, v, q, w.q_heads, w.n_obs, w.caches[0].budget, w.rank, layerwise=w.layerwise)
        t_total += time.perf_counter() - t0
        layers_done += 1
    gbs = per_layer_bytes * layers_done / t_total / 1e9
    return {"value": gbs, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "layers 0..%d of cache 0 of %s (%d of %d heads), %.1f s" % (
                layers_done - 1, w.name, layers_done * w.kv_heads, w.layers * w.kv_heads * len(w.caches), t_total),
            "seconds": t_total, "layers": layers_done}


def run_reference(args):
    """--impl reference: the CPU oracle timed on bounded samples of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2604_13349_b200 import synth
    import oracle
    w = synth.workload(args.workload)
    # one step = layer 0 of cache 0 (kv_heads heads)
    arrays0 = {k: v[:1] for k, v in synth.gen_cache(
        __import__("dataclasses").replace(w, layers=1), 0).items()}
    conv = (lambda a: synth.bf16_bits_to_f32(a)) if w.dtype == "bf16" else (lambda a: a)
    k, v, q = conv(arrays0["K"]), conv(arrays0["V"]), conv(arrays0["Q"])
    T = w.caches[0].T
    ke = min(w.caches[0].budget, T)
    step_bytes = w.kv_heads * (2 * T * w.head.head_dim * w.elem_bytes + w.n_q * w.head.head_dim * w.elem_bytes
                               + 2 * ke * w.head.head_dim * w.elem_bytes + 4 * ke)
    for _ in range(args.warmup):
        oracle.compress(k, v, q, w.q_heads, w.n_obs, w.caches[0].budget, w.rank, layerwise=w.layerwise)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.compress(k, v, q, w.q_heads, w.n_obs, w.caches[0].budget, w.rank, layerwise=w.layerwise)
    dt = time.perf_counter() - t0
    val = step_bytes * args.steps / dt / 1e9
    sample = "each step = layer 0 of cache 0 of %s (%d heads, T=%d)" % (w.name, w.kv_heads, T)
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import paper_2604_13349_b200 as P
    from paper_2604_13349_b200 import dist, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init("nccl")
    P.load()

    w = synth.workload(args.workload)
    params = P.make_params(w.layers, w.kv_heads, w.q_heads, w.head.head_dim, w.n_obs, w.rank,
                           P.OBF_F32 if w.dtype == "f32" else P.OBF_BF16, 1e-12,
                           (P.binding.OBF_FLAG_LAYERWISE if w.layerwise else 0)
                           | (P.binding.OBF_FLAG_FAST_PATH if w.fast_path else 0))
    tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16

    def as_t(a):
        t = torch.from_numpy(a.view(np.int16) if w.dtype == "bf16" else a)
        return t.view(torch.bfloat16) if w.dtype == "bf16" else t

    host_arrays = [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
    dev_in, caches, outs = [], [], []
    for ci, a in enumerate(host_arrays):
        K, V, Q = as_t(a["K"]).cuda(), as_t(a["V"]).cuda(), as_t(a["Q"]).cuda()
        T, budget = w.caches[ci].T, w.caches[ci].budget
        ke = min(budget, T)
        o = {"K_out": torch.empty((w.layers, w.kv_heads, ke, w.head.head_dim), dtype=tdt, device="cuda"),
             "V_out": torch.empty((w.layers, w.kv_heads, ke, w.head.head_dim), dtype=tdt, device="cuda"),
             "idx": torch.empty((w.layers, w.kv_heads, ke), dtype=torch.int32, device="cuda")}
        dev_in.append((K, V, Q)); outs.append(o)
        caches.append(P.make_cache(K, V, Q, T, budget, o["K_out"], o["V_out"], o["idx"]))
    ws = torch.empty(P.obf_workspace_bytes(params, caches), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    step_bytes = w.algorithmic_bytes()

    for _ in range(args.warmup):
        P.obf_compress(params, caches, ws, stream=stream)
    launches_per_step = P.obf_last_launch_count()
    torch.cuda.synchronize()
    status = P.obf_last_device_status(ws)
    if status & 0xFF:
        raise SystemExit("device status %#x after warm-up" % status)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    e0.record(stream)
    for _ in range(args.steps):
        P.obf_compress(params, caches, ws, stream=stream)
    e1.record(stream)
    torch.cuda.synchronize()
    t_wall1 = time.time()
    dist.barrier()
    ms_total = dist.max_over_ranks(e0.elapsed_time(e1))
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    ms_per_step = ms_total / args.steps
    total_bytes = dist.sum_over_ranks(float(step_bytes))
    value = total_bytes / (ms_per_step * 1e-3) / 1e9
    tokens_per_s = dist.sum_over_ranks(float(w.tokens())) / (ms_per_step * 1e-3)

    # per-kernel device times of one step (events between launches, on the same stream)
    phase_acc = {}
    n_prof = 5
    for _ in range(n_prof):
        for name, ms in P.obf_compress_profiled(params, caches, ws, stream=stream):
            phase_acc[name] = phase_acc.get(name, 0.0) + ms / n_prof
    dom = max(phase_acc, key=phase_acc.get)
    peak, peak_kind = load_peaks()
    # algorithmic bytes of the dominant kernel's launch: what that step of the path must move
    e = w.elem_bytes
    d = w.head.head_dim
    hpc = w.layers * w.kv_heads
    kv_bytes = sum(hpc * c.T * d * e for c in w.caches)
    q_bytes = len(w.caches) * hpc * w.n_q * d * e
    out_bytes = sum(hpc * min(c.budget, c.T) * (2 * d * e + 4) for c in w.caches)
    score_bytes = sum(hpc * c.T * 4 for c in w.caches)                 # the mass array A (fp32)
    kernel_bytes = {"k_score_stats": kv_bytes + q_bytes, "k_score_pool": kv_bytes + q_bytes + score_bytes,
                    "k_score_tc": kv_bytes + q_bytes + score_bytes,     # K and Q read once, A written
                    "k_gram": kv_bytes, "k_gram_tc": kv_bytes,          # V read once
                    "k_gather": 2 * out_bytes, "k_select": score_bytes,
                    "k_span_test": 0, "k_obf_algebra": 0}.get(dom, step_bytes)
    achieved = kernel_bytes / (phase_acc[dom] * 1e-3) / 1e9
    traffic = None
    # dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the ncu summaries ("kernel workload bytes")
    tpath = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if os.path.exists(tpath):
        with open(tpath) as f:
            for ln in f:
                parts = ln.split("#")[0].split()
                if len(parts) == 3 and parts[0] == dom and parts[1] == w.name:
                    traffic = int(parts[2])
    # the attention-mass kernel evaluates 2 exponentials per (query, key): its own ceiling is the
    # special-function unit (16 results per clock and SM), not HBM
    n_exp = 2.0 * sum(hpc * c.T * w.n_q for c in w.caches)
    sm_clock = (clocks or {}).get("sm_mhz") or 1965.0
    sfu_peak = 16 * 148 * sm_clock * 1e6 / 1e9
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": peak_kind, "traffic": traffic,
                "kernel_ms": phase_acc[dom], "algorithmic_bytes_per_launch": kernel_bytes,
                "whole_step_frac": (step_bytes / (ms_per_step * 1e-3) / 1e9) / peak,
                "phases_ms": {k: round(v, 4) for k, v in phase_acc.items()}}
    if dom == "k_score_tc":
        roofline["sfu"] = {"unit": "Gexp/s", "achieved": n_exp / (phase_acc[dom] * 1e-3) / 1e9, "peak": sfu_peak,
                           "frac": n_exp / (phase_acc[dom] * 1e-3) / 1e9 / sfu_peak}

    # end to end through the host entry point: pinned host buffers, copies inside the timed region
    e2e = None
    if args.e2e_steps > 0:
        h_caches, keepalive = [], []
        for ci, a in enumerate(host_arrays):
            hk, hv, hq = as_t(a["K"]).pin_memory(), as_t(a["V"]).pin_memory(), as_t(a["Q"]).pin_memory()
            T, budget = w.caches[ci].T, w.caches[ci].budget
            ke = min(budget, T)
            ok = torch.empty((w.layers, w.kv_heads, ke, d), dtype=tdt).pin_memory()
            ov = torch.empty((w.layers, w.kv_heads, ke, d), dtype=tdt).pin_memory()
            oi = torch.empty((w.layers, w.kv_heads, ke), dtype=torch.int32).pin_memory()
            keepalive += [hk, hv, hq, ok, ov, oi]
            h_caches.append(P.make_cache(hk, hv, hq, T, budget, ok, ov, oi))
        arena = torch.empty(P.obf_host_arena_bytes(params, h_caches), dtype=torch.uint8, device="cuda")
        P.obf_compress_host(params, h_caches, arena, stream=stream)
        dist.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            P.obf_compress_host(params, h_caches, arena, stream=stream)   # waits for the stream itself
        torch.cuda.synchronize()
        dt = dist.max_over_ranks((time.perf_counter() - t0) * 1e3) / args.e2e_steps
        e2e = {"value": total_bytes / (dt * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": 2 * kv_bytes + q_bytes, "d2h_bytes_per_step": out_bytes,
               "ms_per_step": dt, "steps": args.e2e_steps}
        # the device-resident outputs and the host-path outputs must agree bit for bit
        for o, hc_out in zip(outs, range(0, len(keepalive), 6)):
            assert torch.equal(o["idx"].cpu(), keepalive[hc_out + 5]), "host path indices differ"
        del arena

    cpu = None
    if rank == 0 and not args.no_cpu_baseline:
        cpu = cpu_baseline(w, host_arrays[0])

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": w.name, "layers": w.layers, "kv_heads": w.kv_heads, "q_heads": w.q_heads,
                       "head_dim": d, "n_obs": w.n_obs, "rank": w.rank, "selector": "layerwise" if w.layerwise else "headwise",
                       "T": [c.T for c in w.caches], "budget": [c.budget for c in w.caches],
                       "l2": "inputs_larger_than_l2" if 2 * kv_bytes > 126e6 else "inputs_fit_l2",
                       "parallelism": "replicas" if world > 1 else "single_gpu"},
            "relay_tokens_per_s": tokens_per_s,
            "algorithmic_bytes_per_step": step_bytes,
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
        }
        print(json.dumps(line))
    dist.finish()
    return 0


if __name__ == "__main__":
    sys.exit(main())
