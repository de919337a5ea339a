#!/usr/bin/env python
"""Benchmark of the relay-boundary prompt-KV compression path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl ours|reference]

One step = one pass of the whole hot path (score, select, gather, OBF) over one
batch of seeded synthetic caches.  Metric: prompt-KV GB/s compressed, i.e. the
algorithmic bytes (K, V and queries read once; compacted K, V and the index list
written once) over the device time of the step.  With N > 1 every rank runs an
independent replica of the workload on its own GPU (the path has no exchange
step) and the aggregate is reported.  Prints ONE JSON line on rank 0.

Timing: a batch is exactly --steps calls between two CUDA events on the launching stream, bracketed by a
barrier and a device synchronisation, max over ranks.  Batches are repeated until at least MIN_TIMED_S seconds
of device time have been measured; `ms_per_step` is the median batch, `best_ms_per_step` the fastest one, and
the SM clock is sampled all the while (`clocks`), so that `ms_per_step_x_sm_ghz` (time x median clock = kilo-cycles
per step) can be compared between runs made at different clocks.
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
MIN_TIMED_S = 2.0          # device time measured per workload (the bench workload; 0.5 s for the side workloads)
MAX_BATCHES = 400


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
        inside = [r for t, r in self.rows if t0 <= t <= t1 + 0.1]
        outside_only = not inside
        if outside_only:
            inside = [r for _, r in self.rows]
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
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons), "samples": len(sm),
                "samples_outside_timed_region": outside_only}


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


# fp32 work of the dense algebra per (layer, KV head) whose retained values do not span R^d, as the kernel
# formulates it (Eq. 2-6): twice-iterated Gram-Schmidt over the k retained rows, P = I - Q^T Q, the two products of
# M = P G P, the Householder reduction of M to tridiagonal form and the way back for rank + 1 vectors.
def algebra_flops(d: int, k: int, rank: int) -> float:
    m = min(k, d)
    gram_schmidt = 2 * 2 * (2.0 * d) * sum(min(i, d) for i in range(k))     # two passes of dot + update against i rows
    projector = 2.0 * m * d * d
    products = 2 * 2.0 * d ** 3
    tridiagonal = 4.0 / 3.0 * d ** 3 * 2                                     # both triangles are updated
    back = (rank + 1) * 2 * 2.0 * d * d
    return gram_schmidt + projector + products + tridiagonal + back


# The source files a kernel's DRAM traffic depends on: its own file, what it includes, and the host file that sizes
# its grid and workspace.
KERNEL_SOURCES = {
    "k_score_tc": ("score_tc.cuh", "tc_common.cuh", "common.cuh", "obf_api.cu"),
    "k_gram_tc": ("gram_tc.cuh", "tc_common.cuh", "common.cuh", "obf_api.cu"),
}


def kernel_source_stamp(kernel: str = "") -> str:
    """Hash of the CUDA sources a kernel is made of (all of them for a kernel that is not listed): an ncu traffic
    figure is only quoted for the sources it was captured on."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2604_13349_b200", "csrc")
    files = KERNEL_SOURCES.get(kernel) or sorted(f for f in os.listdir(csrc) if f.endswith((".cu", ".cuh")))
    for f in files:
        with open(os.path.join(csrc, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:12]


def measured_traffic(kernel: str, workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch, from profiles/dram_traffic.txt
    ("kernel workload bytes stamp"); None when the kernel's sources have changed since the capture."""
    tpath = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(tpath):
        return None
    stamp = kernel_source_stamp(kernel)
    with open(tpath) as f:
        for ln in f:
            parts = ln.split("#")[0].split()
            if len(parts) == 4 and parts[0] == kernel and parts[1] == workload and parts[3] == stamp:
                return int(parts[2])
    return None


class Bench:
    """One workload resident on the device: inputs, outputs, workspace, and the timed loops over it."""

    def __init__(self, name: str):
        import torch
        import paper_2604_13349_b200 as P
        from paper_2604_13349_b200 import synth
        self.torch, self.P = torch, P
        w = self.w = synth.workload(name)
        self.params = P.make_params(w.layers, w.kv_heads, w.q_heads, w.head.head_dim, w.n_obs, w.rank,
                                    P.OBF_F32 if w.dtype == "f32" else P.OBF_BF16, 1e-12,
                                    (P.binding.OBF_FLAG_LAYERWISE if w.layerwise else 0)
                                    | (P.binding.OBF_FLAG_FAST_PATH if w.fast_path else 0)
                                    | (P.binding.OBF_FLAG_MERGE if w.merge else 0)
                                    | (P.binding.OBF_FLAG_EARLY_OUT if w.early_out else 0))
        self.tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16
        self.host_arrays = [synth.gen_cache(w, ci) for ci in range(len(w.caches))]
        self.dev_in, self.caches, self.outs = [], [], []
        for ci, a in enumerate(self.host_arrays):
            K, V, Q = self.as_t(a["K"]).cuda(), self.as_t(a["V"]).cuda(), self.as_t(a["Q"]).cuda()
            T, budget = w.caches[ci].T, w.caches[ci].budget
            ke = min(budget, T)
            o = {"K_out": torch.empty((w.layers, w.kv_heads, ke, w.head.head_dim), dtype=self.tdt, device="cuda"),
                 "V_out": torch.empty((w.layers, w.kv_heads, ke, w.head.head_dim), dtype=self.tdt, device="cuda"),
                 "idx": torch.empty((w.layers, w.kv_heads, ke), dtype=torch.int32, device="cuda")}
            q8 = None
            if w.int8_out:
                o["K_q8"] = torch.empty((w.layers, w.kv_heads, ke, w.head.head_dim), dtype=torch.int8, device="cuda")
                o["V_q8"] = torch.empty_like(o["K_q8"])
                o["K_scale"] = torch.empty((w.layers, w.kv_heads, ke), dtype=torch.float32, device="cuda")
                o["V_scale"] = torch.empty_like(o["K_scale"])
                q8 = (o["K_q8"], o["V_q8"], o["K_scale"], o["V_scale"])
            self.dev_in.append((K, V, Q)); self.outs.append(o)
            self.caches.append(P.make_cache(K, V, Q, T, budget, o["K_out"], o["V_out"], o["idx"], q8=q8))
        self.ws = torch.empty(P.obf_workspace_bytes(self.params, self.caches), dtype=torch.uint8, device="cuda")
        self.stream = torch.cuda.current_stream()
        e, d, hpc = w.elem_bytes, w.head.head_dim, w.layers * w.kv_heads
        self.kv_bytes = sum(hpc * c.T * d * e for c in w.caches)
        self.q_bytes = len(w.caches) * hpc * w.n_q * d * e
        self.out_bytes = sum(hpc * min(c.budget, c.T) * (2 * d * e + 4) for c in w.caches)
        self.score_bytes = sum(hpc * c.T * 4 for c in w.caches)            # the mass array A (fp32)

    def as_t(self, a):
        t = self.torch.from_numpy(a.view(np.int16) if self.w.dtype == "bf16" else a)
        return t.view(self.torch.bfloat16) if self.w.dtype == "bf16" else t

    def step(self):
        self.P.obf_compress(self.params, self.caches, self.ws, stream=self.stream)

    def warm(self, n: int) -> int:
        for _ in range(n):
            self.step()
        launches = self.P.obf_last_launch_count()
        self.torch.cuda.synchronize()
        status = self.P.obf_last_device_status(self.ws)
        if status & 0xFF:
            raise SystemExit("device status %#x after warm-up" % status)
        return launches

    def time_batches(self, steps: int, min_seconds: float, dist):
        """Batches of exactly `steps` calls, each between two events on the launching stream and bracketed by a
        barrier and a synchronisation (max over ranks), until min_seconds of device time are measured.
        Returns the per-step times of the batches in ms."""
        torch = self.torch
        per_step, total_ms = [], 0.0
        while (total_ms < min_seconds * 1e3 or len(per_step) < 5) and len(per_step) < MAX_BATCHES:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            dist.barrier()
            torch.cuda.synchronize()
            e0.record(self.stream)
            for _ in range(steps):
                self.step()
            e1.record(self.stream)
            torch.cuda.synchronize()
            dist.barrier()
            ms = dist.max_over_ranks(e0.elapsed_time(e1))
            per_step.append(ms / steps)
            total_ms += ms
        return per_step

    def phases(self, n_prof: int = 5):
        """Per-kernel device times of one step (events between launches, on the same stream)."""
        acc = {}
        for _ in range(n_prof):
            for name, ms in self.P.obf_compress_profiled(self.params, self.caches, self.ws, stream=self.stream):
                acc[name] = acc.get(name, 0.0) + ms / n_prof
        return acc

    def roofline(self, phase_acc, ms_per_step: float, sm_mhz):
        """Roofline of the dominant kernel: HBM for the streaming kernels, the fp32 pipes for the dense algebra."""
        w = self.w
        dom = max(phase_acc, key=phase_acc.get)
        peak, peak_kind = load_peaks()
        step_bytes = w.algorithmic_bytes()
        kv, q, sc, ob = self.kv_bytes, self.q_bytes, self.score_bytes, self.out_bytes
        # algorithmic bytes of a launch: what that step of the path must move
        kernel_bytes = {"k_score_stats": kv + q, "k_score_pool": kv + q + sc,
                        "k_score_tc": kv + q + sc,                          # K and Q read once, A written
                        "k_gram": kv, "k_gram_tc": kv + sc,                 # V and A read once
                        "k_gather": 2 * ob, "k_select": sc}.get(dom)
        common = {"kernel": dom, "kernel_ms": phase_acc[dom],
                  "whole_step_frac": (step_bytes / (ms_per_step * 1e-3) / 1e9) / peak,
                  "whole_step_peak": peak, "whole_step_peak_kind": peak_kind,
                  "phases_ms": {k: round(v, 4) for k, v in phase_acc.items()}}
        if kernel_bytes is None:
            # the dense algebra (and the span test): no HBM traffic to speak of, fp32 arithmetic in shared memory.
            # Peak: 148 SMs x 128 FMA lanes x 2 flop x SM clock.
            hpc = w.layers * w.kv_heads
            if dom.startswith("k_merge"):
                # cache-merging baseline: the similarities of every position with every retained key
                flops = sum(hpc * 2.0 * c.T * min(c.budget, c.T) * w.head.head_dim for c in w.caches)
            else:
                flops = sum(hpc * algebra_flops(w.head.head_dim, min(c.budget, c.T), w.rank)
                            for c in w.caches if min(c.budget, c.T) < w.head.head_dim)
            clock = sm_mhz or 1965.0
            alu_peak = 148 * 128 * 2 * clock * 1e6 / 1e12
            ach = flops / (phase_acc[dom] * 1e-3) / 1e12
            return dict(common, bound="alu", achieved=ach, peak=alu_peak, unit="TFLOP/s", frac=ach / alu_peak,
                        peak_kind="derived: 148 SMs x 128 fp32 FMA lanes x 2 x %.0f MHz" % clock, traffic=None,
                        algorithmic_flops_per_launch=flops)
        achieved = kernel_bytes / (phase_acc[dom] * 1e-3) / 1e9
        r = dict(common, bound="hbm", achieved=achieved, peak=peak, unit="GB/s", frac=achieved / peak,
                 peak_kind=peak_kind, traffic=measured_traffic(dom, w.name), algorithmic_bytes_per_launch=kernel_bytes)
        if dom == "k_score_tc":
            # the attention-mass kernel evaluates 2 exponentials per (query, key): a second ceiling beside HBM is
            # the special-function unit (16 results per clock and SM)
            n_exp = 2.0 * sum(w.layers * w.kv_heads * c.T * w.n_q for c in w.caches)
            sfu_peak = 16 * 148 * (sm_mhz or 1965.0) * 1e6 / 1e9
            r["sfu"] = {"unit": "Gexp/s", "achieved": n_exp / (phase_acc[dom] * 1e-3) / 1e9, "peak": sfu_peak,
                        "frac": n_exp / (phase_acc[dom] * 1e-3) / 1e9 / sfu_peak}
        return r


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_S,
                    help="device time to measure before stopping (at least 5 batches are always timed)")
    ap.add_argument("--also", default="c4_evict,c4_early,pa", help="workloads reported beside the bench workload at 1 GPU ('none' for none)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import paper_2604_13349_b200 as P
    from paper_2604_13349_b200 import dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init("nccl")
    P.load()

    b = Bench(args.workload)
    w = b.w
    d = w.head.head_dim
    step_bytes = w.algorithmic_bytes()
    launches_per_step = b.warm(args.warmup)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    t_wall0 = time.time()
    per_step = b.time_batches(args.steps, args.min_seconds, dist)
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    ms_per_step = statistics.median(per_step)
    total_bytes = dist.sum_over_ranks(float(step_bytes))
    value = total_bytes / (ms_per_step * 1e-3) / 1e9
    tokens_per_s = dist.sum_over_ranks(float(w.tokens())) / (ms_per_step * 1e-3)

    phase_acc = b.phases()
    sm_mhz = (clocks or {}).get("sm_mhz")
    roofline = b.roofline(phase_acc, ms_per_step, sm_mhz)
    kv_bytes, q_bytes, out_bytes = b.kv_bytes, b.q_bytes, b.out_bytes
    host_arrays, outs, params, tdt, stream = b.host_arrays, b.outs, b.params, b.tdt, b.stream
    as_t = b.as_t

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

    # Beside the bench workload: the same shapes in eviction-only mode (isolates the cost of OBF), the same call with
    # the span test first (OBF_FLAG_EARLY_OUT: the pass over V then skips the heads whose retained values span R^d,
    # which is every head of c2-c5; its GB/s still count |V| as read, so that the figures of the two modes compare),
    # and the paper's own regime (budget 32 < head_dim, where the back-fill is not zero and the dense algebra runs
    # for every head).  1 GPU only.
    others = {}
    if world == 1 and args.also:
        del b
        torch.cuda.empty_cache()
        for name in [n for n in args.also.split(",") if n and n != "none" and n != w.name]:
            ob = Bench(name)
            ob.warm(args.warmup)
            ps = ob.time_batches(args.steps, min(0.5, args.min_seconds), dist)
            ms = statistics.median(ps)
            others[name] = {"ms_per_step": ms, "best_ms_per_step": min(ps), "batches": len(ps),
                            "value": ob.w.algorithmic_bytes() / (ms * 1e-3) / 1e9, "unit": UNIT,
                            "relay_tokens_per_s": ob.w.tokens() / (ms * 1e-3),
                            "roofline": ob.roofline(ob.phases(), ms, sm_mhz)}
            if ob.w.early_out:
                others[name]["bytes_counted"] = "as for the bench workload (|V| included although skipped heads' values are not read)"

            del ob
            torch.cuda.empty_cache()

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "best_ms_per_step": min(per_step),
            "batches": len(per_step), "timed_region_s": sum(per_step) * args.steps * 1e-3,
            "ms_per_step_x_sm_ghz": ms_per_step * sm_mhz * 1e-3 if sm_mhz else None,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": w.name, "layers": w.layers, "kv_heads": w.kv_heads, "q_heads": w.q_heads,
                       "head_dim": d, "n_obs": w.n_obs, "rank": w.rank, "selector": "layerwise" if w.layerwise else "headwise",
                       "T": [c.T for c in w.caches], "budget": [c.budget for c in w.caches],
                       "l2": "inputs_larger_than_l2" if 2 * kv_bytes > 126e6 else "inputs_fit_l2",
                       "parallelism": "replicas" if world > 1 else "single_gpu"},
            "relay_tokens_per_s": tokens_per_s,
            "algorithmic_bytes_per_step": step_bytes,
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps * len(per_step), "gpu_launches_per_step": launches_per_step,
            "clocks": clocks, "other_workloads": others,
        }
        print(json.dumps(line))
    dist.finish()
    return 0


if __name__ == "__main__":
    sys.exit(main())
