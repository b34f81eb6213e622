#!/usr/bin/env python
"""Benchmark of the leapfrog backward pass (arXiv 1801.04928) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--config 1..4] [--variant auto|streams|persistent|fused] [--k K]

A step is one whole backward pass (Eq. bp1, the Eq. bp2 chain, Eq. bp3/bp4 of every layer
under the leapfrog schedule) over one batch of synthetic inputs that are already resident in
device memory.  The metric is backward layers per second (L / step time), reported with the
achieved algorithmic HBM bandwidth of the dominant kernel against the measured copy peak.

The headline workload is the largest single-sample one (configs[2]: L = 64, N = 4096).  The same
JSON line carries, under "per_config", the other named workloads measured in the same run, each
with its own step time, roofline fraction and clock sample: configs[0] (latency-bound), configs[1]
(the width at which the delta hand-off, not bandwidth, is the bound) and configs[3] (mini-batch:
the whole step and the tensor-core weight-gradient contraction alone, next to a same-run TF32
contraction of the library's own at N = 8192, B = 1024).

With N > 1 GPUs every rank runs an independent replica of the workload (the path does not
shard: the delta chain is sequential in depth), so the aggregate is N times the per-GPU rate.

One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "backward_layers_per_sec"
UNIT = "layers/s"
HBM_FALLBACK_GBS = 6650.0  # used only if MEASURED_PEAKS.json is absent
BF16_FALLBACK_TFLOPS = 1590.0
VARIANT_NAMES = {"auto": 0, "streams": 1, "persistent": 2, "fused": 3}
TC_TILING_NAMES = {"auto": 0, "one_sm": 1, "two_sm": 2}
FUSED_TILING_NAMES = {"auto": 0, "clusters": 1, "columns": 2}
CSRC = os.path.join(ROOT, "paper_1801_04928_b200", "csrc")


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=200)
    p.add_argument("--warmup", type=int, default=5)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--config", type=int, default=3)
    p.add_argument("--variant", default="auto", choices=sorted(VARIANT_NAMES))
    p.add_argument("--fused-tiling", default="auto", choices=sorted(FUSED_TILING_NAMES),
                   help="tiling of the fused single-launch pass (B = 1)")
    p.add_argument("--k", type=int, default=0, help="leapfrog workers (0 = the config's k)")
    p.add_argument("--tc-tiling", default="auto", choices=["auto", "one_sm", "two_sm"],
                   help="tiling of the tensor-core contractions (B > 1)")
    p.add_argument("--sgd", type=float, default=None, metavar="ETA",
                   help="time lf_backward_sgd (gradient + weight update in one pass) with this step size "
                        "instead of lf_backward; not the headline metric")
    p.add_argument("--layers", type=int, default=0,
                   help="override the config's L (a smaller case of the same kernels, for profiler captures)")
    p.add_argument("--shards", type=int, default=1, metavar="S",
                   help="time ONE shard (rank 0) of the layer-sharded form on S GPUs: the whole delta chain, "
                        "weight gradients of every S-th layer only; nothing is exchanged, so this is the time "
                        "each of the S GPUs would take")
    p.add_argument("--shard-by-rank", action="store_true",
                   help="with --gpus N > 1: instead of N replicas, run ONE pass layer-sharded over the N ranks "
                        "(rank r = shard r of N, no exchange); value = L / slowest rank's time, strong scaling")
    p.add_argument("--e2e-steps", type=int, default=3)
    p.add_argument("--cpu-seconds", type=float, default=10.0)
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-e2e", action="store_true")
    p.add_argument("--no-per-config", action="store_true",
                   help="skip the other named workloads (the per_config array)")
    return p.parse_args()


def algorithmic_bytes(L, N, B):
    """Bytes one backward pass must move: w^2..w^L read once, gw^1..gw^L written once, plus
    the z/a/delta operand vectors (3 * 4NB per layer)."""
    return 4 * N * N * (2 * L - 1) + 3 * 4 * N * B * L


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                d = json.load(f)
            return float(d["hbm_gbs"]), "measured", d
        except Exception:
            pass
    return HBM_FALLBACK_GBS, "fallback", {}


def shard_plan(world, rank, k, shards, by_rank):
    """Which shard of the layer-sharded form a process runs and with how many leapfrog workers.

    Returns (S, r, k_here): the pass is cut into S shards (layer l belongs to shard (L - l) mod S),
    this process is shard r, and the workload's k workers are spread over the S shards (at least
    one each).  Replicas (no sharding) give (1, 0, k)."""
    if by_rank and world > 1:
        return world, rank, max(1, k // world)
    if shards > 1:
        return shards, 0, max(1, k // shards)
    return 1, 0, k


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [c.strip() for c in r.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def time_oracle(cfg, tensors_cpu, seconds):
    """Times the oracle's backward pass (Algorithm 1 taken literally with k threads, every
    thread recomputing the delta chain) on the host, as it stands.  `tensors_cpu` holds w and b
    for at least the layers of the sample."""
    import numpy as np
    from oracle import lf_oracle as orc
    w = tensors_cpu["w"].numpy(); b = tensors_cpu["b"].numpy()
    x = tensors_cpu["x"].numpy(); y = tensors_cpu["y"].numpy()
    L, N, B, k = cfg["L"], cfg["N"], cfg["B"], cfg["k"]
    L_s = oracle_sample_layers(cfg, seconds)
    w_s = np.ascontiguousarray(w[:L_s]); b_s = np.ascontiguousarray(b[:L_s])
    z, a = orc.forward(w_s, b_s, x)
    reps, t_seq, t_lf = 0, 0.0, 0.0
    t_end = time.perf_counter() + seconds
    while True:
        t0 = time.perf_counter()
        orc.backward_sequential(w_s, z, a, y, want_gw=True)
        t1 = time.perf_counter()
        orc.backward_leapfrog(w_s, z, a, y, k, want_gw=True, threads=True)
        t2 = time.perf_counter()
        t_seq += t1 - t0; t_lf += t2 - t1; reps += 1
        if time.perf_counter() > t_end or reps >= 50:
            break
    cores = os.cpu_count() or 1
    return {
        "value": L_s * reps / t_lf, "unit": UNIT, "cores": min(k, L_s, cores), "kind": "oracle",
        "sample": (f"Algorithm 1 literal with k={k} pthreads, float64, L={L_s} of {L} layers, "
                   f"N={N}, B={B}, {reps} repetitions"),
        "sequential_value": L_s * reps / t_seq, "host_cores": cores,
    }


def oracle_sample_layers(cfg, seconds):
    """Layers of the workload the oracle is timed on: fewer layers of the same width and batch for
    the big workloads, so that a repetition stays within the time given."""
    L_s = cfg["L"]
    per_layer_macs = 3.0 * cfg["N"] * cfg["N"] * cfg["B"]
    while L_s > 2 and per_layer_macs * L_s * max(1, cfg["k"]) > 4e9 * seconds:
        L_s //= 2
    return L_s


def workload_name(index, cfg):
    return (f"configs[{index - 1}]: L={cfg['L']} N={cfg['N']} B={cfg['B']} k={cfg['k']} fp32, "
            f"y={cfg['y']}")


def workload_config(index, cfg):
    """The `config` object of the JSON line: the workload and nothing else, the same for both arms."""
    return {"workload": workload_name(index, cfg), "L": cfg["L"], "N": cfg["N"], "B": cfg["B"],
            "k": cfg["k"], "y": cfg["y"]}


def run_reference(args):
    """The reference arm: the float64 CPU oracle, timed as it stands on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import lf_inputs
    cfg = dict(lf_inputs.CONFIGS[args.config])
    if args.layers:
        cfg["L"] = args.layers
    if args.k:
        cfg["k"] = args.k
    per_step = max(1.0, min(15.0, 90.0 / max(1, args.steps + args.warmup)))
    # only the layers the bounded sample uses are drawn (the full weights of the largest workload
    # would take longer to draw on the host than the sample takes to time)
    L_s = oracle_sample_layers(cfg, per_step)
    cpu = lf_inputs.make_inputs(L_s, cfg["N"], cfg["B"], cfg["y"], lf_inputs.SEED_BASE + args.config, "cpu")
    for _ in range(min(args.warmup, 1)):
        time_oracle(cfg, cpu, 0.01)
    vals, t0 = [], time.perf_counter()
    base = None
    for _ in range(max(1, min(args.steps, 5))):
        base = time_oracle(cfg, cpu, per_step)
        vals.append(base["value"])
    wall = time.perf_counter() - t0
    v = statistics.median(vals)
    base["value"] = v
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1000.0 * cfg["L"] / v, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(args.config, cfg),
            "cpu_baseline": base,
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": wall}
    print(json.dumps(line))
    return 0


def aggregate_rate(total_ms, units_per_rank, dist=None, device=None):
    """Whole-job rate over all ranks: every rank processed `units_per_rank` units in its own
    `total_ms`; the job took as long as its slowest rank (max over ranks).  Returns
    (rate in units/s, max total ms, world size).  Works on any torch.distributed backend."""
    import torch
    world = 1
    t = torch.tensor([float(total_ms)], dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized():
        world = dist.get_world_size()
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    tmax = float(t.item())
    return world * units_per_rank / (tmax * 1e-3), tmax, world


# DRAM traffic of the dominant kernel from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum per
# launch; the summaries are under profiles/).  A figure is reported only for the workload, variant
# and tiling it was captured on, and only while the kernel's source file is byte for byte the one
# that was captured (sha1 below); otherwise `traffic` is null.  configs[2] is too large to capture
# whole: its figure comes from an 8-layer capture of the same kernel at the same width.  Reads grow
# in proportion to the layers read (L - 1: every layer's weights once; the capture shows no
# re-reads); writes are the 4N^2 L bytes of gradients minus what is still dirty in L2 when the
# kernel ends, which the capture gives as a constant (its own 4N^2 L minus its DRAM writes).
NCU_TRAFFIC = {
    # (config, variant, fused tiling): (dram read bytes, dram write bytes per launch of the captured case -- the
    #                                   mean of two launches --, its L, source file, its sha1, summary)
    (1, 3, 2): (150912.0, 0.0, 8, "lf_columns.cu", "5866974fe3e0c9eb3f262f37c4e80b5c28c9ddde",
                "profiles/dram_traffic_single_launch_kernels.md"),
    (2, 2, 0): (130491264.0, 75927168.0, 32, "lf_persistent.cu", "e14e12f511204a4c890f47c1f3d5c2e4c983d116",
                "profiles/dram_traffic_single_launch_kernels.md"),
    (3, 3, 1): (470152192.0, 476112000.0, 8, "lf_persistent.cu", "e14e12f511204a4c890f47c1f3d5c2e4c983d116",
                "profiles/dram_traffic_single_launch_kernels.md"),
}


def source_sha1(name):
    try:
        with open(os.path.join(CSRC, name), "rb") as f:
            return hashlib.sha1(f.read()).hexdigest()
    except OSError:
        return None


def ncu_traffic(index, stats, L, N, B, plain):
    """(traffic bytes per launch or None, provenance string or None)."""
    ent = NCU_TRAFFIC.get((index, stats["variant"], stats.get("fused_tiling", 0)))
    if not ent or not plain:
        return None, None
    cap_read, cap_write, cap_L, src, sha, summary = ent
    if source_sha1(src) != sha:
        return None, f"stale: {src} has changed since the capture in {summary}"
    if cap_L == L:
        return cap_read + cap_write, f"{summary} (as captured; {src} sha1 {sha[:12]})"
    dirty_tail = 4.0 * N * N * cap_L - cap_write
    traffic = cap_read * (L - 1) / max(cap_L - 1, 1) + 4.0 * N * N * L - dirty_tail
    return traffic, (f"{summary} (captured at L={cap_L}: reads scaled by (L-1)/{cap_L - 1}, writes = 4N^2 L minus the "
                     f"{dirty_tail / 1e6:.0f} MB still dirty in L2 at the end; {src} sha1 {sha[:12]})")


def time_gw_gemm(lf, L, N, B, delta_l, a_prev, gw_slabs, stream, steps, tc_tiling=0):
    """Average time of the mini-batch weight-gradient contraction (Eq. bp4 of one layer) launched
    alone through lf_grad_w on delta_l and a_prev [B][N], writing to rotating gw slabs."""
    import torch
    ctx = lf.Leapfrog(L, N, B, 1, stream=stream.cuda_stream)
    ctx.set_option(lf.LF_OPT_TC_TILING, tc_tiling)
    n = len(gw_slabs)
    with torch.cuda.stream(stream):
        for i in range(3):
            ctx.grad_w(delta_l, a_prev, gw_slabs[i % n])
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(steps):
            ctx.grad_w(delta_l, a_prev, gw_slabs[i % n])
        e1.record(stream)
        ctx.sync()
    ms = e0.elapsed_time(e1) / steps
    st = ctx.stats()
    ctx.close()
    return ms, st["gw_math"], st["gw_tiling"]


class Workload:
    """One named workload resident on the device: rotating buffer sets, one context per set."""

    def __init__(self, lf, torch, lf_inputs, index, args, dev, stream, shard=(1, 0), L_override=0, k=None):
        self.lf, self.torch, self.index, self.dev, self.stream = lf, torch, index, dev, stream
        cfg = dict(lf_inputs.CONFIGS[index])
        if L_override:
            cfg["L"] = L_override
        if k is not None:
            cfg["k"] = k
        S, r = shard
        self.cfg = cfg
        L, N, B = cfg["L"], cfg["N"], cfg["B"]
        # Rotating buffer sets: consecutive steps touch different w / gw, so a step never finds
        # its inputs in the 126 MB L2 left there by the step before.
        self.set_bytes = 2 * 4 * L * N * N
        n_sets = max(2, min(8, int((1 << 30) // max(self.set_bytes, 1))))
        self.n_sets = n_sets
        base = lf_inputs.make_inputs(L, N, B, cfg["y"], lf_inputs.SEED_BASE + index, dev)
        self.sets = []
        for i in range(n_sets):
            t = {kk: (v if i == 0 else v.clone()) for kk, v in base.items()}
            t["z"] = torch.empty((L, B, N), dtype=torch.float32, device=dev)
            t["a"] = torch.empty((L + 1, B, N), dtype=torch.float32, device=dev)
            t["delta"] = torch.empty((L, B, N), dtype=torch.float32, device=dev)
            t["gw"] = torch.empty((L, N, N), dtype=torch.float32, device=dev)
            t["gb"] = torch.empty((L, N), dtype=torch.float32, device=dev)
            ctx = lf.Leapfrog(L, N, B, cfg["k"], stream=stream.cuda_stream)
            ctx.set_option(lf.LF_OPT_VARIANT, VARIANT_NAMES[args.variant])
            ctx.set_option(lf.LF_OPT_FUSED_TILING, FUSED_TILING_NAMES[args.fused_tiling])
            ctx.set_option(lf.LF_OPT_TC_TILING, TC_TILING_NAMES[args.tc_tiling])
            ctx.set_option(lf.LF_OPT_SHARD_COUNT, S)
            ctx.set_option(lf.LF_OPT_SHARD_RANK, r)
            t["ctx"] = ctx
            self.sets.append(t)
        torch.cuda.synchronize(dev)
        for t in self.sets:
            t["ctx"].forward(t["w"], t["b"], t["x"], t["z"], t["a"])
            t["ctx"].sync()
        self.sgd = args.sgd

    def step(self, i):
        t = self.sets[i % self.n_sets]
        if self.sgd is not None:   # gw receives the updated weights
            t["ctx"].backward_sgd(t["w"], t["z"], t["a"], t["y"], self.sgd, t["delta"], t["gw"], t["gb"])
        else:
            t["ctx"].backward(t["w"], t["z"], t["a"], t["y"], t["delta"], t["gw"], t["gb"])

    def timed(self, steps, warmup, barrier, sample_clocks, local):
        """W warm-up steps, then exactly `steps` steps between CUDA events on the launching stream.
        Returns (total ms, clocks dict or None)."""
        torch, stream = self.torch, self.stream
        with torch.cuda.stream(stream):
            for i in range(max(3, warmup)):
                self.step(i)
            stream.synchronize()
            barrier()
            sampler = ClockSampler(local) if sample_clocks else None
            if sampler:
                sampler.start()
                time.sleep(0.25)
            ev0 = torch.cuda.Event(enable_timing=True)
            ev1 = torch.cuda.Event(enable_timing=True)
            ev0.record(stream)
            for i in range(steps):
                self.step(i)
            ev1.record(stream)
            stream.synchronize()
            barrier()
            # keep the load on while the sampler collects a few more rows (short regions would
            # otherwise be missed entirely); these extra steps are not timed
            if sampler:
                t_end = time.perf_counter() + 0.5
                i = 0
                while time.perf_counter() < t_end:
                    self.step(i); i += 1
                    if i % 64 == 0:
                        stream.synchronize()
                stream.synchronize()
            clocks = sampler.stop() if sampler else None
        total_ms = ev0.elapsed_time(ev1)
        for t in self.sets:
            t["ctx"].sync()
        return total_ms, clocks

    def stats(self):
        return self.sets[0]["ctx"].stats()

    def close(self):
        for t in self.sets:
            t["ctx"].close()
        self.sets = []
        self.torch.cuda.empty_cache()


def hbm_roofline(wl, stats, ms_per_step, peak, peak_kind, shard_count, args):
    cfg = wl.cfg
    L, N, B = cfg["L"], cfg["N"], cfg["B"]
    alg = algorithmic_bytes(L, N, B)
    if args.sgd is not None:
        alg += 4 * N * N          # the update also reads w^1, which the plain pass never touches
    if shard_count > 1:           # shard r stores only the layers L - r, L - r - S, ... (rank 0's figures)
        alg -= 4 * N * N * (L - len(range(L, 0, -shard_count)))
    launches = stats["launches_backward"]
    if launches == 1:
        tiling = {1: ", cluster tiles", 2: ", whole columns per CTA"}.get(stats.get("fused_tiling", 0), "")
        kernel = {2: "k_backward_persistent (leapfrog CTA groups)",
                  3: ("k_backward_columns" if stats.get("fused_tiling") == 2 else "k_backward_persistent")
                     + " (fused pass" + tiling + ")"}.get(stats["variant"], "persistent backward kernel")
        kernel += ", one launch per step"
    else:
        kernel = f"whole step ({launches} launches replayed from one CUDA graph)"
    achieved = alg / (ms_per_step * 1e-3) / 1e9
    plain = shard_count == 1 and args.sgd is None and not args.k
    traffic, traffic_from = ncu_traffic(wl.index, stats, L, N, B, plain)
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": traffic, "traffic_from": traffic_from, "peak_kind": f"of {peak_kind}",
            "kernel": kernel, "algorithmic_bytes_per_launch": alg, "avg_launch_ms": ms_per_step,
            "frac_of_nominal_8TBs": achieved / 8000.0}


def tensor_roofline(lf, torch, wl, stream, peak, peak_kind, peaks, args, whole_step_gbs):
    """Mini-batch: the weight gradient is a dense N x N x B contraction on the tensor cores.  Its
    launch is timed alone; its bound is the slower of the 4N^2-byte store stream and the 2N^2B
    flops at the TF32 peak.  Two TF32 denominators: the derived one (measured bf16 burst peak x the
    nominal tf32/bf16 ratio 1.1/2.25) and a same-run contraction of the library's own at
    N = 8192, B = 1024 (tensor-bound, the largest point of the sweep grid)."""
    cfg = wl.cfg
    L, N, B = cfg["L"], cfg["N"], cfg["B"]
    t0 = wl.sets[0]
    tiling = TC_TILING_NAMES[args.tc_tiling]
    gemm_ms, gw_math, gw_tiling = time_gw_gemm(lf, L, N, B, t0["delta"][L - 1], t0["a"][L - 1],
                                               [t0["gw"][i] for i in range(L)], stream, 200, tiling)
    flops = 2.0 * N * N * B
    tf32_derived = float(peaks.get("bf16_tflops", BF16_FALLBACK_TFLOPS)) * (1.1 / 2.25)
    # same-run TF32 figure: lf_grad_w at N = 8192, B = 1024 (68.7 GFLOP per launch)
    Nr, Br = 8192, 1024
    g = torch.Generator(device=wl.dev); g.manual_seed(7)
    d_r = torch.empty((Br, Nr), device=wl.dev).normal_(0.0, 1.0, generator=g)
    a_r = torch.empty((Br, Nr), device=wl.dev).uniform_(0.0, 1.0, generator=g)
    slabs = [torch.empty((Nr, Nr), device=wl.dev) for _ in range(2)]
    ref_ms, ref_math, ref_tiling = time_gw_gemm(lf, 1, Nr, Br, d_r, a_r, slabs, stream, 30, tiling)
    same_run = 2.0 * Nr * Nr * Br / (ref_ms * 1e-3) / 1e12 if ref_math == 2 else None
    del d_r, a_r, slabs
    t_store = 4.0 * N * N / (peak * 1e9)
    t_math = flops / (tf32_derived * 1e12)
    if gw_math == 2 and t_math >= t_store:
        ach = flops / (gemm_ms * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": ach, "peak": tf32_derived, "unit": "TFLOP/s",
                "frac": ach / tf32_derived, "traffic": None,
                "peak_kind": f"of {peak_kind} bf16 burst x 1.1/2.25 (tf32)"}
    else:
        gbytes = (4.0 * N * N + 8.0 * N * B) / (gemm_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": gbytes, "peak": peak, "unit": "GB/s",
                "frac": gbytes / peak, "traffic": None, "peak_kind": f"of {peak_kind}"}
    kern = "k_gw_gemm_tf32_pair" if gw_tiling == 2 else "k_gw_gemm_tf32"
    ach_tf = flops / (gemm_ms * 1e-3) / 1e12
    roof.update({"kernel": f"{kern} (one layer, launched alone through lf_grad_w, back to back)"
                           if gw_math == 2 else "k_gemm_simt (weight gradient, fp32)",
                 "avg_launch_ms": gemm_ms, "flops_per_launch": flops, "tflops": ach_tf,
                 "tf32_same_run": {"tflops": same_run, "what": f"lf_grad_w at N={Nr}, B={Br} in this run "
                                   f"({ref_ms:.3f} ms per launch, tiling {ref_tiling})",
                                   "frac": (ach_tf / same_run) if same_run else None},
                 "whole_step_algorithmic_GBs": whole_step_gbs,
                 "note": "the step also holds the 3xTF32 delta-chain contractions "
                         "(three tensor-core products per term)"})
    return roof


def run_ours(args):
    import torch
    import lf_inputs
    import paper_1801_04928_b200 as lf

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    by_rank = args.shard_by_rank and world > 1
    base_k = args.k if args.k else lf_inputs.CONFIGS[args.config]["k"]
    shard_count, shard_rank, k_here = shard_plan(world, rank, base_k, args.shards, args.shard_by_rank)
    stream = torch.cuda.Stream(device=dev)
    peak, peak_kind, peaks = measured_peaks()

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # ---- the headline workload
    wl = Workload(lf, torch, lf_inputs, args.config, args, dev, stream, (shard_count, shard_rank),
                  L_override=args.layers, k=k_here)
    cfg = wl.cfg
    L, N, B, k = cfg["L"], cfg["N"], cfg["B"], cfg["k"]
    total_ms, clocks = wl.timed(args.steps, args.warmup, barrier, rank == 0, local)
    stats = wl.stats()
    # replicas: every rank does L layers per step; sharded by rank: the N ranks share one pass
    value, total_ms_max, _ = aggregate_rate(total_ms, L * args.steps / (world if by_rank else 1), dist, dev)
    ms_per_step = total_ms_max / args.steps

    # ---- end to end through the host-buffer entry point (pinned host memory both ways)
    e2e = None
    if not args.no_e2e:
        t = wl.sets[0]
        host = {n: torch.empty(t[n].shape, dtype=torch.float32, pin_memory=True) for n in
                ("w", "z", "a", "y", "delta", "gw", "gb")}
        for n in ("w", "z", "a", "y"):
            host[n].copy_(t[n])
        # the weights of layer 1 and z are not read by the backward pass and are not uploaded
        h2d = sum(host[n].numel() * 4 for n in ("w", "a", "y")) - host["w"][0].numel() * 4
        d2h = sum(host[n].numel() * 4 for n in ("delta", "gw", "gb"))
        if shard_count > 1:   # only the shard's own layers of gw come back
            d2h -= host["gw"][0].numel() * 4 * (L - len(range(L, 0, -shard_count)))
        ctx = t["ctx"]
        with torch.cuda.stream(stream):
            ctx.backward_host(*(host[n] for n in ("w", "z", "a", "y", "delta", "gw", "gb")))
            ctx.sync()
            barrier()
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.e2e_steps):
                ctx.backward_host(*(host[n] for n in ("w", "z", "a", "y", "delta", "gw", "gb")))
            e1.record(stream)
            ctx.sync()
            barrier()
        e2e_ms = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(e2e_ms, op=dist.ReduceOp.MAX)
        e2e = {"value": (1 if by_rank else world) * L * args.e2e_steps / (float(e2e_ms.item()) * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": float(e2e_ms.item()) / args.e2e_steps}
        del host

    if rank != 0:
        wl.close()
        if dist is not None:
            dist.destroy_process_group()
        return 0

    roofline = hbm_roofline(wl, stats, ms_per_step, peak, peak_kind, shard_count, args)
    if B > 1:
        roofline = tensor_roofline(lf, torch, wl, stream, peak, peak_kind, peaks, args, roofline["achieved"])

    cpu_baseline = None
    if not args.no_cpu_baseline and world == 1:
        L_s = oracle_sample_layers(cfg, args.cpu_seconds)
        t = wl.sets[0]
        cpu = {"w": t["w"][:L_s].cpu(), "b": t["b"][:L_s].cpu(), "x": t["x"].cpu(), "y": t["y"].cpu()}
        cpu_baseline = time_oracle(cfg, cpu, args.cpu_seconds)
    impl = {"variant": stats["variant"], "fused_tiling": stats.get("fused_tiling", 0), "gw_math": stats["gw_math"],
            "launches_per_step": stats["launches_backward"],
            **({"fused_sgd_eta": args.sgd} if args.sgd is not None else {}),
            **({"shard": f"0 of {args.shards} (layer-sharded form, one shard's pass)"}
               if args.shards > 1 and not by_rank else {}),
            "parallelism": ("one pass, layers sharded over the ranks, no exchange" if by_rank else
                            "replicas only") if world > 1 else "single GPU",
            "l2_policy": f"{wl.n_sets} rotating buffer sets of {wl.set_bytes >> 20} MiB (w + gw); "
                         "inputs larger than the 126 MB L2"}
    gpu_launches = stats["launches_backward"] * args.steps
    wl.close()

    # ---- the other named workloads, one after the other, each with its own clock sample
    per_config = []
    plain_run = (world == 1 and shard_count == 1 and args.sgd is None and not args.layers and not args.k)
    if plain_run and not args.no_per_config:
        for idx in (1, 2, 3, 4):
            if idx == args.config:
                continue
            o = Workload(lf, torch, lf_inputs, idx, args, dev, stream)
            oc = o.cfg
            probe_ms, _ = o.timed(5, 3, barrier, False, local)
            steps_i = int(min(4000, max(20, 250.0 / max(probe_ms / 5, 1e-3))))
            tot, clk = o.timed(steps_i, 3, barrier, True, local)
            ost = o.stats()
            ms_i = tot / steps_i
            roof = hbm_roofline(o, ost, ms_i, peak, peak_kind, 1, args)
            entry = {"config": workload_config(idx, oc), "steps": steps_i, "ms_per_step": ms_i,
                     "value": oc["L"] / (ms_i * 1e-3), "unit": UNIT,
                     "impl": {"variant": ost["variant"], "fused_tiling": ost.get("fused_tiling", 0),
                              "gw_math": ost["gw_math"], "launches_per_step": ost["launches_backward"],
                              "l2_policy": f"{o.n_sets} rotating buffer sets of {o.set_bytes >> 20} MiB"},
                     "clocks": clk}
            if oc["B"] > 1:
                entry["roofline_whole_step"] = {"flops_per_step": 2.0 * oc["N"] ** 2 * oc["B"] * (2 * oc["L"] - 1),
                                                "tflops": 2.0 * oc["N"] ** 2 * oc["B"] * (2 * oc["L"] - 1) / (ms_i * 1e-3) / 1e12}
                roof = tensor_roofline(lf, torch, o, stream, peak, peak_kind, peaks, args, roof["achieved"])
            if oc["N"] < 256:
                roof["note"] = "latency-bound workload: no roofline claim"
            entry["roofline"] = roof
            per_config.append(entry)
            o.close()

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "strong" if by_rank else "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(args.config, cfg), "impl_config": impl,
        "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e,
        "gpu_launches": gpu_launches, "clocks": clocks, "per_config": per_config,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
