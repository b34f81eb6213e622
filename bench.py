#!/usr/bin/env python
"""Benchmark of the leapfrog backward pass (arXiv 1801.04928) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--config 1..4] [--variant auto|streams|persistent|fused] [--k K]

A step is one whole backward pass (Eq. bp1, the Eq. bp2 chain, Eq. bp3/bp4 of every layer
under the leapfrog schedule) over one batch of synthetic inputs that are already resident in
device memory.  The metric is backward layers per second (L / step time), reported with the
achieved algorithmic HBM bandwidth of the dominant kernel against the measured copy peak.
With N > 1 GPUs every rank runs an independent replica of the workload (the path does not
shard: the delta chain is sequential in depth), so the aggregate is N times the per-GPU rate.

One JSON line is printed by rank 0.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "backward_layers_per_sec"
UNIT = "layers/s"
HBM_FALLBACK_GBS = 6650.0  # used only if MEASURED_PEAKS.json is absent
VARIANT_NAMES = {"auto": 0, "streams": 1, "persistent": 2, "fused": 3}
TC_TILING_NAMES = {"auto": 0, "one_sm": 1, "two_sm": 2}


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=4000)
    p.add_argument("--warmup", type=int, default=10)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--config", type=int, default=2)
    p.add_argument("--variant", default="auto", choices=sorted(VARIANT_NAMES))
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
    p.add_argument("--e2e-steps", type=int, default=5)
    p.add_argument("--cpu-seconds", type=float, default=10.0)
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-e2e", action="store_true")
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
    thread recomputing the delta chain) on the host, as it stands."""
    import numpy as np
    from oracle import lf_oracle as orc
    w = tensors_cpu["w"].numpy(); b = tensors_cpu["b"].numpy()
    x = tensors_cpu["x"].numpy(); y = tensors_cpu["y"].numpy()
    L, N, B, k = cfg["L"], cfg["N"], cfg["B"], cfg["k"]
    # bound the sample for the big workloads: fewer layers of the same width, same batch
    L_s = L
    per_layer_macs = 3.0 * N * N * B
    while L_s > 2 and per_layer_macs * L_s * max(1, k) > 4e9 * seconds:
        L_s //= 2
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


def run_reference(args):
    """The reference arm: the float64 CPU oracle, timed as it stands on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import lf_inputs
    cfg, cpu = lf_inputs.make_config(args.config, **({"L": args.layers} if args.layers else {}))
    if args.k:
        cfg["k"] = args.k
    per_step = max(1.0, min(15.0, 90.0 / max(1, args.steps + args.warmup)))
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
            "config": {"workload": workload_name(args.config, cfg), **cfg},
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


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu capture
# summarised under profiles/) of the dominant kernel, keyed by (config, variant); null elsewhere.
NCU_TRAFFIC = {(2, 2): 206.4e6}


def time_gw_gemm(lf, L, N, B, t, stream, steps, tc_tiling=0):
    """Average time of the mini-batch weight-gradient contraction (Eq. bp4 of one layer) launched
    alone through lf_grad_w, on the top layer's delta and activations, writing to rotating gw slabs."""
    import torch
    ctx = lf.Leapfrog(L, N, B, 1, stream=stream.cuda_stream)
    ctx.set_option(lf.LF_OPT_TC_TILING, tc_tiling)
    d, a_prev = t["delta"][L - 1], t["a"][L - 1]
    with torch.cuda.stream(stream):
        for i in range(3):
            ctx.grad_w(d, a_prev, t["gw"][i % L])
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(steps):
            ctx.grad_w(d, a_prev, t["gw"][i % L])
        e1.record(stream)
        ctx.sync()
    ms = e0.elapsed_time(e1) / steps
    st = ctx.stats()
    ctx.close()
    return ms, st["gw_math"], st["gw_tiling"]


def workload_name(index, cfg):
    return (f"configs[{index - 1}]: L={cfg['L']} N={cfg['N']} B={cfg['B']} k={cfg['k']} fp32, "
            f"y={cfg['y']}")


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

    cfg, cpu = lf_inputs.make_config(args.config, **({"L": args.layers} if args.layers else {}))
    if args.k:
        cfg["k"] = args.k
    elif args.shards > 1 or (args.shard_by_rank and world > 1):
        # the workload's k leapfrog workers are spread over the S GPUs: k / S of them work here
        cfg["k"] = max(1, cfg["k"] // (world if args.shard_by_rank and world > 1 else args.shards))
    L, N, B, k = cfg["L"], cfg["N"], cfg["B"], cfg["k"]
    variant = VARIANT_NAMES[args.variant]
    by_rank = args.shard_by_rank and world > 1
    shard_count, shard_rank = (world, rank) if by_rank else (args.shards, 0)

    # Rotating buffer sets: consecutive steps touch different w / gw, so a step never finds
    # its inputs in the 126 MB L2 left there by the step before.
    set_bytes = 2 * 4 * L * N * N
    n_sets = max(2, min(8, int((1 << 30) // max(set_bytes, 1))))
    if set_bytes * n_sets > 64 << 30:
        n_sets = 2
    stream = torch.cuda.Stream(device=dev)
    base = {kk: v.to(dev) for kk, v in cpu.items()}
    sets = []
    for i in range(n_sets):
        t = {kk: (v if i == 0 else v.clone()) for kk, v in base.items()}
        t["z"] = torch.empty((L, B, N), dtype=torch.float32, device=dev)
        t["a"] = torch.empty((L + 1, B, N), dtype=torch.float32, device=dev)
        t["delta"] = torch.empty((L, B, N), dtype=torch.float32, device=dev)
        t["gw"] = torch.empty((L, N, N), dtype=torch.float32, device=dev)
        t["gb"] = torch.empty((L, N), dtype=torch.float32, device=dev)
        ctx = lf.Leapfrog(L, N, B, k, stream=stream.cuda_stream)
        ctx.set_option(lf.LF_OPT_VARIANT, variant)
        ctx.set_option(lf.LF_OPT_TC_TILING, TC_TILING_NAMES[args.tc_tiling])
        ctx.set_option(lf.LF_OPT_SHARD_COUNT, shard_count)
        ctx.set_option(lf.LF_OPT_SHARD_RANK, shard_rank)
        t["ctx"] = ctx
        sets.append(t)
    torch.cuda.synchronize(dev)
    for t in sets:
        t["ctx"].forward(t["w"], t["b"], t["x"], t["z"], t["a"])
        t["ctx"].sync()

    def step(i):
        t = sets[i % n_sets]
        if args.sgd is not None:   # gw receives the updated weights
            t["ctx"].backward_sgd(t["w"], t["z"], t["a"], t["y"], args.sgd, t["delta"], t["gw"], t["gb"])
        else:
            t["ctx"].backward(t["w"], t["z"], t["a"], t["y"], t["delta"], t["gw"], t["gb"])

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    with torch.cuda.stream(stream):
        for i in range(max(3, args.warmup)):
            step(i)
        stream.synchronize()
        barrier()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
            time.sleep(0.25)
        ev0 = torch.cuda.Event(enable_timing=True)
        ev1 = torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for i in range(args.steps):
            step(i)
        ev1.record(stream)
        stream.synchronize()
        barrier()
        # keep the load on while the sampler collects a few more rows (short regions would
        # otherwise be missed entirely); these extra steps are not timed
        if rank == 0:
            t_end = time.perf_counter() + 0.6
            i = 0
            while time.perf_counter() < t_end:
                step(i); i += 1
                if i % 64 == 0:
                    stream.synchronize()
            stream.synchronize()
        clocks = sampler.stop() if rank == 0 else None
    total_ms = ev0.elapsed_time(ev1)
    for t in sets:
        t["ctx"].sync()
    stats = sets[0]["ctx"].stats()

    # replicas: every rank does L layers per step; sharded by rank: the N ranks share one pass
    value, total_ms_max, _ = aggregate_rate(total_ms, L * args.steps / (world if by_rank else 1), dist, dev)
    ms_per_step = total_ms_max / args.steps

    # ---- end to end through the host-buffer entry point (pinned host memory both ways)
    e2e = None
    if not args.no_e2e:
        t = sets[0]
        host = {n: torch.empty_like(t[n], device="cpu").pin_memory() for n in
                ("w", "z", "a", "y", "delta", "gw", "gb")}
        for n in ("w", "z", "a", "y"):
            host[n].copy_(t[n])
        # the weights of layer 1 are not read by the backward pass and are not uploaded
        h2d = sum(host[n].numel() * 4 for n in ("w", "z", "a", "y")) - host["w"][0].numel() * 4
        d2h = sum(host[n].numel() * 4 for n in ("delta", "gw", "gb"))
        if shard_count > 1:   # only the shard's own layers of gw come back
            d2h -= host["gw"][0].numel() * 4 * (L - len(range(L, 0, -shard_count)))
        ctx = t["ctx"]
        with torch.cuda.stream(stream):
            for _ in range(2):
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

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    peak, peak_kind, peaks = measured_peaks()
    alg = algorithmic_bytes(L, N, B)
    if args.sgd is not None:
        alg += 4 * N * N          # the update also reads w^1, which the plain pass never touches
    if shard_count > 1:           # shard r stores only the layers L - r, L - r - S, ... (rank 0's figures)
        owned = len(range(L, 0, -shard_count))
        alg -= 4 * N * N * (L - owned)
    launches_per_step = stats["launches_backward"]
    if launches_per_step == 1:
        kernel_name = "persistent backward kernel (one launch per step)"
    else:
        kernel_name = f"whole step ({launches_per_step} launches replayed from one CUDA graph)"
    achieved = alg / (ms_per_step * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak,
                # counters exist for the plain pass of the named workload only
                "traffic": NCU_TRAFFIC.get((args.config, stats["variant"]))
                if shard_count == 1 and args.sgd is None and not args.layers and not args.k else None,
                "peak_kind": f"of {peak_kind}",
                "kernel": kernel_name, "algorithmic_bytes_per_launch": alg,
                "avg_launch_ms": ms_per_step,
                "frac_of_nominal_8TBs": achieved / 8000.0}
    if B > 1:
        # Mini-batch: the weight gradient is a dense N x N x B contraction on the tensor cores.
        # Its launch is timed alone; its bound is the slower of the 4N^2-byte store stream and
        # the 2N^2B flops at the TF32 peak (measured bf16 burst peak x nominal tf32/bf16 ratio).
        gemm_ms, gw_math, gw_tiling = time_gw_gemm(lf, L, N, B, sets[0], stream, 200,
                                                   TC_TILING_NAMES[args.tc_tiling])
        flops = 2.0 * N * N * B
        tf32_peak = float(peaks.get("bf16_tflops", 1590.0)) * (1.1 / 2.25)
        t_store = 4.0 * N * N / (peak * 1e9)
        t_math = flops / (tf32_peak * 1e12)
        if gw_math == 2 and t_math >= t_store:
            ach = flops / (gemm_ms * 1e-3) / 1e12
            roofline = {"bound": "tensor", "achieved": ach, "peak": tf32_peak, "unit": "TFLOP/s",
                        "frac": ach / tf32_peak, "traffic": None,
                        "peak_kind": f"of {peak_kind} bf16 burst x 1.1/2.25 (tf32)"}
        else:
            gbytes = (4.0 * N * N + 8.0 * N * B) / (gemm_ms * 1e-3) / 1e9
            roofline = {"bound": "hbm", "achieved": gbytes, "peak": peak, "unit": "GB/s",
                        "frac": gbytes / peak, "traffic": None, "peak_kind": f"of {peak_kind}"}
        tf32_kernel = "k_gw_gemm_tf32_pair" if gw_tiling == 2 else "k_gw_gemm_tf32"
        roofline.update({"kernel": f"{tf32_kernel} (one layer, launched alone through lf_grad_w, back to back)"
                                   if gw_math == 2 else "k_gemm_simt (weight gradient, fp32)",
                         "avg_launch_ms": gemm_ms, "flops_per_launch": flops,
                         "tflops": flops / (gemm_ms * 1e-3) / 1e12,
                         "whole_step_algorithmic_GBs": achieved,
                         "note": "the step also holds the 3xTF32 delta-chain contractions "
                                 "(three tensor-core products per term)"})

    cpu_baseline = None
    if not args.no_cpu_baseline and world == 1:
        cpu_baseline = time_oracle(cfg, cpu, args.cpu_seconds)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "strong" if by_rank else "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(args.config, cfg), "L": L, "N": N, "B": B, "k": k,
                   "variant": stats["variant"], "gw_math": stats["gw_math"],
                   **({"fused_sgd_eta": args.sgd} if args.sgd is not None else {}),
                   **({"shard": f"0 of {args.shards} (layer-sharded form, one shard's pass)"}
                      if args.shards > 1 and not by_rank else {}),
                   "parallelism": ("one pass, layers sharded over the ranks, no exchange" if by_rank else
                                   "replicas only") if world > 1 else "single GPU",
                   "l2_policy": f"{n_sets} rotating buffer sets of {set_bytes >> 20} MiB (w + gw); "
                                "inputs larger than the 126 MB L2"},
        "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e,
        "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
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
