"""Sweep of the backward pass over width, batch, leapfrog workers and variant.

    python -m paper_1801_04928_b200.sweep [--L 48] [--out sweep.jsonl] [--quick]

For every point of the grid (L fixed; N in {256, 1024, 4096, 8192}; B in {1, 16, 128, 1024};
k in {1, 2, 4, 8, 16}) the backward pass is timed with CUDA events for each variant that
exists at that point: for B = 1 the stream schedule, the persistent leapfrog CTA groups and
the fused pass; for B > 1 the stream schedule with the fp32 and the TF32 weight gradient.
One JSON object per line is written, and a table of the fastest variant per (N, B) is printed.
Inputs are the seeded synthetic tensors of ``lf_inputs`` drawn on the GPU.  With ``--rotate`` the
single-sample points run on several buffer sets in turn (as ``bench.py`` does), so that a pass never
finds its weights in L2; without it widths up to about 1024 are partly L2-resident.

    python -m paper_1801_04928_b200.sweep --emit-table sweep.jsonl

prints, from the single-sample rows of an earlier run, the fastest variant per width and worker
class (k <= 4, k > 4) and the width ranges in which each one wins: the table
``LF_VARIANT_AUTO`` encodes.

    python -m paper_1801_04928_b200.sweep --widths 4096,8192,2048,4096,1024 [--B 1 256]

times instead one network whose layers differ in width (``lf_create_widths``: one launch per
layer and step), for every k of the grid, with the bytes the method must move per pass
(4 n_l n_{l-1} written for every layer, read for every layer but the first) and, for B > 1, the
multiply-adds of its contractions (2 B n_l n_{l-1} for every Eq. bp4 and every Eq. bp2) over the time.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def time_point(lf, torch, sets, L, N, B, k, variant, gw_math, steps, warmup, fused_tiling=0):
    """`sets`: one or more buffer sets (dicts of tensors) used in turn."""
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    ctxs = []
    for _ in sets:     # one context per set: the single-launch kernels keep a descriptor of w
        ctx = lf.Leapfrog(L, N, B, k, stream=stream.cuda_stream)
        ctx.set_option(lf.LF_OPT_VARIANT, variant)
        ctx.set_option(lf.LF_OPT_GW_MATH, gw_math)
        ctx.set_option(lf.LF_OPT_FUSED_TILING, fused_tiling)
        ctxs.append(ctx)

    def step(i):
        t, ctx = sets[i % len(sets)], ctxs[i % len(sets)]
        ctx.backward(t["w"], t["z"], t["a"], t["y"], t["delta"], t["gw"], t["gb"])

    with torch.cuda.stream(stream):
        for i in range(max(warmup, len(sets))):
            step(i)
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(steps):
            step(i)
        e1.record(stream)
        for ctx in ctxs:
            ctx.sync()
    st = ctxs[0].stats()
    for ctx in ctxs:
        ctx.close()
    return e0.elapsed_time(e1) / steps, st


def emit_table(path):
    """The choice LF_VARIANT_AUTO should make for one sample, from the rows of a sweep."""
    rows = [json.loads(l) for l in open(path) if l.strip()]
    rows = [r for r in rows if r.get("B") == 1 and "N" in r]
    if not rows:
        print("no single-sample rows in", path)
        return
    label = lambda r: r["variant"] + ("/" + r["fused_tiling"] if r.get("fused_tiling") else "")
    print("| N | workers | fastest | ms | runner-up | ms |")
    print("|---|---|---|---|---|---|")
    winners = {"k<=4": [], "k>4": []}
    for N in sorted({r["N"] for r in rows}):
        for cls, pick in (("k<=4", lambda k: k <= 4), ("k>4", lambda k: k > 4)):
            # the fused pass has no workers: its one row competes in both classes
            cand = [r for r in rows if r["N"] == N and (pick(r["k"]) or r["variant"] == "fused")]
            if not cand:
                continue
            best = {}
            for r in cand:                      # best k of every variant
                if label(r) not in best or r["ms"] < best[label(r)]["ms"]:
                    best[label(r)] = r
            order = sorted(best.values(), key=lambda r: r["ms"])
            second = order[1] if len(order) > 1 else order[0]
            print(f"| {N} | {cls} | {label(order[0])} | {order[0]['ms']:.4f} | {label(second)} | {second['ms']:.4f} |")
            winners[cls].append((N, label(order[0])))
    for cls, seq in winners.items():
        runs, start, prev_n, cur = [], None, None, None
        for N, w in seq:
            if w != cur:
                if cur is not None:
                    runs.append(f"{cur}: N = {start}..{prev_n}")
                cur, start = w, N
            prev_n = N
        if cur is not None:
            runs.append(f"{cur}: N = {start}..{prev_n}")
        print(f"{cls}: " + "; ".join(runs))


def sweep_widths(lf, lf_inputs, torch, widths, Bs, ks, out):
    n = [int(v) for v in widths]
    L = len(n) - 1
    mats = [n[l] * n[l - 1] for l in range(1, L + 1)]
    with open(out, "w") as f:
        for B in Bs:
            t = lf_inputs.make_inputs_widths(n, B, "uniform" if B == 1 else "onehot",
                                             lf_inputs.SEED_BASE + lf_inputs.SWEEP_CONFIG_INDEX, "cuda")
            hidden = sum(n[1:])
            t["z"] = torch.empty(B * hidden, device="cuda"); t["a"] = torch.empty(B * sum(n), device="cuda")
            t["delta"] = torch.empty(B * hidden, device="cuda")
            t["gw"] = torch.empty(sum(mats), device="cuda"); t["gb"] = torch.empty(hidden, device="cuda")
            alg = 4.0 * (2 * sum(mats) - mats[0]) + 12.0 * B * hidden
            flops = 2.0 * B * (2 * sum(mats) - mats[0])
            steps, warmup = (3, 1) if flops > 2e11 else (30, 5)
            # one sample: the stream schedule, and whatever LF_VARIANT_AUTO picks (the single-launch pass
            # when the hidden layers share a width)
            for k, variant in [(k, v) for k in ks for v in ((1, 0) if B == 1 else (1,))]:
                stream = torch.cuda.Stream()
                stream.wait_stream(torch.cuda.current_stream())
                with lf.Leapfrog(0, 0, B, k, stream=stream.cuda_stream, widths=n) as ctx:
                    ctx.set_option(lf.LF_OPT_VARIANT, variant)
                    with torch.cuda.stream(stream):
                        ctx.forward(t["w"], t["b"], t["x"], t["z"], t["a"])
                        for _ in range(warmup):
                            ctx.backward(t["w"], t["z"], t["a"], t["y"], t["delta"], t["gw"], t["gb"])
                        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                        e0.record(stream)
                        for _ in range(steps):
                            ctx.backward(t["w"], t["z"], t["a"], t["y"], t["delta"], t["gw"], t["gb"])
                        e1.record(stream)
                        ctx.sync()
                    st = ctx.stats()
                ms = e0.elapsed_time(e1) / steps
                row = dict(widths=n, B=B, k=k, variant={1: "streams", 2: "persistent", 3: "fused"}[st["variant"]], ms=ms, layers_per_s=L / (ms * 1e-3),
                           alg_GBs=alg / (ms * 1e-3) / 1e9, alg_TFLOPs=flops / (ms * 1e-3) / 1e12 if B > 1 else None,
                           launches=st["launches_backward"])
                f.write(json.dumps(row) + "\n"); f.flush()
                print(json.dumps(row), flush=True)
            del t
            torch.cuda.empty_cache()


SWEEP_L = 48
SWEEP_N = (256, 1024, 4096, 8192)
SWEEP_B = (1, 16, 128, 1024)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--L", type=int, default=SWEEP_L)
    ap.add_argument("--out", default="sweep.jsonl")
    ap.add_argument("--quick", action="store_true", help="k in {1, 4} only")
    ap.add_argument("--N", type=int, nargs="*", default=list(SWEEP_N))
    ap.add_argument("--B", type=int, nargs="*", default=list(SWEEP_B))
    ap.add_argument("--widths", default=None, help="n_0,n_1,...,n_L: time one network of these layer widths")
    ap.add_argument("--rotate", action="store_true",
                    help="single-sample points: run on rotating buffer sets of at least 1 GiB in total")
    ap.add_argument("--emit-table", default=None, metavar="SWEEP_JSONL",
                    help="print the fastest variant per width and worker class from an earlier run, and exit")
    args = ap.parse_args()
    if args.emit_table:
        emit_table(args.emit_table)
        return
    import torch
    import lf_inputs
    import paper_1801_04928_b200 as lf
    assert (SWEEP_L, SWEEP_N, SWEEP_B) == (lf_inputs.SWEEP["L"], lf_inputs.SWEEP["N"], lf_inputs.SWEEP["B"])
    ks = (1, 4) if args.quick else lf_inputs.SWEEP["k"]
    if args.widths:
        sweep_widths(lf, lf_inputs, torch, args.widths.split(","), args.B, ks, args.out)
        return
    L = args.L
    names = {1: "streams", 2: "persistent", 3: "fused"}
    rows = []
    with open(args.out, "w") as f:
        for N in args.N:
            for B in args.B:
                y_kind = "uniform" if B == 1 else "onehot"
                t = lf_inputs.make_inputs(L, N, B, y_kind, lf_inputs.SEED_BASE + lf_inputs.SWEEP_CONFIG_INDEX,
                                          "cuda")
                t["z"] = torch.empty((L, B, N), device="cuda"); t["a"] = torch.empty((L + 1, B, N), device="cuda")
                t["delta"] = torch.empty((L, B, N), device="cuda")
                t["gw"] = torch.empty((L, N, N), device="cuda"); t["gb"] = torch.empty((L, N), device="cuda")
                with lf.Leapfrog(L, N, B, 1) as ctx:
                    ctx.forward(t["w"], t["b"], t["x"], t["z"], t["a"])
                    ctx.sync()
                sets = [t]
                if args.rotate and B == 1:
                    n_sets = max(2, min(8, int((1 << 30) // (8 * L * N * N))))
                    for _ in range(n_sets - 1):
                        sets.append({kk: v.clone() for kk, v in t.items()})
                flops = 2.0 * N * N * B
                slow = flops * L > 2e12            # seconds per step on the fp32 chain
                steps, warmup = (2, 1) if slow else ((5, 2) if N >= 4096 or B > 1 else (50, 5))
                points = []
                if B == 1:
                    for k in ks:
                        points += [(k, 1, lf.LF_GW_MATH_AUTO), (k, 2, lf.LF_GW_MATH_AUTO)]
                    # the fused pass has no k; both of its tilings
                    points += [(1, 3, lf.LF_GW_MATH_AUTO, lf.LF_FUSED_TILING_CLUSTERS),
                               (1, 3, lf.LF_GW_MATH_AUTO, lf.LF_FUSED_TILING_COLUMNS)]
                else:
                    for k in ks:
                        points.append((k, 1, lf.LF_GW_MATH_TF32))
                    points.append((ks[-1] if len(ks) < 3 else 4, 1, lf.LF_GW_MATH_FP32))
                for point in points:
                    k, variant, gw_math = point[:3]
                    tiling = point[3] if len(point) > 3 else 0
                    ms, st = time_point(lf, torch, sets, L, N, B, k, variant, gw_math, steps, warmup, tiling)
                    alg = 4.0 * N * N * (2 * L - 1) + 12.0 * N * B * L
                    row = dict(L=L, N=N, B=B, k=k, variant=names[st["variant"]], requested=names[variant],
                               gw_math={1: "fp32", 2: "tf32"}[st["gw_math"]], ms=ms,
                               fused_tiling={0: None, 1: "clusters", 2: "columns"}[st["fused_tiling"]],
                               buffer_sets=len(sets),
                               layers_per_s=L / (ms * 1e-3), alg_GBs=alg / (ms * 1e-3) / 1e9,
                               chain_ctas=st["chain_ctas"], worker_ctas=st["worker_ctas"],
                               gw_tiling=st["gw_tiling"], delta_tiling=st["delta_tiling"])
                    rows.append(row)
                    f.write(json.dumps(row) + "\n"); f.flush()
                    print(json.dumps(row), flush=True)
                del t, sets
                torch.cuda.empty_cache()
    print("\n| N | B | fastest | k | ms | layers/s | algorithmic GB/s |")
    print("|---|---|---|---|---|---|---|")
    for N in args.N:
        for B in args.B:
            cand = [r for r in rows if r["N"] == N and r["B"] == B]
            if not cand:
                continue
            b = min(cand, key=lambda r: r["ms"])
            print(f"| {N} | {B} | {b['variant']}/{b['gw_math']} | {b['k']} | {b['ms']:.4f} | "
                  f"{b['layers_per_s']:.0f} | {b['alg_GBs']:.0f} |")


if __name__ == "__main__":
    main()
