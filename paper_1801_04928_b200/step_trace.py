"""Where the time goes inside the single-launch backward kernels (B = 1), one layer step at a time,
and inside the two-SM tensor-core kernel of the mini-batch chain, one K stage at a time.

    python -m paper_1801_04928_b200.step_trace [--N 1024] [--L 32] [--k 4]
                                               [--kernel groups|clusters|columns|all]
    python -m paper_1801_04928_b200.step_trace --kernel pair [--N 4096] [--B 256] [--delta-math 2|3]
    python -m paper_1801_04928_b200.step_trace --kernel gwpair [--N 4096] [--B 256]

Builds a DEBUG copy of the library (``-DLF_PK_TRACE -DLF_CK_TRACE -DLF_DG_TRACE -DLF_TG_TRACE``: thread 0 of two
CTAs, or the leader CTA of the first CTA pair, writes SM-clock stamps at fixed points of every
layer step or K stage; the release library carries none of this) under ``_build/trace/``, runs a
few passes of the chosen kernel on seeded inputs and prints the median number of SM cycles
between consecutive stamps, the whole step or stage, and the event-timed pass.  For the B = 1
kernels the weights of the one buffer set stay in L2 between passes, so the figures describe the
hand-off, not the memory system.

Stamps of the cluster kernel (``groups``: leapfrog CTA groups; ``clusters``: fused pass):
0 step starts, 1 first weight sub-tile is there, 3 all column blocks multiplied and the partial
sums sent, 4 the cluster's partial sums for my columns have arrived, 5 delta published,
6 delta of my rows has arrived from the other clusters.
Stamps of the whole-columns kernel (``columns``): 0 step starts, 1 delta of this warp's rows has
arrived, 2 multiplied, 3 the CTA's barrier is passed, 4 delta published.
Stamps of the two-SM contraction kernel (``pair``; k_delta_gemm_tc_pair, Eq. z with --what forward,
Eq. bp2 with --what backward), per 32-wide K stage of the first pair's leader CTA: 0 the stage's
loads are issued, 1 they have landed, 2 the second-ring slot is free, 3 the split is written,
4 the issuing thread sees the split, 5 it has the accumulator, 6 the products and commits are
issued, 7 the products are done (seen by a summing warp), 8 that warp has added the stage.
"""
from __future__ import annotations

import argparse
import ctypes
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1801_04928_b200 import build as lfbuild   # noqa: E402  (sources and flags of the release build)

TRACE_DIR = os.path.join(lfbuild.OBJ, "trace")
TRACE_LIB = os.path.join(TRACE_DIR, "libleapfrog_trace.so")

KERNELS = {  # name -> (LF_OPT_VARIANT, LF_OPT_FUSED_TILING, stamps in order, names of the intervals)
    "groups": (2, 0, [0, 1, 3, 4, 5, 6], ["wait for the first weight sub-tile", "multiply, reduce, send partial sums",
                                          "wait for the cluster's partial sums", "add them, sigma', publish",
                                          "wait for delta of my rows"]),
    "clusters": (3, 1, [0, 1, 3, 4, 5, 6], ["wait for the first weight sub-tile", "multiply, reduce, send partial sums",
                                            "wait for the cluster's partial sums", "add them, sigma', publish",
                                            "wait for delta of my rows"]),
    "columns": (3, 2, [0, 1, 2, 3, 4], ["wait for delta of the warp's rows (one hop through L2)", "multiply",
                                        "reduce in the warp, CTA barrier", "add the warps' sums, sigma', publish"]),
}


def build_trace_library() -> str:
    os.makedirs(TRACE_DIR, exist_ok=True)
    nvcc = lfbuild._nvcc()
    flags = [f for f in lfbuild.NVCC_FLAGS if f not in ("-Xptxas", "-v")] + ["-DLF_PK_TRACE", "-DLF_CK_TRACE", "-DLF_DG_TRACE", "-DLF_TG_TRACE"]

    def one(src):
        obj = os.path.join(TRACE_DIR, src.replace(".cu", ".o"))
        r = subprocess.run([nvcc, *flags, "-c", os.path.join(lfbuild.CSRC, src), "-o", obj], capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n{r.stderr}")
        return obj

    with ThreadPoolExecutor(max_workers=len(lfbuild.SOURCES)) as ex:
        objs = list(ex.map(one, lfbuild.SOURCES))
    r = subprocess.run([nvcc, "-shared", "-o", TRACE_LIB, *objs, "-gencode", "arch=compute_100a,code=sm_100a"],
                       capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stderr}")
    return TRACE_LIB


def trace(lib, torch, lf_inputs, np, name, L, N, k):
    variant, tiling, stamps, names = KERNELS[name]
    vp = ctypes.c_void_p
    P = lambda x: vp(x.data_ptr())
    t = lf_inputs.make_inputs(L, N, 1, "uniform", lf_inputs.SEED_BASE + 2, "cuda")
    z = torch.empty((L, 1, N), device="cuda"); a = torch.empty((L + 1, 1, N), device="cuda")
    d = torch.empty((L, 1, N), device="cuda"); gw = torch.empty((L, N, N), device="cuda"); gb = torch.empty((L, N), device="cuda")
    h = vp()
    assert lib.lf_create(ctypes.byref(h), L, N, 1, k) == 0
    lib.lf_set_option(h, 1, variant); lib.lf_set_option(h, 12, tiling)
    lib.lf_forward(h, P(t["w"]), P(t["b"]), P(t["x"]), P(z), P(a))
    back = lambda: lib.lf_backward(h, P(t["w"]), P(z), P(a), P(t["y"]), P(d), P(gw), P(gb))
    for _ in range(3):
        assert back() == 0
    assert lib.lf_sync(h) == 0
    buf = (ctypes.c_ulonglong * (2 * L * 16))()
    assert lib.lf_debug_read_trace(h, buf) == 0
    stride = 8 if name == "columns" else 16
    tr = np.array(buf, dtype=np.int64)[:2 * L * stride].reshape(2, L, stride)
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(); e0.record()
    for _ in range(20):
        back()
    e1.record(); torch.cuda.synchronize()
    assert lib.lf_sync(h) == 0
    lib.lf_destroy(h)
    print(f"\n## {name}: L = {L}, N = {N}, k = {k}; pass (weights L2-warm, debug build): {e0.elapsed_time(e1) / 20 * 1e3:.1f} us")
    print("| interval | " + " | ".join(f"CTA {'0' if c == 0 else 'other'} (median cycles)" for c in range(2)) + " |")
    print("|---|---|---|")
    med = []
    for c in range(2):
        seg = []
        for i in range(2, L - 3):          # steady-state layers: not the first two, not the last two
            r, nx = tr[c][i], tr[c][i + 1]
            if r[stamps[0]] == 0 or nx[stamps[0]] == 0:
                continue
            seg.append([r[stamps[j + 1]] - r[stamps[j]] for j in range(len(stamps) - 1)] +
                       [nx[stamps[0]] - r[stamps[-1]], nx[stamps[0]] - r[stamps[0]]])
        med.append(np.median(np.array(seg), axis=0) if seg else None)
    rows = names + ["rest of the step (housekeeping off the chain)", "whole layer step"]
    for j, nm in enumerate(rows):
        print(f"| {nm} | " + " | ".join("n/a" if m is None else f"{int(m[j])}" for m in med) + " |")


PAIR_STAMPS = ["loads issued -> landed", "landed -> second-ring slot free (the splitting warp gets to the stage)",
               "split (high parts in place, the rest to the second ring)", "split written -> seen by the issuing thread",
               "issuing thread waits for the accumulator", "issue of the stage's products and commits",
               "issued -> products done", "summing warp adds the stage"]


def trace_pair(lib, torch, lf_inputs, np, N, B, what, delta_math):
    """One contraction of the CTA-pair kernel: Eq. z of a one-layer net, or Eq. bp2 of a two-layer net."""
    vp = ctypes.c_void_p
    P = lambda x: vp(x.data_ptr())
    L = 1 if what == "forward" else 2
    t = lf_inputs.make_inputs(L, N, B, "onehot", lf_inputs.SEED_BASE + 3, "cuda")
    z = torch.empty((L, B, N), device="cuda"); a = torch.empty((L + 1, B, N), device="cuda")
    d = torch.empty((L, B, N), device="cuda"); gw = torch.empty((L, N, N), device="cuda"); gb = torch.empty((L, N), device="cuda")
    h = vp()
    assert lib.lf_create(ctypes.byref(h), L, N, B, 1) == 0
    lib.lf_set_option(h, 6, delta_math); lib.lf_set_option(h, 7, 2)      # LF_OPT_DELTA_MATH, LF_OPT_TC_TILING = two-SM
    for _ in range(3):
        assert lib.lf_forward(h, P(t["w"]), P(t["b"]), P(t["x"]), P(z), P(a)) == 0
        if what == "backward":
            assert lib.lf_backward(h, P(t["w"]), P(z), P(a), P(t["y"]), P(d), P(gw), P(gb)) == 0
    assert lib.lf_sync(h) == 0
    buf = (ctypes.c_longlong * (128 * 16))()
    assert lib.lf_debug_read_pair_trace(buf) == 0
    lib.lf_destroy(h)
    once = np.array(buf, dtype=np.int64)[9:13]        # kernel entered, set-up done, last partial sums written, before the exit
    tr = np.array(buf, dtype=np.int64).reshape(128, 16)[:, :9]
    n = 0
    while n < 128 and tr[n, 6] != 0 and (n == 0 or tr[n, 6] > tr[n - 1, 6]):
        n += 1
    print(f"\n## pair kernel, {what} (Eq. {'z' if what == 'forward' else 'bp2'}): N = {N}, B = {B}, delta math {delta_math}; "
          f"{n} K stages in the first pair's run")
    if n < 8:
        print("(too few stages for a steady state)")
        return
    body = tr[3:n - 1]                       # steady state: the rings are full, the last stage is not special
    print("| interval | median cycles |")
    print("|---|---|")
    for j, nm in enumerate(PAIR_STAMPS):
        print(f"| {nm} | {int(np.median(body[:, j + 1] - body[:, j]))} |")
    print(f"| **stage period** (products issued, stage to stage) | {int(np.median(np.diff(tr[3:n, 6])))} |")
    print(f"| whole run of the pair: first load issued -> last stage added | {int(tr[n - 1, 8] - tr[0, 0])} |")
    print(f"| kernel entered -> set-up done (barriers, tensor memory, cluster barrier) | {int(once[1] - once[0])} |")
    print(f"| set-up done -> first load issued | {int(tr[0, 0] - once[1])} |")
    print(f"| last stage added -> last partial sums written | {int(once[2] - tr[n - 1, 8])} |")
    print(f"| last partial sums written -> cluster barrier before the exit passed | {int(once[3] - once[2])} |")
    print(f"| kernel entered -> before the exit | {int(once[3] - once[0])} |")


def trace_gw_pair(lib, torch, np, N, B):
    """Eq. bp4 of one layer through lf_grad_w on the two-SM kernel: stamps per 256 x 256 tile of the
    first pair's leader CTA: 0 the issuing thread has the accumulator, 1 it sees the first stage's
    operands, 2 all products and commits of the tile are issued, 3 an epilogue warp sees the finished
    accumulator, 4 that warp has stored its part of the tile."""
    vp = ctypes.c_void_p
    P = lambda x: vp(x.data_ptr())
    g = torch.Generator(device="cuda"); g.manual_seed(7)
    d = torch.empty((B, N), device="cuda").normal_(0.0, 1.0, generator=g)
    a = torch.empty((B, N), device="cuda").uniform_(0.0, 1.0, generator=g)
    gw = torch.empty((N, N), device="cuda")
    h = vp()
    assert lib.lf_create(ctypes.byref(h), 1, N, B, 1) == 0
    lib.lf_set_option(h, 2, 2); lib.lf_set_option(h, 7, 2)      # LF_OPT_GW_MATH = TF32, LF_OPT_TC_TILING = two-SM
    for _ in range(3):
        assert lib.lf_grad_w(h, P(d), P(a), P(gw)) == 0
    assert lib.lf_sync(h) == 0
    buf = (ctypes.c_longlong * (32 * 16))()
    assert lib.lf_debug_read_gw_pair_trace(buf) == 0
    lib.lf_destroy(h)
    tr = np.array(buf, dtype=np.int64).reshape(32, 16)
    n = 0
    while n < 32 and tr[n, 2] != 0 and (n == 0 or tr[n, 2] > tr[n - 1, 2]):
        n += 1
    t0 = tr[0, 8]
    print(f"\n## weight-gradient pair kernel (Eq. bp4): N = {N}, B = {B}; {n} tiles in the first pair's run; cycles since the kernel was entered")
    print(f"set-up done {int(tr[0, 9] - t0)}, first operand load issued {int(tr[0, 10] - t0)}")
    print("| tile | issuer has the accumulator | first operands seen | products issued | epilogue sees the accumulator | epilogue warp done |")
    print("|---|---|---|---|---|---|")
    for t in range(n):
        print(f"| {t} | " + " | ".join(str(int(tr[t, j] - t0)) for j in range(5)) + " |")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--N", type=int, default=1024)
    ap.add_argument("--L", type=int, default=32)
    ap.add_argument("--k", type=int, default=4)
    ap.add_argument("--kernel", default="all", choices=["all", "pair", "gwpair"] + sorted(KERNELS))
    ap.add_argument("--B", type=int, default=256, help="pair: samples")
    ap.add_argument("--delta-math", type=int, default=2, help="pair: 2 = three TF32 products, 3 = cross terms in BF16")
    ap.add_argument("--what", default="both", choices=["forward", "backward", "both"], help="pair: which contraction")
    args = ap.parse_args()
    import numpy as np
    import torch
    import lf_inputs
    if not torch.cuda.is_available():
        raise SystemExit("step_trace: no CUDA device")
    lib = ctypes.CDLL(build_trace_library())
    lib.lf_set_option.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong]
    clock = subprocess.run(["nvidia-smi", "--query-gpu=clocks.sm,clocks.max.sm", "--format=csv,noheader"],
                           capture_output=True, text=True).stdout.strip()
    print(f"SM clock now / max: {clock} (cycles -> ns: divide by the GHz under load)")
    if args.kernel == "gwpair":
        trace_gw_pair(lib, torch, np, args.N, args.B)
        return
    if args.kernel == "pair":
        for what in (("forward", "backward") if args.what == "both" else (args.what,)):
            trace_pair(lib, torch, lf_inputs, np, args.N, args.B, what, args.delta_math)
        return
    for name in (sorted(KERNELS) if args.kernel == "all" else [args.kernel]):
        trace(lib, torch, lf_inputs, np, name, args.L, args.N, args.k)


if __name__ == "__main__":
    main()
