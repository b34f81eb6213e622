"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI binding, run
the oracle on a host copy of the same inputs, and compare tensor by tensor, layer by layer."""
from __future__ import annotations

import numpy as np
import torch

import paper_1801_04928_b200 as lf
from oracle import lf_oracle as orc

FP32_TOL = 1e-5      # max|diff| / max|ref| per tensor per layer, fp32 CUDA-core paths
TF32_TOL = 5e-3      # relative Frobenius error, TF32 tensor-core weight gradients
DENORMAL = 2.0 ** -149


GUARD = 256                      # floats of sentinel on either side of every output buffer
_SENTINEL = -0x12345679          # an int32 bit pattern no result takes by accident (a NaN with a payload)


class Guarded:
    """An output tensor with a guard band on each side: `t` is what the library gets (NaN-filled),
    `check()` says whether anything wrote outside it."""

    def __init__(self, shape, device, fill=float("nan")):
        n = int(np.prod(shape))
        self.raw = torch.empty(n + 2 * GUARD, dtype=torch.float32, device=device)
        self.raw.view(torch.int32).fill_(_SENTINEL)
        self.t = self.raw[GUARD:GUARD + n].view(shape)
        self.t.fill_(fill)

    def check(self, name):
        g = self.raw.view(torch.int32)
        lo, hi = g[:GUARD], g[-GUARD:]
        assert bool((lo == _SENTINEL).all()), f"{name}: something wrote below the buffer"
        assert bool((hi == _SENTINEL).all()), f"{name}: something wrote past the end of the buffer"


def gpu_pass(cfg, t, variant=lf.LF_VARIANT_AUTO, gw_math=lf.LF_GW_MATH_AUTO, k=None,
             use_graph=True, stream=None, repeat=1, delta_math=0, tc_tiling=0, cost=0, act=0,
             fused_tiling=0):
    """lf_forward + lf_backward on device tensors t (w,b,x,y).  Returns dict of device tensors
    and the stats of the context."""
    L, N, B = cfg["L"], cfg["N"], cfg["B"]
    k = cfg["k"] if k is None else k
    dev = t["w"].device
    # every output sits between two guard bands that are checked after the pass
    guards = dict(z=Guarded((L, B, N), dev), a=Guarded((L + 1, B, N), dev), delta=Guarded((L, B, N), dev),
                  gw=Guarded((L, N, N), dev), gb=Guarded((L, N), dev))
    z, a, delta, gw, gb = (guards[n].t for n in ("z", "a", "delta", "gw", "gb"))
    st = stream if stream is not None else torch.cuda.Stream(device=dev)
    st.wait_stream(torch.cuda.current_stream(dev))
    with lf.Leapfrog(L, N, B, k, stream=st.cuda_stream) as ctx:
        ctx.set_option(lf.LF_OPT_VARIANT, variant)
        ctx.set_option(lf.LF_OPT_GW_MATH, gw_math)
        ctx.set_option(lf.LF_OPT_DELTA_MATH, delta_math)
        ctx.set_option(lf.LF_OPT_TC_TILING, tc_tiling)
        ctx.set_option(lf.LF_OPT_COST, cost)
        ctx.set_option(lf.LF_OPT_ACTIVATION, act)
        ctx.set_option(lf.LF_OPT_FUSED_TILING, fused_tiling)
        ctx.set_option(lf.LF_OPT_USE_GRAPH, 1 if use_graph else 0)
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        for _ in range(repeat):
            ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
        ctx.sync()
        stats = ctx.stats()
    torch.cuda.current_stream(dev).wait_stream(st)
    torch.cuda.synchronize(dev)
    for name, g in guards.items():
        g.check(name)
    return dict(z=z, a=a, delta=delta, gw=gw, gb=gb), stats


def oracle_pass(t, want_gw=False, cross_entropy=False):
    """Forward + sequential backward of the oracle on host copies (fp32 weights promoted)."""
    w = t["w"].detach().cpu().numpy()
    b = t["b"].detach().cpu().numpy()
    x = t["x"].detach().cpu().numpy()
    y = t["y"].detach().cpu().numpy()
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y, want_gw=want_gw, cross_entropy=cross_entropy)
    return dict(z=z, a=a, delta=delta, gw=gw, gb=gb)


def rel_max_err(got: np.ndarray, ref: np.ndarray) -> tuple[float, float]:
    """(max|got-ref| / max|ref|, max|ref|) in float64."""
    got = np.asarray(got, dtype=np.float64)
    m = float(np.max(np.abs(ref))) if ref.size else 0.0
    d = float(np.max(np.abs(got - ref))) if ref.size else 0.0
    return (d / m if m > 0 else d), m


def assert_layer_close(name, l, got, ref, tol=FP32_TOL, n_terms=1):
    """Per-layer gate: max|diff| <= tol * max|ref| + a floor for results in the fp32
    denormal range (absolute error there is a few multiples of 2^-149 per term added)."""
    got = np.asarray(got, dtype=np.float64)
    assert np.all(np.isfinite(got)), f"{name}[{l}] holds non-finite values"
    m = float(np.max(np.abs(ref)))
    d = float(np.max(np.abs(got - ref)))
    bound = tol * m + 4.0 * n_terms * DENORMAL
    assert d <= bound, f"{name}[{l}]: max|diff| {d:.3e} > {bound:.3e} (max|ref| {m:.3e}, rel {d / max(m, 1e-300):.3e})"
    if m < 1e3 * 1.1754944e-38:   # layer lives in (or next to) the fp32 denormal range:
        return 0.0                #   gated by the absolute floor, not counted as a relative figure
    return d / m


def rel_frobenius(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    den = float(np.linalg.norm(ref))
    return float(np.linalg.norm(got - ref)) / den if den > 0 else float(np.linalg.norm(got - ref))


def compare_all(cfg, out, ref, gw_tf32=False):
    """Element-by-element parity of z, a, delta, gb and gw for every layer.  ref['gw'] may be
    None: then each layer's gw is formed by the oracle's Eq. bp4 on the fly."""
    L, N, B = cfg["L"], cfg["N"], cfg["B"]
    worst = {}
    for name in ("z", "a", "delta", "gb"):
        g = out[name].cpu().numpy()
        r = ref[name]
        w = 0.0
        for l in range(r.shape[0]):
            w = max(w, assert_layer_close(name, l, g[l], r[l], n_terms=N))
        worst[name] = w
    w = 0.0
    for l in range(L):
        r = ref["gw"][l] if ref.get("gw") is not None else orc.grad_w(ref["delta"][l], ref["a"][l])
        g = out["gw"][l].cpu().numpy()
        if gw_tf32:
            assert np.all(np.isfinite(g))
            e = rel_frobenius(g, r)
            assert e <= TF32_TOL, f"gw[{l}]: relative Frobenius error {e:.3e} > {TF32_TOL}"
            w = max(w, e)
        else:
            w = max(w, assert_layer_close("gw", l, g, r, n_terms=N + B))  # inherits delta's absolute error
    worst["gw"] = w
    return worst
