"""GPU parity of lf_backward_sgd (the backward pass fused with a gradient-descent step on the
weights) against the float64 oracle: w_new = w - eta * gw with gw from the oracle's Eq. bp4.
The paper has no such step; the oracle's definition of it is pinned in test_oracle_pins.py."""
import numpy as np
import pytest
import torch

import lf_inputs
import paper_1801_04928_b200 as lf
from lf_testlib import FP32_TOL, TF32_TOL, compare_all, oracle_pass
from oracle import lf_oracle as orc

pytestmark = pytest.mark.gpu

VARIANTS = [lf.LF_VARIANT_STREAMS, lf.LF_VARIANT_PERSISTENT, lf.LF_VARIANT_FUSED]


def _inputs(L, N, B, y="uniform", seed=1):
    cpu = lf_inputs.make_inputs(L, N, B, y, lf_inputs.SEED_BASE + 300 + seed, "cpu")
    return {k: v.cuda() for k, v in cpu.items()}


def _sgd_pass(cfg, t, eta, variant=lf.LF_VARIANT_AUTO, gw_math=lf.LF_GW_MATH_AUTO, tc_tiling=0, also_plain=False):
    """lf_forward + lf_backward_sgd (and, if asked, lf_backward before and after it on the same
    context and buffers).  Returns dict of device tensors and stats."""
    L, N, B = cfg["L"], cfg["N"], cfg["B"]
    dev = t["w"].device
    z = torch.empty((L, B, N), device=dev); a = torch.empty((L + 1, B, N), device=dev)
    delta = torch.full((L, B, N), float("nan"), device=dev)
    w_new = torch.full((L, N, N), float("nan"), device=dev)
    gw = torch.full((L, N, N), float("nan"), device=dev)
    gb = torch.full((L, N), float("nan"), device=dev)
    st = torch.cuda.Stream(device=dev)
    st.wait_stream(torch.cuda.current_stream(dev))
    out = {}
    with lf.Leapfrog(L, N, B, cfg["k"], stream=st.cuda_stream) as ctx:
        ctx.set_option(lf.LF_OPT_VARIANT, variant)
        ctx.set_option(lf.LF_OPT_GW_MATH, gw_math)
        ctx.set_option(lf.LF_OPT_TC_TILING, tc_tiling)
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        if also_plain:
            ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
            ctx.sync()
            out["gw_before"] = gw.clone()
        ctx.backward_sgd(t["w"], z, a, t["y"], eta, delta, w_new, gb)
        ctx.sync()
        stats = ctx.stats()
        if also_plain:
            with torch.cuda.stream(st):
                gw.fill_(float("nan"))
            ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
            ctx.sync()
            out["gw_after"] = gw
    torch.cuda.current_stream(dev).wait_stream(st)
    torch.cuda.synchronize(dev)
    out.update(z=z, a=a, delta=delta, w_new=w_new, gb=gb)
    return out, stats


def _check_update(t, out, ref, eta, tf32=False):
    """Per layer: |w_new - (w - eta gw_ref)| within the gradient's own gate scaled by eta, plus
    one rounding of the result."""
    w = t["w"].cpu().numpy()
    want = orc.sgd_step(w, ref["gw"], eta)
    got = out["w_new"].cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    for l in range(w.shape[0]):
        round_off = 2.0 ** -23 * float(np.max(np.abs(want[l])))
        if tf32:
            err = float(np.linalg.norm(got[l] - want[l]))
            bound = abs(eta) * TF32_TOL * float(np.linalg.norm(ref["gw"][l])) + round_off * w.shape[1]
        else:
            err = float(np.max(np.abs(got[l] - want[l])))
            bound = abs(eta) * FP32_TOL * float(np.max(np.abs(ref["gw"][l]))) + round_off
        assert err <= bound, (l, err, bound)


def _assert_is_fma_of(w_new, w, gw, eta):
    # fma(-eta, gw, w) evaluated in float64 and rounded to fp32: identical to the fp32 fused
    # multiply-add except where the float64 sum lands within 2^-29 of a rounding boundary
    # (double rounding), so allow a handful of one-ulp differences.
    eta32 = float(np.float32(eta))
    want = (w.double() - eta32 * gw.double()).float()
    bad = w_new != want
    n_bad = int(bad.sum())
    assert n_bad <= max(2, w_new.numel() // 10_000_000), n_bad
    if n_bad:
        assert torch.allclose(w_new[bad], want[bad], rtol=2.0 ** -22, atol=0.0)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("L,N,k", [(1, 4, 1), (3, 64, 2), (5, 260, 4), (4, 516, 16), (3, 1156, 2), (3, 3072, 2)])
def test_single_sample_sgd_parity(L, N, k, variant):
    cfg = dict(L=L, N=N, B=1, k=k)
    t = _inputs(L, N, 1, seed=L * 1000 + N)
    eta = 0.37
    out, stats = _sgd_pass(cfg, t, eta, variant=variant, also_plain=True)
    assert stats["variant"] == variant and stats["device_status"] == 0
    ref = oracle_pass(t, want_gw=True)
    compare_all(cfg, dict(out, gw=out["gw_after"]), ref)      # delta, gb (and the plain gw afterwards)
    _check_update(t, out, ref, eta)
    # the plain call gives the same gradients before and after the fused one (no state leaks) ...
    assert torch.equal(out["gw_before"], out["gw_after"])
    # ... and the fused result is one fused multiply-add of exactly those gradients
    _assert_is_fma_of(out["w_new"], t["w"], out["gw_after"], eta)


@pytest.mark.parametrize("variant", VARIANTS)
def test_update_does_not_depend_on_k(variant):
    # Theorem 1 carried over to the fused step: the schedule changes who writes a layer, never
    # what is written, so the updated weights are bitwise the same for every k.
    L, N = 5, 1028
    t = _inputs(L, N, 1, seed=11)
    base = _sgd_pass(dict(L=L, N=N, B=1, k=1), t, -0.05, variant=variant)[0]["w_new"]
    for k in (2, 3, 7):
        assert torch.equal(_sgd_pass(dict(L=L, N=N, B=1, k=k), t, -0.05, variant=variant)[0]["w_new"], base), k


@pytest.mark.parametrize("gw_math,tiling", [(lf.LF_GW_MATH_FP32, 0), (lf.LF_GW_MATH_TF32, lf.LF_TC_TILING_ONE_SM),
                                            (lf.LF_GW_MATH_TF32, lf.LF_TC_TILING_TWO_SM)])
@pytest.mark.parametrize("L,N,B,k", [(2, 68, 3, 2), (3, 512, 256, 2), (2, 388, 70, 2), (2, 1028, 129, 3)])
def test_minibatch_sgd_parity(L, N, B, k, gw_math, tiling):
    cfg = dict(L=L, N=N, B=B, k=k)
    t = _inputs(L, N, B, y="onehot", seed=7 * N + B)
    eta = 0.01
    out, stats = _sgd_pass(cfg, t, eta, gw_math=gw_math, tc_tiling=tiling, also_plain=True)
    assert stats["gw_math"] == gw_math and stats["device_status"] == 0
    ref = oracle_pass(t, want_gw=True)
    _check_update(t, out, ref, eta, tf32=gw_math == lf.LF_GW_MATH_TF32)
    assert torch.equal(out["gw_before"], out["gw_after"])
    _assert_is_fma_of(out["w_new"], t["w"], out["gw_after"], eta)


def test_sgd_rejects_overlap_and_bad_eta():
    L, N = 2, 64
    t = _inputs(L, N, 1, seed=2)
    z = torch.empty((L, 1, N), device="cuda"); a = torch.empty((L + 1, 1, N), device="cuda")
    delta = torch.empty((L, 1, N), device="cuda"); gb = torch.empty((L, N), device="cuda")
    both = torch.empty((2 * L, N, N), device="cuda")
    with lf.Leapfrog(L, N, 1, 1) as ctx:
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        assert lf.lf_backward_sgd(ctx._h, t["w"], z, a, t["y"], 0.1, delta, t["w"], gb) == lf.LF_EINVAL
        both[:L].copy_(t["w"])
        assert lf.lf_backward_sgd(ctx._h, both[:L], z, a, t["y"], 0.1, delta, both[1:L + 1], gb) == lf.LF_EINVAL
        assert lf.lf_backward_sgd(ctx._h, t["w"], z, a, t["y"], float("nan"), delta, both[:L], gb) == lf.LF_EINVAL
        assert lf.lf_backward_sgd(ctx._h, t["w"], z, a, t["y"], float("inf"), delta, both[:L], gb) == lf.LF_EINVAL
        assert lf.lf_backward_sgd(ctx._h, both[:L], z, a, t["y"], 0.1, delta, both[L:], gb) == lf.LF_OK   # adjacent is fine
        ctx.sync()
