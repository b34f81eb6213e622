"""GPU parity at the largest widths and batches of the sweep grid (N = 8192; B = 1024), at a
reduced depth so that the float64 oracle still finishes in seconds.

Single sample: the whole pass is compared element by element (the weight gradient one layer at a
time).  Mini-batch: samples never mix before Eq. bp3/bp4, so the oracle runs the whole chain on a
few sample columns; gb, which sums over all samples, is compared in full; for gw the oracle's
Eq. bp4 is applied to the GPU's own delta and activations on a grid of rows and columns chosen so
that every 256 x 256 output tile holds some hundred entries of it, plus sampled single entries.
"""
import numpy as np
import pytest
import torch

import lf_inputs
import paper_1801_04928_b200 as lf
from lf_testlib import (TF32_TOL, assert_layer_close, compare_all, gpu_pass, oracle_pass,
                        rel_frobenius)
from oracle import lf_oracle as orc

pytestmark = pytest.mark.gpu


def _inputs(L, N, B, y, seed):
    return lf_inputs.make_inputs(L, N, B, y, lf_inputs.SEED_BASE + lf_inputs.SWEEP_CONFIG_INDEX * 1000 + seed,
                                 "cuda")


@pytest.mark.parametrize("variant", [lf.LF_VARIANT_STREAMS, lf.LF_VARIANT_PERSISTENT, lf.LF_VARIANT_FUSED])
def test_width_8192_single_sample(variant):
    # N = 8192, B = 1: the widest plan of the single-launch kernels (2048 tile rows per CTA in the
    # fused pass, two column blocks per strip on the leapfrog groups' chain).
    L, N = 3, 8192
    cfg = dict(L=L, N=N, B=1, k=2)
    t = _inputs(L, N, 1, "uniform", 1)
    out, stats = gpu_pass(cfg, t, variant=variant)
    assert stats["variant"] == variant and stats["device_status"] == 0
    worst = compare_all(cfg, out, oracle_pass(t))
    assert torch.equal(out["gb"], out["delta"][:, 0])
    print("N=8192 B=1 variant", variant, worst)


def _sampled_minibatch_parity(L, N, B, tiling, seed, n_chain=3, grid=512):
    cfg = dict(L=L, N=N, B=B, k=2)
    t = _inputs(L, N, B, "onehot", seed)
    out, stats = gpu_pass(cfg, t, tc_tiling=tiling)
    # the library's own choice for Eq. bp4: up to 16 samples the fp32 store stream, beyond that TF32 tensor cores
    assert stats["gw_math"] == (lf.LF_GW_MATH_FP32 if B <= 16 else lf.LF_GW_MATH_TF32) and stats["device_status"] == 0
    tol = 2e-5 if B <= 16 else TF32_TOL      # the fp32 writer is held to fp32 level
    # CTA pairs serve more than 128 samples; below that one CTA per tile (from a width of 4096 the
    # warp-specialised kernel on single CTAs)
    if tiling == lf.LF_TC_TILING_TWO_SM and B > 128:
        assert stats["delta_tiling"] == lf.LF_TC_TILING_TWO_SM
    if B <= 128:
        assert stats["delta_tiling"] == lf.LF_TC_TILING_ONE_SM
    # the library's own choice: a handful of samples (up to 8, or up to 16 from a width of 2048) keeps Eq. bp2 in fp32 on the CUDA cores
    assert stats["delta_math"] == (lf.LF_DELTA_MATH_FP32 if (B <= 8 or (B <= 16 and N >= 2048)) else lf.LF_DELTA_MATH_3XTF32)

    # (i) the chain, for a few samples spread over the 256-sample blocks (first, last, inside)
    sel = sorted({0, B - 1, (5 * B) // 8 + 1})[:n_chain]
    w = t["w"].cpu().numpy()
    z, a = orc.forward(w, t["b"].cpu().numpy(), t["x"][sel].cpu().numpy())
    delta, _, _ = orc.backward_sequential(w, z, a, t["y"][sel].cpu().numpy(), want_gw=False)
    for name, ref in (("z", z), ("a", a), ("delta", delta)):
        g = out[name][:, sel].cpu().numpy()
        for l in range(ref.shape[0]):
            assert_layer_close(name, l, g[l], ref[l], n_terms=N)

    # (ii) Eq. bp3 in full; Eq. bp4 on a grid of M x M entries -- M/blocks rows and as many
    # columns drawn inside every 256-wide block, so every 256 x 256 output tile holds
    # (M/blocks)^2 of them -- and on single entries drawn anywhere
    d_gpu = out["delta"].cpu().numpy().astype(np.float64)
    a_gpu = out["a"].cpu().numpy().astype(np.float64)
    rng = np.random.default_rng(seed)
    blocks = N // 256
    per = grid // blocks
    rows = np.concatenate([256 * q + np.sort(rng.choice(256, per, replace=False)) for q in range(blocks)])
    cols = np.concatenate([256 * q + np.sort(rng.choice(256, per, replace=False)) for q in range(blocks)])
    rows[0], rows[-1], cols[0], cols[-1] = 0, N - 1, 0, N - 1
    for l in range(L):
        assert_layer_close("gb", l, out["gb"][l].cpu().numpy(), orc.grad_b(d_gpu[l]), n_terms=B)
        g = out["gw"][l].cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(g)), l
        # the oracle's Eq. bp4 on the selected neurons of layer l (rows) and l-1 (columns)
        ref = orc.grad_w(np.ascontiguousarray(d_gpu[l][:, rows]), np.ascontiguousarray(a_gpu[l][:, cols]))
        got = g[np.ix_(rows, cols)]
        e = rel_frobenius(got, ref)
        assert e <= tol, ("grid", l, e)
        # tile by tile as well: a wrong tile must not hide in the whole-matrix norm
        gt = (got - ref).reshape(blocks, per, blocks, per)
        rt = ref.reshape(blocks, per, blocks, per)
        et = np.sqrt((gt * gt).sum(axis=(1, 3)) / (rt * rt).sum(axis=(1, 3)))
        assert float(et.max()) <= 4 * tol, ("tile", l, np.unravel_index(et.argmax(), et.shape), et.max())
        rms = np.sqrt(np.mean(g * g))
        for _ in range(32):
            j, k = int(rng.integers(N)), int(rng.integers(N))
            r1 = orc.grad_w_entry(d_gpu[l], a_gpu[l], j, k)
            assert abs(g[j, k] - r1) <= tol * max(abs(r1), rms), (l, j, k, g[j, k], r1)
    return stats


@pytest.mark.parametrize("tiling", [lf.LF_TC_TILING_ONE_SM, lf.LF_TC_TILING_TWO_SM])
@pytest.mark.parametrize("N,B", [(8192, 16), (8192, 128), (4096, 1024), (8192, 1024)])
def test_sweep_grid_minibatch_corners(N, B, tiling):
    # The grid's largest width with a small, a middle and the largest batch, and the largest batch
    # at the middle width: B = 1024 is four 256-sample blocks in the two-SM delta kernel and 32
    # contraction stages per tile in the weight-gradient kernels.
    stats = _sampled_minibatch_parity(2, N, B, tiling, seed=N // 64 + B)
    print("sweep corner", N, B, "tiling", tiling, "delta_tiling", stats["delta_tiling"],
          "gw_tiling", stats["gw_tiling"])
