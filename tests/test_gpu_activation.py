"""GPU parity under the other activation functions (LF_OPT_ACTIVATION): tanh and the rectifier in
Eq. a, and their derivatives (taken from the stored activations) in Eq. bp1 / bp2.

For the rectifier the derivative is a yes/no decision, [z > 0].  Both sides must take it on the
same numbers, so the oracle's backward pass is given the GPU's own z and a (promoted to float64);
the forward pass is compared separately, oracle against GPU, on the same inputs."""
import numpy as np
import pytest
import torch

import lf_inputs
import paper_1801_04928_b200 as lf
from lf_testlib import compare_all, gpu_pass
from oracle import lf_oracle as orc

pytestmark = pytest.mark.gpu

VARIANTS = [lf.LF_VARIANT_STREAMS, lf.LF_VARIANT_PERSISTENT, lf.LF_VARIANT_FUSED]
ACTS = [("tanh", lf.LF_ACT_TANH), ("relu", lf.LF_ACT_RELU)]


def _inputs(L, N, B, y, seed):
    cpu = lf_inputs.make_inputs(L, N, B, y, lf_inputs.SEED_BASE + 500 + seed, "cpu")
    return {k: v.cuda() for k, v in cpu.items()}


def _reference(t, out, name, want_gw):
    """Oracle forward on the inputs; oracle backward on the GPU's own z and a."""
    w = t["w"].cpu().numpy()
    with orc.activation(name):
        z, a = orc.forward(w, t["b"].cpu().numpy(), t["x"].cpu().numpy())
        zg = out["z"].cpu().numpy().astype(np.float64); ag = out["a"].cpu().numpy().astype(np.float64)
        delta, gw, gb = orc.backward_sequential(w, zg, ag, t["y"].cpu().numpy(), want_gw=want_gw)
    return dict(z=z, a=a, delta=delta, gw=gw, gb=gb), ag


@pytest.mark.parametrize("name,act", ACTS)
@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("L,N,k", [(1, 8, 1), (4, 260, 2), (5, 1028, 3)])
def test_single_sample_activation_parity(L, N, k, variant, name, act):
    cfg = dict(L=L, N=N, B=1, k=k)
    t = _inputs(L, N, 1, "uniform", seed=L * 100 + N)
    out, stats = gpu_pass(cfg, t, variant=variant, act=act)
    assert stats["variant"] == variant and stats["activation"] == act and stats["device_status"] == 0
    ref, ag = _reference(t, out, name, want_gw=False)
    ref["gw"] = None
    # gw is formed by the oracle from its delta and the GPU's activations (what the GPU multiplied)
    ref_for_gw = dict(ref, a=ag)
    compare_all(cfg, out, dict(ref, gw=[orc.grad_w(ref["delta"][l], ref_for_gw["a"][l]) for l in range(L)]))
    if name == "relu":
        if N >= 256:
            assert float((out["a"][1:] == 0).float().mean()) > 0.2   # the rectifier really cut something off
        assert torch.all(out["delta"][out["a"][1:] == 0] == 0)   # and delta vanishes there


@pytest.mark.parametrize("name,act", ACTS)
@pytest.mark.parametrize("delta_math", [lf.LF_DELTA_MATH_FP32, lf.LF_DELTA_MATH_3XTF32])
@pytest.mark.parametrize("L,N,B,k", [(3, 132, 5, 2), (3, 516, 130, 2)])
def test_minibatch_activation_parity(L, N, B, k, delta_math, name, act):
    cfg = dict(L=L, N=N, B=B, k=k)
    t = _inputs(L, N, B, "onehot", seed=N + B)
    out, stats = gpu_pass(cfg, t, gw_math=lf.LF_GW_MATH_FP32, delta_math=delta_math, act=act)
    assert stats["activation"] == act and stats["device_status"] == 0
    ref, ag = _reference(t, out, name, want_gw=False)
    compare_all(cfg, out, dict(ref, gw=[orc.grad_w(ref["delta"][l], ag[l]) for l in range(L)]))


def test_cross_entropy_needs_the_sigmoid():
    L, N = 2, 64
    t = _inputs(L, N, 1, "uniform", seed=1)
    z = torch.empty((L, 1, N), device="cuda"); a = torch.empty((L + 1, 1, N), device="cuda")
    delta = torch.empty((L, 1, N), device="cuda"); gw = torch.empty((L, N, N), device="cuda"); gb = torch.empty((L, N), device="cuda")
    with lf.Leapfrog(L, N, 1, 1) as ctx:
        assert lf.lf_set_option(ctx._h, lf.LF_OPT_ACTIVATION, 3) == lf.LF_EINVAL
        ctx.set_option(lf.LF_OPT_ACTIVATION, lf.LF_ACT_TANH)
        ctx.set_option(lf.LF_OPT_COST, lf.LF_COST_CROSS_ENTROPY)
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        assert lf.lf_backward(ctx._h, t["w"], z, a, t["y"], delta, gw, gb) == lf.LF_EINVAL
        ctx.set_option(lf.LF_OPT_COST, lf.LF_COST_QUADRATIC)
        ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
        ctx.sync()
