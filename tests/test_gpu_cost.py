"""GPU parity under the cross-entropy cost (LF_OPT_COST): Eq. bp1 with grad_a C of the
cross-entropy, everything below it unchanged.  The oracle applies Eq. bp1 as printed
(grad_a C times sigma'); the kernels use the collapsed form a^L - y."""
import pytest
import torch

import lf_inputs
import paper_1801_04928_b200 as lf
from lf_testlib import compare_all, gpu_pass, oracle_pass

pytestmark = pytest.mark.gpu

VARIANTS = [lf.LF_VARIANT_STREAMS, lf.LF_VARIANT_PERSISTENT, lf.LF_VARIANT_FUSED]


def _inputs(L, N, B, y, seed):
    cpu = lf_inputs.make_inputs(L, N, B, y, lf_inputs.SEED_BASE + 400 + seed, "cpu")
    return {k: v.cuda() for k, v in cpu.items()}


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("L,N,k,y", [(1, 8, 1, "onehot"), (3, 64, 2, "uniform"), (5, 516, 3, "onehot"), (4, 1156, 2, "uniform")])
def test_single_sample_cross_entropy_parity(L, N, k, y, variant):
    cfg = dict(L=L, N=N, B=1, k=k)
    t = _inputs(L, N, 1, y, seed=L * 100 + N)
    out, stats = gpu_pass(cfg, t, variant=variant, cost=lf.LF_COST_CROSS_ENTROPY)
    assert stats["variant"] == variant and stats["cost"] == lf.LF_COST_CROSS_ENTROPY and stats["device_status"] == 0
    compare_all(cfg, out, oracle_pass(t, cross_entropy=True))
    # the option really changes Eq. bp1: the quadratic pass on the same inputs differs at the top
    quad, qstats = gpu_pass(cfg, t, variant=variant)
    assert qstats["cost"] == lf.LF_COST_QUADRATIC
    assert not torch.equal(quad["delta"][L - 1], out["delta"][L - 1])
    compare_all(cfg, quad, oracle_pass(t))


@pytest.mark.parametrize("delta_math", [lf.LF_DELTA_MATH_FP32, lf.LF_DELTA_MATH_3XTF32])
@pytest.mark.parametrize("L,N,B,k", [(2, 68, 3, 2), (3, 516, 130, 2), (2, 388, 70, 1)])
def test_minibatch_cross_entropy_parity(L, N, B, k, delta_math):
    cfg = dict(L=L, N=N, B=B, k=k)
    t = _inputs(L, N, B, "onehot", seed=N + B)
    out, stats = gpu_pass(cfg, t, gw_math=lf.LF_GW_MATH_FP32, delta_math=delta_math, cost=lf.LF_COST_CROSS_ENTROPY)
    assert stats["cost"] == lf.LF_COST_CROSS_ENTROPY and stats["device_status"] == 0
    compare_all(cfg, out, oracle_pass(t, want_gw=True, cross_entropy=True))


def test_cost_option_rejects_unknown_values_and_survives_graph_replay():
    # the STREAMS variant replays a captured graph: switching the cost must not replay the old Eq. bp1
    L, N = 3, 260
    cfg = dict(L=L, N=N, B=1, k=2)
    t = _inputs(L, N, 1, "uniform", seed=9)
    z = torch.empty((L, 1, N), device="cuda"); a = torch.empty((L + 1, 1, N), device="cuda")
    delta = torch.empty((L, 1, N), device="cuda"); gw = torch.empty((L, N, N), device="cuda")
    gb = torch.empty((L, N), device="cuda")
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with lf.Leapfrog(L, N, 1, 2, stream=st.cuda_stream) as ctx:
        assert lf.lf_set_option(ctx._h, lf.LF_OPT_COST, 2) == lf.LF_EINVAL
        ctx.set_option(lf.LF_OPT_VARIANT, lf.LF_VARIANT_STREAMS)
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        ctx.backward(t["w"], z, a, t["y"], delta, gw, gb); ctx.sync()
        d_quad = delta.clone()
        ctx.set_option(lf.LF_OPT_COST, lf.LF_COST_CROSS_ENTROPY)
        ctx.backward(t["w"], z, a, t["y"], delta, gw, gb); ctx.sync()
        d_ce = delta.clone()
        ctx.set_option(lf.LF_OPT_COST, lf.LF_COST_QUADRATIC)
        ctx.backward(t["w"], z, a, t["y"], delta, gw, gb); ctx.sync()
    torch.cuda.synchronize()
    assert torch.equal(delta, d_quad) and not torch.equal(d_ce, d_quad)
    assert torch.equal(d_ce[L - 1, 0], a[L, 0] - t["y"][0])
