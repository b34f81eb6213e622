"""GPU-side behaviour of the C ABI other than numerics: argument errors, options, the
bounded device-side waits and the host-buffer entry point."""
import numpy as np
import pytest
import torch

import lf_inputs
import paper_1801_04928_b200 as lf
from lf_testlib import compare_all, gpu_pass, oracle_pass

pytestmark = pytest.mark.gpu


def _buffers(L, N, B=1):
    t = {k: v.cuda() for k, v in lf_inputs.make_inputs(L, N, B, "uniform", 7, "cpu").items()}
    t["z"] = torch.empty((L, B, N), device="cuda"); t["a"] = torch.empty((L + 1, B, N), device="cuda")
    t["delta"] = torch.empty((L, B, N), device="cuda")
    t["gw"] = torch.empty((L, N, N), device="cuda"); t["gb"] = torch.empty((L, N), device="cuda")
    return t


def test_argument_errors():
    L, N = 3, 64
    t = _buffers(L, N)
    rc, h = lf.lf_create(L, N, 1, 2)
    assert rc == lf.LF_OK
    try:
        assert lf.lf_forward(h, None, t["b"], t["x"], t["z"], t["a"]) == lf.LF_ENULL
        assert lf.lf_forward(h, t["w"].data_ptr() + 4, t["b"], t["x"], t["z"], t["a"]) == lf.LF_EALIGN
        assert lf.lf_backward(h, t["w"], t["z"], t["a"], t["y"], t["delta"], None, t["gb"]) == lf.LF_ENULL
        assert lf.lf_backward(h, t["w"], t["z"], t["a"], t["y"], t["delta"].data_ptr() + 8, t["gw"],
                              t["gb"]) == lf.LF_EALIGN
        assert lf.lf_set_option(h, 99, 1) == lf.LF_EINVAL
        assert lf.lf_set_option(h, lf.LF_OPT_VARIANT, 7) == lf.LF_EINVAL
        assert lf.lf_set_option(h, lf.LF_OPT_WAIT_BUDGET_US, 0) == lf.LF_EINVAL
        assert lf.lf_owner(h, 0) == -1 and lf.lf_owner(h, L + 1) == -1
        assert [lf.lf_owner(h, l) for l in (3, 2, 1)] == [0, 1, 0]   # (L - l) mod k
        assert lf.lf_sync(h) == lf.LF_OK
    finally:
        assert lf.lf_destroy(h) == lf.LF_OK


@pytest.mark.parametrize("variant", [lf.LF_VARIANT_FUSED, lf.LF_VARIANT_PERSISTENT])
def test_bounded_waits_expire_and_the_context_recovers(variant):
    # One CTA withholds its share of delta: every wait that depends on it must run out after
    # the budget, the kernel must end, lf_sync must say LF_ETIMEOUT, and the next call (hook
    # off) must be correct again.
    L, N = 6, 1024
    cfg = dict(L=L, N=N, B=1, k=2)
    t = _buffers(L, N)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with lf.Leapfrog(L, N, 1, 2, stream=st.cuda_stream) as ctx:
        ctx.set_option(lf.LF_OPT_VARIANT, variant)
        ctx.set_option(lf.LF_OPT_WAIT_BUDGET_US, 20000)
        ctx.forward(t["w"], t["b"], t["x"], t["z"], t["a"])
        ctx.sync()
        ctx.set_option(lf.LF_OPT_WITHHOLD, 1)
        ctx.backward(t["w"], t["z"], t["a"], t["y"], t["delta"], t["gw"], t["gb"])
        rc = lf.lf_sync(ctx._h)
        assert rc == lf.LF_ETIMEOUT, lf.lf_strerror(rc)
        assert ctx.stats()["device_status"] != 0
        ctx.set_option(lf.LF_OPT_WITHHOLD, 0)
        ctx.backward(t["w"], t["z"], t["a"], t["y"], t["delta"], t["gw"], t["gb"])
        ctx.sync()
        assert ctx.stats()["device_status"] == 0
    torch.cuda.synchronize()
    ref = oracle_pass(t)
    compare_all(cfg, {k: t[k] for k in ("z", "a", "delta", "gw", "gb")}, ref)


@pytest.mark.parametrize("N,B,tiling", [(256, 32, lf.LF_TC_TILING_ONE_SM), (512, 96, lf.LF_TC_TILING_ONE_SM),
                                        (512, 64, lf.LF_TC_TILING_TWO_SM), (772, 320, lf.LF_TC_TILING_TWO_SM)])
def test_tensor_core_kernels_give_up_cleanly(N, B, tiling):
    # LF_OPT_WITHHOLD = 2: one producer of the weight-gradient kernel arms a stage and never loads it,
    # so the multiplications behind it never start and every wait runs out (budget 20 ms).  The
    # kernel must end -- the one-SM kernel, the CTA pairs with the delta operand resident (B <= 256)
    # and with both operands streaming --, lf_sync must say LF_ETIMEOUT, and the next call must be
    # right again: Eq. bp4 against the oracle.
    from oracle import lf_oracle as orc
    from lf_testlib import rel_frobenius, TF32_TOL
    g = torch.Generator(device="cuda"); g.manual_seed(N + B)
    d = torch.empty((B, N), device="cuda").normal_(0.0, 1.0, generator=g)
    a = torch.empty((B, N), device="cuda").uniform_(0.0, 1.0, generator=g)
    gw = torch.full((N, N), float("nan"), device="cuda")
    with lf.Leapfrog(1, N, B, 1) as ctx:
        ctx.set_option(lf.LF_OPT_GW_MATH, lf.LF_GW_MATH_TF32)
        ctx.set_option(lf.LF_OPT_TC_TILING, tiling)
        ctx.set_option(lf.LF_OPT_WAIT_BUDGET_US, 20000)
        ctx.set_option(lf.LF_OPT_WITHHOLD, 2)
        ctx.grad_w(d, a, gw)
        assert lf.lf_sync(ctx._h) == lf.LF_ETIMEOUT
        assert ctx.stats()["device_status"] != 0 and ctx.stats()["gw_tiling"] == tiling
        ctx.set_option(lf.LF_OPT_WITHHOLD, 0)
        gw.fill_(float("nan"))
        ctx.grad_w(d, a, gw)
        ctx.sync()
        assert ctx.stats()["device_status"] == 0
    ref = orc.grad_w(d.double().cpu().numpy(), a.double().cpu().numpy())
    assert rel_frobenius(gw.cpu().numpy(), ref) <= TF32_TOL


def test_host_buffer_entry_point_matches_device_path():
    L, N = 4, 516
    cfg = dict(L=L, N=N, B=1, k=2)
    t = _buffers(L, N)
    out, _ = gpu_pass(cfg, t, variant=lf.LF_VARIANT_STREAMS)   # the host entry pipelines the per-layer schedule
    host = {k: out[k].cpu() if k in ("z", "a") else t[k].cpu() for k in ("w", "z", "a", "y")}
    res = {k: torch.empty_like(out[k], device="cpu").pin_memory() for k in ("delta", "gw", "gb")}
    with lf.Leapfrog(L, N, 1, 2) as ctx:
        ctx.backward_host(host["w"], host["z"], host["a"], host["y"], res["delta"], res["gw"], res["gb"])
        ctx.sync()
        assert ctx.stats()["workspace_bytes"] > 4 * 2 * L * N * N
    for k in ("delta", "gw", "gb"):
        assert torch.equal(res[k], out[k].cpu())
    ref = oracle_pass(t)
    compare_all(cfg, dict(z=out["z"], a=out["a"], **{k: v.cuda() for k, v in res.items()}), ref)


def test_last_backward_time_is_reported_when_asked_for():
    # LF_OPT_TIME_CALLS: two events around the call on the context's stream; lf_sync reads them
    L, N = 8, 1024
    t = _buffers(L, N)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with lf.Leapfrog(L, N, 1, 2, stream=st.cuda_stream) as ctx:
        ctx.forward(t["w"], t["b"], t["x"], t["z"], t["a"])
        ctx.backward(t["w"], t["z"], t["a"], t["y"], t["delta"], t["gw"], t["gb"])
        ctx.sync()
        assert ctx.stats()["last_backward_ms"] == 0.0            # off by default
        ctx.set_option(lf.LF_OPT_TIME_CALLS, 1)
        for variant in (lf.LF_VARIANT_STREAMS, lf.LF_VARIANT_AUTO):
            ctx.set_option(lf.LF_OPT_VARIANT, variant)
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(st)
            ctx.backward(t["w"], t["z"], t["a"], t["y"], t["delta"], t["gw"], t["gb"])
            e1.record(st)
            ctx.sync()
            ms = ctx.stats()["last_backward_ms"]
            assert 0.0 < ms <= e0.elapsed_time(e1) + 1e-3, (variant, ms, e0.elapsed_time(e1))
    torch.cuda.synchronize()


def test_binding_refuses_buffers_of_the_wrong_size_or_type():
    L, N = 3, 64
    t = _buffers(L, N)
    with lf.Leapfrog(L, N, 1, 2) as ctx:
        small = torch.empty((L, N, N - 4), device="cuda")
        for bad in (small, t["gw"].double(), t["gw"].cpu(), t["gw"].transpose(1, 2)):
            with pytest.raises(lf.LeapfrogError) as e:
                ctx.backward(t["w"], t["z"], t["a"], t["y"], t["delta"], bad, t["gb"])
            assert e.value.status == lf.LF_EINVAL
        with pytest.raises(lf.LeapfrogError):
            ctx.backward_host(t["w"], t["z"], t["a"], t["y"], t["delta"], t["gw"], t["gb"])   # device tensors
