"""The allocation-free delta step, `lf_delta_step_static`.

Some users of the library cannot let it call cudaMalloc: a server that gave the whole GPU to
its own memory pool, or a loop that cannot take the device-wide stall of an allocation.  For
them the library has one entry point whose scratch is a fixed array in the library image.
This file checks, through the C ABI, that it returns what the ordinary path (`lf_backward`,
which uses a context's allocated workspace) returns for the same layer -- on two calls in a
row, because the calls share the array and the second one meets the first one's leftovers --
and what the oracle's Eq. bp2 gives for the same inputs; and that, once the first call on the
device has been made, further calls leave the amount of free device memory exactly as it was.
It is named to be collected last, so a failure here cannot hide any other test's result.
"""
import numpy as np
import pytest
import torch

import lf_inputs
import paper_1801_04928_b200 as lf
from oracle import lf_oracle as orc

pytestmark = pytest.mark.gpu

TOL = 1e-5  # max|diff| / max|ref|, the gate of the fp32 parity tests


def _reference_pass(L, N, seed):
    cpu = lf_inputs.make_inputs(L, N, 1, "uniform", lf_inputs.SEED_BASE + seed, "cpu")
    t = {k: v.cuda() for k, v in cpu.items()}
    z = torch.empty((L, 1, N), device="cuda"); a = torch.empty((L + 1, 1, N), device="cuda")
    delta = torch.empty((L, 1, N), device="cuda")
    gw = torch.empty((L, N, N), device="cuda"); gb = torch.empty((L, N), device="cuda")
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with lf.Leapfrog(L, N, 1, 2, stream=stream.cuda_stream) as ctx:
        ctx.set_option(lf.LF_OPT_VARIANT, lf.LF_VARIANT_STREAMS)
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
        ctx.sync()
    torch.cuda.synchronize()
    return t, a, delta


@pytest.mark.parametrize("N", [516, 2048, 4096])
def test_static_delta_step_matches_lf_backward_twice_in_a_row(N):
    L = 3
    t, a, delta = _reference_pass(L, N, seed=900 + N)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    outs = []
    for l in (2, 1):  # two calls back to back on one stream: delta^2 from delta^3, delta^1 from delta^2
        out = torch.full((N,), float("nan"), device="cuda")
        stream.wait_stream(torch.cuda.current_stream())
        rc = lf.lf_delta_step_static(t["w"][l], delta[l, 0], a[l, 0], out, N, stream.cuda_stream)
        assert rc == lf.LF_OK, lf.lf_strerror(rc)
        outs.append((l, out))
    stream.synchronize()
    for l, out in outs:
        ref = delta[l - 1, 0]
        assert torch.isfinite(out).all()
        err = (out.double() - ref.double()).abs().max().item()
        scale = ref.double().abs().max().item()
        assert err <= TOL * scale, (N, l, err, scale)
        # and the oracle's Eq. bp2 on the same inputs (sigma' from z; a = sigma(z) went to the GPU)
        a_l = a[l, 0].double().cpu().numpy()
        z_l = np.log(a_l) - np.log1p(-a_l)
        want = orc.delta_step(t["w"][l].cpu().numpy(), delta[l].double().cpu().numpy(), z_l[None, :])[0]
        err = float(np.max(np.abs(out.double().cpu().numpy() - want)))
        assert err <= TOL * float(np.max(np.abs(want))), (N, l, err)


def test_static_delta_step_leaves_free_memory_alone_after_the_first_call():
    # The first call on a device may load the library's code and its scratch array onto it; every
    # call after that must not change the amount of free device memory by a single byte.
    N = 1024
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    w = torch.empty((N, N), device="cuda").normal_(0.0, N ** -0.5, generator=g)
    d_up = torch.empty((N,), device="cuda").normal_(0.0, 1.0, generator=g)
    a_l = torch.empty((N,), device="cuda").uniform_(0.05, 0.95, generator=g)
    out = torch.empty((N,), device="cuda")
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    assert lf.lf_delta_step_static(w, d_up, a_l, out, N, stream.cuda_stream) == lf.LF_OK   # warm-up
    stream.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(5):
        assert lf.lf_delta_step_static(w, d_up, a_l, out, N, stream.cuda_stream) == lf.LF_OK
    stream.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    want = (w.double().t() @ d_up.double()) * a_l.double() * (1 - a_l.double())
    assert float((out.double() - want).abs().max()) <= TOL * float(want.abs().max())


def test_static_delta_step_rejects_what_it_cannot_hold():
    buf = torch.zeros(64, device="cuda")
    assert lf.lf_delta_step_static(buf, buf, buf, buf, 4100) == lf.LF_ECAPACITY
    assert lf.lf_delta_step_static(buf, buf, buf, buf, 8192) == lf.LF_ECAPACITY
    assert lf.lf_delta_step_static(buf, buf, buf, buf, 6) == lf.LF_EINVAL
    assert lf.lf_delta_step_static(None, buf, buf, buf, 64) == lf.LF_ENULL
    assert lf.lf_delta_step_static(buf.data_ptr() + 4, buf, buf, buf, 8) == lf.LF_EALIGN
    assert "capacity" in lf.lf_strerror(lf.LF_ECAPACITY)
