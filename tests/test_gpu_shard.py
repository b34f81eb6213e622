"""GPU parity of the layer-sharded form (LF_OPT_SHARD_COUNT / LF_OPT_SHARD_RANK): the paper's
schedule on "k gpus" (Section 1).  Each shard is an independent context that runs the whole delta
chain and writes the weight gradients of its own layers only; here the S shards run one after the
other on the one GPU, writing into one gw array that was filled with NaN, and are compared with the
oracle's pass of the same shard."""
import numpy as np
import pytest
import torch

import lf_inputs
import paper_1801_04928_b200 as lf
from lf_testlib import FP32_TOL, TF32_TOL, assert_layer_close, rel_frobenius
from oracle import lf_oracle as orc

pytestmark = pytest.mark.gpu


def _inputs(L, N, B, seed):
    cpu = lf_inputs.make_inputs(L, N, B, "uniform" if B == 1 else "onehot", lf_inputs.SEED_BASE + 900 + seed, "cpu")
    return cpu, {k: v.cuda() for k, v in cpu.items()}


def _shard_pass(L, N, B, k, S, r, t, variant, bufs=None, sgd_eta=None, host=False, fp32=True):
    dev = t["w"].device
    z = torch.empty((L, B, N), device=dev); a = torch.empty((L + 1, B, N), device=dev)
    if bufs is None:
        bufs = dict(delta=torch.full((L, B, N), float("nan"), device=dev),
                    gw=torch.full((L, N, N), float("nan"), device=dev),
                    gb=torch.full((L, N), float("nan"), device=dev))
    with lf.Leapfrog(L, N, B, k) as ctx:
        ctx.set_option(lf.LF_OPT_VARIANT, variant)
        if fp32:
            ctx.set_option(lf.LF_OPT_GW_MATH, lf.LF_GW_MATH_FP32)
        ctx.set_option(lf.LF_OPT_SHARD_COUNT, S)
        ctx.set_option(lf.LF_OPT_SHARD_RANK, r)
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        if host:
            ctx.sync()
            h = {n: v.cpu().pin_memory() for n, v in dict(w=t["w"], z=z, a=a, y=t["y"], **bufs).items()}
            ctx.backward_host(h["w"], h["z"], h["a"], h["y"], h["delta"], h["gw"], h["gb"])
            ctx.sync()
            for n in ("delta", "gw", "gb"):
                bufs[n].copy_(h[n])
        elif sgd_eta is not None:
            ctx.backward_sgd(t["w"], z, a, t["y"], sgd_eta, bufs["delta"], bufs["gw"], bufs["gb"])
        else:
            ctx.backward(t["w"], z, a, t["y"], bufs["delta"], bufs["gw"], bufs["gb"])
        ctx.sync()
        stats = ctx.stats()
        owners = [ctx.owner(l) for l in range(1, L + 1)]
    torch.cuda.synchronize()
    return bufs, stats, owners


def _oracle(cpu):
    w = cpu["w"].numpy()
    z, a = orc.forward(w, cpu["b"].numpy(), cpu["x"].numpy())
    return w, z, a, cpu["y"].numpy()


@pytest.mark.parametrize("variant", [lf.LF_VARIANT_STREAMS, lf.LF_VARIANT_PERSISTENT, lf.LF_VARIANT_FUSED,
                                     lf.LF_VARIANT_AUTO])
@pytest.mark.parametrize("L,N,k,S", [(5, 260, 2, 2), (7, 516, 3, 3), (4, 1028, 1, 8), (9, 132, 4, 2)])
def test_single_sample_shards(L, N, k, S, variant):
    cpu, t = _inputs(L, N, 1, seed=L * 10 + S)
    w, z, a, y = _oracle(cpu)
    n_terms = N + 1
    union = None
    for r in range(S):
        bufs, stats, owners = _shard_pass(L, N, 1, k, S, r, t, variant)
        assert stats["device_status"] == 0 and stats["shard_count"] == S and stats["shard_rank"] == r
        if variant != lf.LF_VARIANT_AUTO:
            assert stats["variant"] == variant
        d_ref, gw_ref, gb_ref, wrote = orc.backward_shard(w, z, a, y, S, r)
        gw = bufs["gw"].cpu().numpy(); gb = bufs["gb"].cpu().numpy(); d = bufs["delta"].cpu().numpy()
        keff = min(k, L)
        for l in range(1, L + 1):
            assert_layer_close("delta", l - 1, d[l - 1], d_ref[l - 1], n_terms=n_terms)
            assert_layer_close("gb", l - 1, gb[l - 1], d_ref[l - 1, 0], n_terms=n_terms)   # B = 1: gb is delta
            if wrote[l - 1]:
                assert_layer_close("gw", l - 1, gw[l - 1], gw_ref[l - 1], n_terms=n_terms)
                assert owners[l - 1] == ((L - l) // S) % keff
            else:
                assert np.all(np.isnan(gw[l - 1])), f"shard {r} wrote layer {l} of another shard"
                assert owners[l - 1] == -1
        union = gw if union is None else np.where(np.isnan(union), gw, union)
    assert np.all(np.isfinite(union))          # together the shards wrote every layer


def test_stream_shards_are_bitwise_the_unsharded_pass():
    # same kernels, same launch shapes: what a shard writes is bit for bit the unsharded result
    L, N, k, S = 6, 516, 2, 3
    cpu, t = _inputs(L, N, 1, seed=77)
    full, _, _ = _shard_pass(L, N, 1, k, 1, 0, t, lf.LF_VARIANT_STREAMS)
    bufs = None
    for r in range(S):
        bufs, _, _ = _shard_pass(L, N, 1, k, S, r, t, lf.LF_VARIANT_STREAMS, bufs=bufs)
    for n in ("delta", "gw", "gb"):
        assert torch.equal(bufs[n], full[n])


@pytest.mark.parametrize("fp32", [True, False])
@pytest.mark.parametrize("L,N,B,k,S", [(4, 132, 5, 2, 2), (5, 516, 130, 2, 3)])
def test_minibatch_shards(L, N, B, k, S, fp32):
    cpu, t = _inputs(L, N, B, seed=L + B)
    w, z, a, y = _oracle(cpu)
    for r in range(S):
        bufs, stats, _ = _shard_pass(L, N, B, k, S, r, t, lf.LF_VARIANT_AUTO, fp32=fp32)
        assert stats["device_status"] == 0 and stats["variant"] == lf.LF_VARIANT_STREAMS
        d_ref, gw_ref, gb_ref, wrote = orc.backward_shard(w, z, a, y, S, r)
        gw = bufs["gw"].cpu().numpy(); gb = bufs["gb"].cpu().numpy(); d = bufs["delta"].cpu().numpy()
        for l in range(1, L + 1):
            assert_layer_close("delta", l - 1, d[l - 1], d_ref[l - 1], n_terms=N + B)
            if wrote[l - 1]:
                assert_layer_close("gb", l - 1, gb[l - 1], gb_ref[l - 1], n_terms=N + B)
                if fp32:
                    assert_layer_close("gw", l - 1, gw[l - 1], gw_ref[l - 1], n_terms=N + B)
                else:
                    assert rel_frobenius(gw[l - 1], gw_ref[l - 1]) <= TF32_TOL
            else:
                assert np.all(np.isnan(gw[l - 1])) and np.all(np.isnan(gb[l - 1]))


@pytest.mark.parametrize("B", [1, 6])
def test_shards_of_the_fused_update_and_of_the_host_entry_point(B):
    L, N, k, S, eta = 5, 260, 2, 2, 0.25
    cpu, t = _inputs(L, N, B, seed=50 + B)
    w, z, a, y = _oracle(cpu)
    for r in range(S):
        d_ref, gw_ref, gb_ref, wrote = orc.backward_shard(w, z, a, y, S, r)
        upd, _, _ = _shard_pass(L, N, B, k, S, r, t, lf.LF_VARIANT_AUTO, sgd_eta=eta)
        hst, _, _ = _shard_pass(L, N, B, k, S, r, t, lf.LF_VARIANT_AUTO, host=True)
        w_new = upd["gw"].cpu().numpy(); gw_h = hst["gw"].cpu().numpy(); gb_h = hst["gb"].cpu().numpy()
        for l in range(1, L + 1):
            assert_layer_close("delta", l - 1, hst["delta"].cpu().numpy()[l - 1], d_ref[l - 1], n_terms=N + B)
            if wrote[l - 1]:
                want = w[l - 1].astype(np.float64) - eta * gw_ref[l - 1]
                bound = eta * FP32_TOL * np.max(np.abs(gw_ref[l - 1])) + 2.0 ** -23 * np.max(np.abs(want))
                assert np.max(np.abs(w_new[l - 1] - want)) <= bound
                assert_layer_close("gw", l - 1, gw_h[l - 1], gw_ref[l - 1], n_terms=N + B)
                assert_layer_close("gb", l - 1, gb_h[l - 1], gb_ref[l - 1], n_terms=N + B)
            else:
                assert np.all(np.isnan(w_new[l - 1])) and np.all(np.isnan(gw_h[l - 1]))
                if B > 1:
                    assert np.all(np.isnan(gb_h[l - 1]))


@pytest.mark.parametrize("variant", [lf.LF_VARIANT_PERSISTENT, lf.LF_VARIANT_FUSED])
def test_shards_of_the_fused_update_in_the_single_launch_variants(variant):
    # the fused pass takes w from the chain's shared-memory stages; for another shard's layer it must
    # still hand every stage back without storing anything
    L, N, k, S, eta = 7, 516, 2, 3, 0.25
    cpu, t = _inputs(L, N, 1, seed=63)
    w, z, a, y = _oracle(cpu)
    for r in range(S):
        d_ref, gw_ref, gb_ref, wrote = orc.backward_shard(w, z, a, y, S, r)
        upd, stats, _ = _shard_pass(L, N, 1, k, S, r, t, variant, sgd_eta=eta)
        assert stats["variant"] == variant and stats["device_status"] == 0
        w_new = upd["gw"].cpu().numpy()
        for l in range(1, L + 1):
            assert_layer_close("delta", l - 1, upd["delta"].cpu().numpy()[l - 1], d_ref[l - 1], n_terms=N + 1)
            if wrote[l - 1]:
                want = w[l - 1].astype(np.float64) - eta * gw_ref[l - 1]
                bound = eta * FP32_TOL * np.max(np.abs(gw_ref[l - 1])) + 2.0 ** -23 * np.max(np.abs(want))
                assert np.max(np.abs(w_new[l - 1] - want)) <= bound
            else:
                assert np.all(np.isnan(w_new[l - 1]))


def test_shard_option_checks():
    with lf.Leapfrog(4, 64, 1, 2) as ctx:
        for key, value in [(lf.LF_OPT_SHARD_COUNT, 0), (lf.LF_OPT_SHARD_RANK, 1), (lf.LF_OPT_SHARD_RANK, -1)]:
            with pytest.raises(lf.LeapfrogError):
                ctx.set_option(key, value)
        ctx.set_option(lf.LF_OPT_SHARD_COUNT, 3)
        ctx.set_option(lf.LF_OPT_SHARD_RANK, 2)
        with pytest.raises(lf.LeapfrogError):
            ctx.set_option(lf.LF_OPT_SHARD_RANK, 3)
        ctx.set_option(lf.LF_OPT_SHARD_COUNT, 2)       # the rank goes back to 0
        assert ctx.owner(4) == 0 and ctx.owner(3) == -1


def test_one_context_switching_shards_recaptures_its_graph():
    # the stream schedule is replayed from a captured graph on a non-default stream; the shard is part
    # of what the graph was captured for, so changing it must not replay the old shard's launches
    L, N, k, S = 6, 260, 2, 2
    cpu, t = _inputs(L, N, 1, seed=88)
    full, _, _ = _shard_pass(L, N, 1, k, 1, 0, t, lf.LF_VARIANT_STREAMS)
    dev = t["w"].device
    z = torch.empty((L, 1, N), device=dev); a = torch.empty((L + 1, 1, N), device=dev)
    delta = torch.full((L, 1, N), float("nan"), device=dev)
    gw = torch.full((L, N, N), float("nan"), device=dev)
    gb = torch.full((L, N), float("nan"), device=dev)
    st = torch.cuda.Stream(device=dev)
    st.wait_stream(torch.cuda.current_stream(dev))
    with lf.Leapfrog(L, N, 1, k, stream=st.cuda_stream) as ctx:
        ctx.set_option(lf.LF_OPT_VARIANT, lf.LF_VARIANT_STREAMS)
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        ctx.set_option(lf.LF_OPT_SHARD_COUNT, S)
        for _ in range(2):                               # second call replays the graph
            ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
        ctx.sync()
        assert torch.isnan(gw[L - 2]).all() and torch.equal(gw[L - 1], full["gw"][L - 1])
        ctx.set_option(lf.LF_OPT_SHARD_RANK, 1)
        ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
        ctx.sync()
    torch.cuda.synchronize()
    assert torch.equal(gw, full["gw"]) and torch.equal(delta, full["delta"])
