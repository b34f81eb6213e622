"""The fused single-launch pass exists in two tilings (clusters of CTAs sharing a column strip;
whole columns per CTA).  Every property the fused pass is held to is checked here for both,
requested explicitly: parity with the oracle over the shapes of the other single-sample tests,
both costs, every activation, shards, a run of equal hidden widths, independence of k, and the
bounded waits."""
import numpy as np
import pytest
import torch

import lf_inputs
import paper_1801_04928_b200 as lf
from lf_testlib import assert_layer_close, compare_all, gpu_pass, oracle_pass
from oracle import lf_oracle as orc

pytestmark = pytest.mark.gpu

TILINGS = [lf.LF_FUSED_TILING_CLUSTERS, lf.LF_FUSED_TILING_COLUMNS]
TILING_NAMES = {lf.LF_FUSED_TILING_CLUSTERS: "clusters", lf.LF_FUSED_TILING_COLUMNS: "columns"}
FUSED = lf.LF_VARIANT_FUSED


def _inputs(L, N, seed, y="uniform"):
    cpu = lf_inputs.make_inputs(L, N, 1, y, lf_inputs.SEED_BASE + 900 + seed, "cpu")
    return {k: v.cuda() for k, v in cpu.items()}


# below one tile, one strip, ragged strips, N with no large divisor (4 x 257: rows of a TMA box
# come in blocks of four), N = 12 x 67 (an odd largest divisor), wide layers with many sub-tiles
SHAPES = [(1, 4, 1), (2, 8, 3), (3, 64, 2), (5, 260, 4), (4, 516, 16), (3, 804, 2), (6, 1024, 3),
          (3, 1028, 2), (3, 1156, 2), (2, 1536, 1), (2, 2052, 1), (3, 3072, 2), (2, 4096, 8)]


@pytest.mark.parametrize("tiling", TILINGS)
@pytest.mark.parametrize("L,N,k", SHAPES)
def test_fused_pass_parity_in_both_tilings(L, N, k, tiling):
    cfg = dict(L=L, N=N, B=1, k=k)
    t = _inputs(L, N, seed=L * 1000 + N)
    out, stats = gpu_pass(cfg, t, variant=FUSED, fused_tiling=tiling, repeat=2)
    assert stats["variant"] == FUSED and stats["fused_tiling"] == tiling and stats["device_status"] == 0
    assert stats["launches_backward"] == 1
    compare_all(cfg, out, oracle_pass(t))
    assert torch.equal(out["gb"], out["delta"][:, 0])                        # Eq. bp3, single sample
    # Eq. bp4: one rounding of delta_j * a_k
    assert torch.equal(out["gw"], torch.einsum("lj,lk->ljk", out["delta"][:, 0], out["a"][:-1, 0]))


@pytest.mark.parametrize("tiling", TILINGS)
def test_result_does_not_depend_on_k(tiling):
    L, N = 7, 516
    t = _inputs(L, N, seed=5)
    base, _ = gpu_pass(dict(L=L, N=N, B=1, k=1), t, variant=FUSED, fused_tiling=tiling)
    for k in (2, 7, 12):
        out, _ = gpu_pass(dict(L=L, N=N, B=1, k=k), t, variant=FUSED, fused_tiling=tiling)
        for name in ("delta", "gw", "gb"):
            assert torch.equal(out[name], base[name]), (name, k)


@pytest.mark.parametrize("tiling", TILINGS)
@pytest.mark.parametrize("act", [lf.LF_ACT_SIGMOID, lf.LF_ACT_TANH])
@pytest.mark.parametrize("cost", [lf.LF_COST_QUADRATIC, lf.LF_COST_CROSS_ENTROPY])
def test_costs_and_activations(cost, act, tiling):
    if cost == lf.LF_COST_CROSS_ENTROPY and act != lf.LF_ACT_SIGMOID:
        pytest.skip("the cross-entropy cost is offered with the sigmoid only")
    L, N = 4, 388
    cfg = dict(L=L, N=N, B=1, k=2)
    t = _inputs(L, N, seed=cost * 10 + act, y="onehot" if cost else "uniform")
    out, stats = gpu_pass(cfg, t, variant=FUSED, fused_tiling=tiling, cost=cost, act=act)
    assert stats["fused_tiling"] == tiling and stats["cost"] == cost and stats["activation"] == act
    w = t["w"].cpu().numpy()
    with orc.activation({lf.LF_ACT_SIGMOID: "sigmoid", lf.LF_ACT_TANH: "tanh"}[act]):
        z, a = orc.forward(w, t["b"].cpu().numpy(), t["x"].cpu().numpy())
        delta, _, gb = orc.backward_sequential(w, z, a, t["y"].cpu().numpy(), want_gw=False,
                                               cross_entropy=bool(cost))
    compare_all(cfg, out, dict(z=z, a=a, delta=delta, gb=gb, gw=None))


@pytest.mark.parametrize("tiling", TILINGS)
@pytest.mark.parametrize("S", [2, 3])
def test_shards_write_their_own_layers_only(S, tiling):
    # the layer-sharded form: shard r stores gw of the layers with (L - l) mod S = r and leaves the
    # rest of gw untouched; the S shards together give the whole pass
    L, N = 7, 516
    t = _inputs(L, N, seed=40 + S)
    ref = oracle_pass(t, want_gw=True)
    gw = torch.full((L, N, N), float("nan"), device="cuda")
    z = torch.empty((L, 1, N), device="cuda"); a = torch.empty((L + 1, 1, N), device="cuda")
    st = torch.cuda.Stream(); st.wait_stream(torch.cuda.current_stream())
    for r in range(S):
        delta = torch.full((L, 1, N), float("nan"), device="cuda"); gb = torch.full((L, N), float("nan"), device="cuda")
        before = gw.clone()
        with lf.Leapfrog(L, N, 1, 2, stream=st.cuda_stream) as ctx:
            ctx.set_option(lf.LF_OPT_VARIANT, FUSED)
            ctx.set_option(lf.LF_OPT_FUSED_TILING, tiling)
            ctx.set_option(lf.LF_OPT_SHARD_COUNT, S)
            ctx.set_option(lf.LF_OPT_SHARD_RANK, r)
            ctx.forward(t["w"], t["b"], t["x"], z, a)
            ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
            ctx.sync()
            stats = ctx.stats()
        torch.cuda.synchronize()
        assert stats["fused_tiling"] == tiling and stats["device_status"] == 0
        for l in range(1, L + 1):
            assert_layer_close("delta", l - 1, delta[l - 1].cpu().numpy(), ref["delta"][l - 1], n_terms=N)
            if (L - l) % S == r:
                assert_layer_close("gw", l - 1, gw[l - 1].cpu().numpy(), ref["gw"][l - 1], n_terms=N + 1)
            else:   # not this shard's layer: bit for bit what was there before
                assert torch.equal(gw[l - 1].view(torch.int32), before[l - 1].view(torch.int32)), (r, l)
    assert not torch.isnan(gw).any()


@pytest.mark.parametrize("tiling", TILINGS)
def test_run_of_equal_hidden_widths(tiling, monkeypatch):
    # input and output of another width than the hidden layers: layers 2..L-1 run as the fused
    # single launch (delta of its top layer given, depths shifted by one), in the tiling asked for
    monkeypatch.setenv("LF_FUSED_TILING", TILING_NAMES[tiling])
    import test_gpu_widths as tw
    for widths, k in (([260, 516, 516, 516, 516, 132], 2), ([64, 1028, 1028, 1028, 8], 3)):
        n, cpu, out, stats = tw._run_variant(widths, k, FUSED, seed=70 + k)
        assert stats["variant"] == FUSED and stats["fused_tiling"] == tiling and stats["device_status"] == 0
        tw._compare(n, 1, cpu, out)


@pytest.mark.parametrize("tiling", TILINGS)
def test_fused_weight_update(tiling, monkeypatch):
    # lf_backward_sgd: w - eta * gw in one fused multiply-add of exactly the gradients the plain
    # pass of the same tiling gives, and within the gradient's gate of the oracle's update
    monkeypatch.setenv("LF_FUSED_TILING", TILING_NAMES[tiling])
    import test_gpu_sgd as tsgd
    eta = 0.37
    for L, N, k in ((3, 64, 2), (4, 516, 16), (3, 1156, 2)):
        cfg = dict(L=L, N=N, B=1, k=k)
        t = _inputs(L, N, seed=L + N)
        out, stats = tsgd._sgd_pass(cfg, t, eta, variant=FUSED, also_plain=True)
        assert stats["variant"] == FUSED and stats["fused_tiling"] == tiling and stats["device_status"] == 0
        ref = oracle_pass(t, want_gw=True)
        compare_all(cfg, dict(out, gw=out["gw_after"]), ref)
        tsgd._check_update(t, out, ref, eta)
        assert torch.equal(out["gw_before"], out["gw_after"])
        tsgd._assert_is_fma_of(out["w_new"], t["w"], out["gw_after"], eta)


@pytest.mark.parametrize("tiling", TILINGS)
def test_bounded_waits_expire_and_the_context_recovers(tiling):
    # one CTA publishes nothing: every other CTA's wait must run out, the kernel must end, lf_sync
    # must say LF_ETIMEOUT, and the next call (hook off) must be correct again
    L, N = 6, 516
    cfg = dict(L=L, N=N, B=1, k=2)
    t = _inputs(L, N, seed=77)
    bufs = dict(z=torch.empty((L, 1, N), device="cuda"), a=torch.empty((L + 1, 1, N), device="cuda"),
                delta=torch.empty((L, 1, N), device="cuda"), gw=torch.empty((L, N, N), device="cuda"),
                gb=torch.empty((L, N), device="cuda"))
    st = torch.cuda.Stream(); st.wait_stream(torch.cuda.current_stream())
    with lf.Leapfrog(L, N, 1, 2, stream=st.cuda_stream) as ctx:
        ctx.set_option(lf.LF_OPT_VARIANT, FUSED)
        ctx.set_option(lf.LF_OPT_FUSED_TILING, tiling)
        ctx.set_option(lf.LF_OPT_WAIT_BUDGET_US, 20000)
        ctx.forward(t["w"], t["b"], t["x"], bufs["z"], bufs["a"])
        ctx.sync()
        ctx.set_option(lf.LF_OPT_WITHHOLD, 1)
        ctx.backward(t["w"], bufs["z"], bufs["a"], t["y"], bufs["delta"], bufs["gw"], bufs["gb"])
        assert lf.lf_sync(ctx._h) == lf.LF_ETIMEOUT
        assert ctx.stats()["device_status"] != 0 and ctx.stats()["fused_tiling"] == tiling
        ctx.set_option(lf.LF_OPT_WITHHOLD, 0)
        ctx.backward(t["w"], bufs["z"], bufs["a"], t["y"], bufs["delta"], bufs["gw"], bufs["gb"])
        ctx.sync()
        assert ctx.stats()["device_status"] == 0
    torch.cuda.synchronize()
    compare_all(cfg, bufs, oracle_pass(t))


def test_environment_sets_the_initial_variant_and_tiling(monkeypatch):
    L, N = 3, 260
    t = _inputs(L, N, seed=3)
    monkeypatch.setenv("LF_VARIANT", "fused")
    monkeypatch.setenv("LF_FUSED_TILING", "clusters")
    z = torch.empty((L, 1, N), device="cuda"); a = torch.empty((L + 1, 1, N), device="cuda")
    d = torch.empty((L, 1, N), device="cuda"); gw = torch.empty((L, N, N), device="cuda"); gb = torch.empty((L, N), device="cuda")
    with lf.Leapfrog(L, N, 1, 2) as ctx:
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        ctx.backward(t["w"], z, a, t["y"], d, gw, gb)
        ctx.sync()
        assert ctx.stats()["variant"] == FUSED and ctx.stats()["fused_tiling"] == lf.LF_FUSED_TILING_CLUSTERS
        ctx.set_option(lf.LF_OPT_VARIANT, lf.LF_VARIANT_STREAMS)      # an explicit option wins
        ctx.backward(t["w"], z, a, t["y"], d, gw, gb)
        ctx.sync()
        assert ctx.stats()["variant"] == lf.LF_VARIANT_STREAMS
    monkeypatch.setenv("LF_VARIANT", "no-such-variant")               # ignored
    with lf.Leapfrog(L, N, 1, 2) as ctx:
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        ctx.backward(t["w"], z, a, t["y"], d, gw, gb)
        ctx.sync()
        assert ctx.stats()["device_status"] == 0
