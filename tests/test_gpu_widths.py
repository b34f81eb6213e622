"""GPU parity for networks whose layers differ in width (lf_create_widths): Eq. x, z, a and
Eq. bp1-bp4 with w^l of shape n_l x n_{l-1}, flat per-layer-block layouts, against the oracle's
functions for the same layout on the same seeded inputs, layer by layer, to the fp32 gate."""
import numpy as np
import pytest
import torch

import lf_inputs
import paper_1801_04928_b200 as lf
from lf_testlib import FP32_TOL, TF32_TOL, assert_layer_close, rel_frobenius
from oracle import lf_oracle as orc

pytestmark = pytest.mark.gpu

# widths span several tiles of every kernel with ragged tails: the forward matvec's 128-column
# loop, the delta matvec's 128-column strips and 32/64-row chunks, the 64 x 64 x 16 GEMM tiles
SHAPES = [
    [8, 4],                          # one layer, wider below than above
    [4, 12, 8],
    [260, 132, 516, 64, 200],        # up and down, nothing a multiple of 128
    [1028, 2052, 36, 772],           # a row count beyond 2048 (64-row chunks) and a 36-wide bottleneck
    [784, 512, 512, 256, 12],        # the shape of a small classifier
]


def _run(widths, B, k, y="uniform", cost=0, act=0, sgd_eta=None, host=False, seed=0, variant=None,
         gw_math=lf.LF_GW_MATH_FP32, tiling=0, delta_math=lf.LF_DELTA_MATH_FP32):
    n = [int(v) for v in widths]
    L = len(n) - 1
    cpu = lf_inputs.make_inputs_widths(n, B, y, lf_inputs.SEED_BASE + 700 + seed, "cpu")
    t = {key: v.cuda() for key, v in cpu.items()}
    sz = orc.sizes_widths(n, B)
    dev = t["w"].device
    z = torch.empty(sz["z"], dtype=torch.float32, device=dev)
    a = torch.empty(sz["a"], dtype=torch.float32, device=dev)
    delta = torch.full((sz["z"],), float("nan"), dtype=torch.float32, device=dev)
    gw = torch.full((sz["w"],), float("nan"), dtype=torch.float32, device=dev)
    gb = torch.full((sz["b"],), float("nan"), dtype=torch.float32, device=dev)
    st = torch.cuda.Stream(device=dev)
    st.wait_stream(torch.cuda.current_stream(dev))
    with lf.Leapfrog(0, 0, B, k, stream=st.cuda_stream, widths=n) as ctx:
        ctx.set_option(lf.LF_OPT_COST, cost)
        ctx.set_option(lf.LF_OPT_ACTIVATION, act)
        # the fused pass is accepted by every context: one sample runs it as one launch over all layers
        # (whole columns per CTA), a mini-batch runs one launch per layer
        ctx.set_option(lf.LF_OPT_VARIANT, lf.LF_VARIANT_FUSED if variant is None else variant)
        ctx.set_option(lf.LF_OPT_GW_MATH, gw_math)
        ctx.set_option(lf.LF_OPT_DELTA_MATH, delta_math)
        ctx.set_option(lf.LF_OPT_TC_TILING, tiling)
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        if host:
            ctx.sync()
            hz, ha = z.cpu().pin_memory(), a.cpu().pin_memory()
            hw, hy = cpu["w"].pin_memory(), cpu["y"].pin_memory()
            hd = torch.full((sz["z"],), float("nan")).pin_memory()
            hgw = torch.full((sz["w"],), float("nan")).pin_memory()
            hgb = torch.full((sz["b"],), float("nan")).pin_memory()
            ctx.backward_host(hw, hz, ha, hy, hd, hgw, hgb)
            ctx.sync()
            delta, gw, gb = hd, hgw, hgb
        elif sgd_eta is not None:
            ctx.backward_sgd(t["w"], z, a, t["y"], sgd_eta, delta, gw, gb)
        else:
            ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
        ctx.sync()
        stats = ctx.stats()
    torch.cuda.current_stream(dev).wait_stream(st)
    torch.cuda.synchronize(dev)
    out = {key: v.cpu().numpy() for key, v in dict(z=z, a=a, delta=delta, gw=gw, gb=gb).items()}
    return n, L, cpu, out, stats


def _compare(n, B, cpu, out, cross_entropy=False, sgd_eta=None, tf32=False):
    w = cpu["w"].numpy()
    z, a = orc.forward_widths(n, w, cpu["b"].numpy(), cpu["x"].numpy())
    delta, gw, gb = orc.backward_widths(n, w, z, a, cpu["y"].numpy(), cross_entropy=cross_entropy)
    ref = dict(z=z, a=a, delta=delta, gb=gb)
    kinds = dict(z="z", a="a", delta="z", gb="b")
    for name, kind in kinds.items():
        Bk = 1 if kind == "b" else B
        got = orc.split(out[name], n, kind, Bk)
        want = orc.split(ref[name], n, kind, Bk)
        for l, (g, r) in enumerate(zip(got, want)):
            assert_layer_close(name, l, g, r, tol=FP32_TOL, n_terms=max(n) + B)
    # the weight gradients (or, under the fused update, w - eta * gw) layer by layer
    got = orc.split(out["gw"], n, "w")
    for l, (g, r, wl) in enumerate(zip(got, orc.split(gw, n, "w"), orc.split(w, n, "w"))):
        assert np.all(np.isfinite(g))
        if sgd_eta is None:
            if tf32:
                e = rel_frobenius(g, r)
                assert e <= TF32_TOL, f"gw[{l}]: relative Frobenius error {e:.3e}"
            else:
                assert_layer_close("gw", l, g, r, tol=FP32_TOL, n_terms=max(n) + B)
        else:
            want = wl.astype(np.float64) - sgd_eta * r
            round_off = 2.0 ** -23 * float(np.max(np.abs(want)))
            if tf32:
                err = float(np.linalg.norm(g - want))
                bound = abs(sgd_eta) * TF32_TOL * float(np.linalg.norm(r)) + round_off * r.shape[1]
            else:
                err = float(np.max(np.abs(g - want)))
                bound = abs(sgd_eta) * FP32_TOL * float(np.max(np.abs(r))) + round_off
            assert err <= bound, (l, err, bound)


@pytest.mark.parametrize("variant", [lf.LF_VARIANT_STREAMS, lf.LF_VARIANT_FUSED])
@pytest.mark.parametrize("B,k", [(1, 1), (1, 3), (5, 2), (130, 2)])
@pytest.mark.parametrize("widths", SHAPES, ids=lambda s: "-".join(map(str, s)))
def test_widths_parity(widths, B, k, variant):
    if B > 1 and variant == lf.LF_VARIANT_FUSED:
        pytest.skip("a mini-batch runs one launch per layer whatever is asked for")
    n, L, cpu, out, stats = _run(widths, B, k, y="onehot" if B > 1 else "uniform", seed=len(widths) + B, variant=variant)
    assert stats["device_status"] == 0 and stats["N"] == max(n)
    if B == 1 and variant == lf.LF_VARIANT_FUSED:       # one launch over all layers, whatever their widths
        assert stats["variant"] == lf.LF_VARIANT_FUSED and stats["launches_backward"] == 1
        assert stats["fused_tiling"] == lf.LF_FUSED_TILING_COLUMNS
    else:
        assert stats["variant"] == lf.LF_VARIANT_STREAMS
    assert stats["gw_math"] == lf.LF_GW_MATH_FP32 and stats["delta_math"] == lf.LF_DELTA_MATH_FP32
    _compare(n, B, cpu, out)


@pytest.mark.parametrize("tiling", [lf.LF_TC_TILING_ONE_SM, lf.LF_TC_TILING_TWO_SM])
@pytest.mark.parametrize("B", [5, 130, 300])
@pytest.mark.parametrize("widths", SHAPES[1:], ids=lambda s: "-".join(map(str, s)))
def test_widths_chain_and_forward_on_the_tensor_cores(widths, B, tiling):
    # Eq. z and Eq. bp2 of rectangular layers as 3xTF32 contractions (B x n_l x n_{l-1} and
    # B x n_l x n_{l+1}): fp32-level accuracy, so the fp32 gate applies; the weight gradient stays fp32
    # here so that every tensor is held to it.  The two-SM kernel serves layers of at least 512 x 512
    # with more than 128 samples, the one-SM kernel the rest.
    n, L, cpu, out, stats = _run(widths, B, 2, y="onehot", seed=80 + B, delta_math=lf.LF_DELTA_MATH_3XTF32,
                                 tiling=tiling)
    assert stats["device_status"] == 0 and stats["delta_math"] == lf.LF_DELTA_MATH_3XTF32
    assert stats["delta_tiling"] in (lf.LF_TC_TILING_ONE_SM, lf.LF_TC_TILING_TWO_SM)
    if tiling == lf.LF_TC_TILING_ONE_SM or B <= 128:
        assert stats["delta_tiling"] == lf.LF_TC_TILING_ONE_SM
    _compare(n, B, cpu, out)


@pytest.mark.parametrize("tiling", [lf.LF_TC_TILING_ONE_SM, lf.LF_TC_TILING_TWO_SM])
@pytest.mark.parametrize("B", [5, 130, 256, 300])
@pytest.mark.parametrize("widths", SHAPES[2:], ids=lambda s: "-".join(map(str, s)))
def test_widths_weight_gradient_on_the_tensor_cores(widths, B, tiling):
    # Eq. bp4 of a rectangular layer as an n_l x n_{l-1} x B contraction with TF32 inputs; the two-SM
    # kernel takes batches up to 256, beyond that the one-SM kernel runs whatever was asked for
    n, L, cpu, out, stats = _run(widths, B, 2, y="onehot", seed=60 + B, gw_math=lf.LF_GW_MATH_TF32, tiling=tiling)
    assert stats["device_status"] == 0 and stats["gw_math"] == lf.LF_GW_MATH_TF32
    assert stats["gw_tiling"] == tiling      # CTA pairs at every batch (beyond 256 samples both operands stream)
    _compare(n, B, cpu, out, tf32=True)


@pytest.mark.parametrize("B", [9, 130])
def test_widths_fused_update_on_the_tensor_cores(B):
    n, L, cpu, out, stats = _run([132, 516, 260, 8], B, 2, sgd_eta=0.37, seed=43, gw_math=lf.LF_GW_MATH_TF32)
    assert stats["gw_math"] == lf.LF_GW_MATH_TF32
    _compare(n, B, cpu, out, sgd_eta=0.37, tf32=True)


@pytest.mark.parametrize("B", [1, 6])
def test_widths_cross_entropy_and_tanh(B):
    widths = [260, 132, 516, 64]
    n, L, cpu, out, stats = _run(widths, B, 2, cost=lf.LF_COST_CROSS_ENTROPY, seed=31)
    assert stats["cost"] == lf.LF_COST_CROSS_ENTROPY
    _compare(n, B, cpu, out, cross_entropy=True)
    n, L, cpu, out, stats = _run(widths, B, 2, act=lf.LF_ACT_TANH, seed=32)
    with orc.activation("tanh"):
        _compare(n, B, cpu, out)


@pytest.mark.parametrize("B", [1, 9])
def test_widths_fused_update(B):
    n, L, cpu, out, stats = _run([132, 516, 260, 8], B, 2, sgd_eta=0.37, seed=41)
    _compare(n, B, cpu, out, sgd_eta=0.37)


@pytest.mark.parametrize("B", [1, 7])
def test_widths_host_entry_point(B):
    n, L, cpu, out, stats = _run([200, 64, 328, 12], B, 3, host=True, seed=51)
    _compare(n, B, cpu, out)


def test_equal_widths_give_the_uniform_context():
    # all widths equal: lf_create_widths is lf_create -- same kernels (the single-launch pass for one
    # sample), same bits
    L, N = 6, 516
    cpu = lf_inputs.make_inputs(L, N, 1, "uniform", lf_inputs.SEED_BASE + 761, "cpu")
    t = {key: v.cuda() for key, v in cpu.items()}
    res = []
    for widths in (None, [N] * (L + 1)):
        z = torch.empty((L, 1, N), device="cuda"); a = torch.empty((L + 1, 1, N), device="cuda")
        d = torch.empty((L, 1, N), device="cuda"); gw = torch.empty((L, N, N), device="cuda")
        gb = torch.empty((L, N), device="cuda")
        with lf.Leapfrog(L, N, 1, 2, widths=widths) as ctx:
            ctx.forward(t["w"], t["b"], t["x"], z, a)
            ctx.backward(t["w"], z, a, t["y"], d, gw, gb)
            ctx.sync()
            res.append((ctx.stats()["variant"], z, a, d, gw, gb))
    assert res[0][0] == res[1][0] != lf.LF_VARIANT_STREAMS
    for u, v in zip(res[0][1:], res[1][1:]):
        assert torch.equal(u, v)


def test_widths_argument_checks():
    assert lf.lf_create_widths([8, 6, 8], 1, 1)[0] == lf.LF_EINVAL      # 6 is not a multiple of 4
    assert lf.lf_create_widths([8, 0, 8], 1, 1)[0] == lf.LF_EINVAL
    assert lf.lf_create_widths([8], 1, 1)[0] == lf.LF_EINVAL            # no weight layer
    rc, h = lf.lf_create_widths([8, 4, 12], 1, 1)
    assert rc == lf.LF_OK
    try:
        buf = torch.zeros(64, device="cuda")
        assert lf.lf_grad_w(h, buf, buf, buf) == lf.LF_EINVAL           # names no layer
        assert lf.lf_owner(h, 2) == 0 and lf.lf_owner(h, 1) == 0
    finally:
        lf.lf_destroy(h)


def test_widths_full_size_single_sample():
    # the network the widths timing runs on (63 M weights): delta, gb, z, a of every layer element by
    # element; the weight gradients -- rank one for a single sample -- on every 97th row of every layer
    # against the oracle's delta_j * a_k (one float64 product per entry)
    widths = [4096, 8192, 2048, 4096, 1024]
    n, L, cpu, out, stats = _run(widths, 1, 4, seed=91)
    assert stats["device_status"] == 0
    w = cpu["w"].numpy()
    z, a = orc.forward_widths(n, w, cpu["b"].numpy(), cpu["x"].numpy())
    delta, _, gb = orc.backward_widths(n, w, z, a, cpu["y"].numpy(), want_gw=False)
    ref = dict(z=z, a=a, delta=delta, gb=gb)
    for name, kind in dict(z="z", a="a", delta="z", gb="b").items():
        for l, (g, r) in enumerate(zip(orc.split(out[name], n, kind, 1), orc.split(ref[name], n, kind, 1))):
            assert_layer_close(name, l, g, r, tol=FP32_TOL, n_terms=max(n))
    d_l = orc.split(delta, n, "z", 1); a_l = orc.split(a, n, "a", 1)
    for l, g in enumerate(orc.split(out["gw"], n, "w"), start=1):
        rows = np.arange(0, n[l], 97)
        want = d_l[l - 1][0][rows, None] * a_l[l - 1][0][None, :]
        assert_layer_close("gw", l - 1, g[rows], want, tol=FP32_TOL, n_terms=max(n))
        assert np.all(np.isfinite(g))


# ---- hidden layers of one width, input / output of another: the single-launch pass over the hidden run
HIDDEN_RUN_SHAPES = [
    [260, 516, 516, 516, 516, 132],     # both ends differ
    [516, 516, 516, 516, 12],           # only the output differs
    [36, 1028, 1028, 1028],             # only the input differs
    [200, 132, 132, 64],                # L = 3: a run of one layer
    [8, 64, 64, 64, 64, 64, 64, 4],
]


def _run_variant(widths, k, variant, seed, sgd_eta=None, shard=None):
    n = [int(v) for v in widths]
    cpu = lf_inputs.make_inputs_widths(n, 1, "uniform", lf_inputs.SEED_BASE + 800 + seed, "cpu")
    t = {key: v.cuda() for key, v in cpu.items()}
    sz = orc.sizes_widths(n, 1)
    z = torch.empty(sz["z"], device="cuda"); a = torch.empty(sz["a"], device="cuda")
    delta = torch.full((sz["z"],), float("nan"), device="cuda")
    gw = torch.full((sz["w"],), float("nan"), device="cuda")
    gb = torch.full((sz["b"],), float("nan"), device="cuda")
    with lf.Leapfrog(0, 0, 1, k, widths=n) as ctx:
        ctx.set_option(lf.LF_OPT_VARIANT, variant)
        if shard is not None:
            ctx.set_option(lf.LF_OPT_SHARD_COUNT, shard[1])
            ctx.set_option(lf.LF_OPT_SHARD_RANK, shard[0])
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        for _ in range(2):     # twice: the second call meets the flags and slots the first one left
            if sgd_eta is not None:
                ctx.backward_sgd(t["w"], z, a, t["y"], sgd_eta, delta, gw, gb)
            else:
                ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
        ctx.sync()
        stats = ctx.stats()
    torch.cuda.synchronize()
    out = {key: v.cpu().numpy() for key, v in dict(z=z, a=a, delta=delta, gw=gw, gb=gb).items()}
    return n, cpu, out, stats


@pytest.mark.parametrize("variant", [lf.LF_VARIANT_AUTO, lf.LF_VARIANT_PERSISTENT, lf.LF_VARIANT_FUSED])
@pytest.mark.parametrize("k", [1, 3])
@pytest.mark.parametrize("widths", HIDDEN_RUN_SHAPES, ids=lambda s: "-".join(map(str, s)))
def test_hidden_run_goes_through_the_single_launch_pass(widths, k, variant):
    n, cpu, out, stats = _run_variant(widths, k, variant, seed=len(widths) + k)
    assert stats["device_status"] == 0
    assert stats["variant"] in (lf.LF_VARIANT_PERSISTENT, lf.LF_VARIANT_FUSED)
    if variant != lf.LF_VARIANT_AUTO:
        assert stats["variant"] == variant
    if variant == lf.LF_VARIANT_PERSISTENT:
        assert stats["launches_backward"] == 6        # bp1, 2 x bp2, 2 x rank-1 writer, 1 persistent launch
    else:                                             # the fused pass with whole columns takes all layers at once
        assert stats["launches_backward"] == 1 and stats["fused_tiling"] == lf.LF_FUSED_TILING_COLUMNS
    _compare(n, 1, cpu, out)


@pytest.mark.parametrize("widths", HIDDEN_RUN_SHAPES[:3], ids=lambda s: "-".join(map(str, s)))
def test_hidden_run_between_per_layer_launches_with_cluster_tiles(widths, monkeypatch):
    # the cluster-tile fused kernel needs one width: asked for by name it runs over the hidden run,
    # with per-layer launches for the rectangular top and bottom layer
    monkeypatch.setenv("LF_FUSED_TILING", "clusters")
    n, cpu, out, stats = _run_variant(widths, 2, lf.LF_VARIANT_FUSED, seed=len(widths))
    assert stats["variant"] == lf.LF_VARIANT_FUSED and stats["fused_tiling"] == lf.LF_FUSED_TILING_CLUSTERS
    assert stats["launches_backward"] == 6 and stats["device_status"] == 0
    _compare(n, 1, cpu, out)


@pytest.mark.parametrize("cost,act", [(lf.LF_COST_CROSS_ENTROPY, lf.LF_ACT_SIGMOID), (lf.LF_COST_QUADRATIC, lf.LF_ACT_TANH)])
def test_single_launch_over_different_widths_costs_and_activations(cost, act):
    widths = [260, 132, 516, 64, 200]
    n, L, cpu, out, stats = _run(widths, 1, 2, y="onehot" if cost else "uniform", cost=cost, act=act, seed=33)
    assert stats["variant"] == lf.LF_VARIANT_FUSED and stats["launches_backward"] == 1 and stats["device_status"] == 0
    with orc.activation({lf.LF_ACT_SIGMOID: "sigmoid", lf.LF_ACT_TANH: "tanh"}[act]):
        _compare(n, 1, cpu, out, cross_entropy=bool(cost))


def test_single_launch_over_different_widths_shards_and_bounded_waits():
    widths = [260, 516, 132, 516, 64, 200]
    L = len(widths) - 1
    # two shards: each stores the gradients of its own layers only
    for S in (2, 3):
        seen = np.zeros(L, dtype=int)
        for r in range(S):
            n, cpu, out, stats = _run_variant(widths, 2, lf.LF_VARIANT_FUSED, seed=12, shard=(r, S))
            assert stats["launches_backward"] == 1 and stats["device_status"] == 0
            w = cpu["w"].numpy()
            z, a = orc.forward_widths(n, w, cpu["b"].numpy(), cpu["x"].numpy())
            delta, gw, gb = orc.backward_widths(n, w, z, a, cpu["y"].numpy())
            for l, (g, ref) in enumerate(zip(orc.split(out["gw"], n, "w"), orc.split(gw, n, "w")), start=1):
                if (L - l) % S == r:
                    assert_layer_close("gw", l - 1, g, ref, tol=FP32_TOL, n_terms=max(n))
                    seen[l - 1] += 1
                else:
                    assert np.all(np.isnan(g)), (S, r, l)
        assert np.all(seen == 1)
    # one CTA publishes nothing: the others give up within the budget and the next call is right again
    n = widths
    cpu = lf_inputs.make_inputs_widths(n, 1, "uniform", lf_inputs.SEED_BASE + 5, "cpu")
    t = {key: v.cuda() for key, v in cpu.items()}
    sz = orc.sizes_widths(n, 1)
    z = torch.empty(sz["z"], device="cuda"); a = torch.empty(sz["a"], device="cuda")
    delta = torch.empty(sz["z"], device="cuda"); gw = torch.empty(sz["w"], device="cuda"); gb = torch.empty(sz["b"], device="cuda")
    with lf.Leapfrog(0, 0, 1, 2, widths=n) as ctx:
        ctx.set_option(lf.LF_OPT_VARIANT, lf.LF_VARIANT_FUSED)
        ctx.set_option(lf.LF_OPT_WAIT_BUDGET_US, 20000)
        ctx.forward(t["w"], t["b"], t["x"], z, a)
        ctx.set_option(lf.LF_OPT_WITHHOLD, 1)
        ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
        assert lf.lf_sync(ctx._h) == lf.LF_ETIMEOUT
        ctx.set_option(lf.LF_OPT_WITHHOLD, 0)
        ctx.backward(t["w"], z, a, t["y"], delta, gw, gb)
        ctx.sync()
        assert ctx.stats()["device_status"] == 0 and ctx.stats()["launches_backward"] == 1
    out = {key: v.cpu().numpy() for key, v in dict(z=z, a=a, delta=delta, gw=gw, gb=gb).items()}
    _compare(n, 1, cpu, out)


@pytest.mark.parametrize("variant", [lf.LF_VARIANT_PERSISTENT, lf.LF_VARIANT_FUSED])
def test_hidden_run_fused_update(variant):
    n, cpu, out, stats = _run_variant([260, 516, 516, 516, 132], 2, variant, seed=5, sgd_eta=0.3)
    assert stats["variant"] == variant
    _compare(n, 1, cpu, out, sgd_eta=0.3)


def test_hidden_run_shards():
    widths, S = [260, 516, 516, 516, 516, 516, 132], 2
    n = widths
    L = len(n) - 1
    union = None
    for r in range(S):
        n, cpu, out, stats = _run_variant(widths, 2, lf.LF_VARIANT_AUTO, seed=9, shard=(r, S))
        assert stats["variant"] == lf.LF_VARIANT_FUSED and stats["device_status"] == 0   # what AUTO picks at 516
        w = cpu["w"].numpy()
        z, a = orc.forward_widths(n, w, cpu["b"].numpy(), cpu["x"].numpy())
        delta, gw, gb = orc.backward_widths(n, w, z, a, cpu["y"].numpy())
        for l, (g, ref) in enumerate(zip(orc.split(out["gw"], n, "w"), orc.split(gw, n, "w")), start=1):
            if (L - l) % S == r:
                assert_layer_close("gw", l - 1, g, ref, n_terms=max(n))
            else:
                assert np.all(np.isnan(g)), f"shard {r} wrote layer {l}"
        for l, (g, ref) in enumerate(zip(orc.split(out["delta"], n, "z", 1), orc.split(delta, n, "z", 1)), start=1):
            assert_layer_close("delta", l - 1, g, ref, n_terms=max(n))
        union = out["gw"] if union is None else np.where(np.isnan(union), out["gw"], union)
    assert np.all(np.isfinite(union))
