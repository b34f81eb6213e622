"""GPU parity: the CUDA path, called through the C ABI binding, against the float64 oracle on
the same seeded inputs.  Gate (fp32 paths): per tensor, per layer, max|diff| <= 1e-5 max|ref|."""
import numpy as np
import pytest
import torch

import lf_inputs
import paper_1801_04928_b200 as lf
from lf_testlib import compare_all, gpu_pass, oracle_pass

pytestmark = pytest.mark.gpu

VARIANTS = [lf.LF_VARIANT_STREAMS, lf.LF_VARIANT_PERSISTENT, lf.LF_VARIANT_FUSED]


def _inputs(L, N, B, y="uniform", seed=1):
    cpu = lf_inputs.make_inputs(L, N, B, y, lf_inputs.SEED_BASE + 100 + seed, "cpu")
    return {k: v.cuda() for k, v in cpu.items()}


# sizes: below one tile, exactly one strip, several strips with a ragged tail, N not a
# multiple of 128, L < k, L = 1.
SMALL_B1 = [(1, 4, 1), (2, 8, 3), (3, 64, 2), (5, 260, 4), (4, 516, 16), (6, 1024, 3),
            (3, 1156, 2), (2, 2052, 1), (3, 3072, 2)]   # 3072: 256-column strips, 32 columns per finisher


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("L,N,k", SMALL_B1)
def test_single_sample_parity(L, N, k, variant):
    cfg = dict(L=L, N=N, B=1, k=k)
    t = _inputs(L, N, 1, seed=L * 1000 + N)
    out, stats = gpu_pass(cfg, t, variant=variant)
    assert stats["variant"] == variant and stats["device_status"] == 0
    ref = oracle_pass(t)
    compare_all(cfg, out, ref)
    assert torch.equal(out["a"][0], t["x"])            # Eq. x
    assert torch.equal(out["gb"], out["delta"][:, 0])  # Eq. bp3, single sample


@pytest.mark.parametrize("delta_math,tiling", [(lf.LF_DELTA_MATH_FP32, lf.LF_TC_TILING_AUTO),
                                               (lf.LF_DELTA_MATH_3XTF32, lf.LF_TC_TILING_ONE_SM),
                                               (lf.LF_DELTA_MATH_3XTF32, lf.LF_TC_TILING_TWO_SM),
                                               (lf.LF_DELTA_MATH_TF32_BF16, lf.LF_TC_TILING_TWO_SM)])
@pytest.mark.parametrize("L,N,B,k", [(2, 8, 2, 1), (3, 68, 3, 2), (3, 256, 16, 4),
                                     (4, 132, 70, 3), (2, 320, 129, 2), (5, 1028, 260, 2),
                                     (3, 772, 256, 1), (2, 2052, 515, 2), (2, 4100, 70, 2), (2, 4608, 17, 1)])
def test_minibatch_fp32_parity(L, N, B, k, delta_math, tiling):
    # fp32 gate (1e-5 per tensor per layer) for every form of the delta recurrence (and of the
    # forward pass, which shares its kernels): fp32 on the CUDA cores, and the tensor cores with
    # every operand split into two TF32 numbers, one CTA per tile or a CTA pair per tile (pairs
    # take over above 128 samples and from 512 columns: B = 260 leaves a pair's second half nearly
    # empty, B = 515 needs three 256-sample blocks, N = 2052 gives runs that end inside a tile);
    # and the CTA pairs with the two cross terms in BF16 (one-CTA tiles keep three TF32 products).
    # N = 4100 and 4608 with up to 128 samples: the warp-specialised kernel on single CTAs (from a
    # width of 4096), with a ragged last column tile and with a nearly empty sample tile.
    cfg = dict(L=L, N=N, B=B, k=k)
    t = _inputs(L, N, B, y="onehot", seed=N + B)
    out, stats = gpu_pass(cfg, t, gw_math=lf.LF_GW_MATH_FP32, delta_math=delta_math, tc_tiling=tiling)
    assert stats["gw_math"] == lf.LF_GW_MATH_FP32 and stats["delta_math"] == delta_math
    assert stats["device_status"] == 0
    if delta_math >= lf.LF_DELTA_MATH_3XTF32 and L > 1:
        pairs = tiling == lf.LF_TC_TILING_TWO_SM and B > 128 and N >= 512   # the library's rule for CTA pairs
        want = lf.LF_TC_TILING_TWO_SM if pairs else lf.LF_TC_TILING_ONE_SM
        assert stats["delta_tiling"] == want
    ref = oracle_pass(t, want_gw=True)
    compare_all(cfg, out, ref)


@pytest.mark.parametrize("L,N,B,k", [(3, 516, 2, 2), (3, 1028, 5, 1), (2, 2052, 12, 2), (3, 4096, 16, 2),
                                     (2, 8, 4, 1), (4, 644, 9, 3)])
def test_small_batch_delta_chain(L, N, B, k):
    # For a handful of samples Eq. bp2 has an fp32 kernel on the CUDA cores (a batched matrix-vector
    # product that reads w once; what LF_DELTA_MATH_FP32 runs up to 16 samples); the forward pass keeps
    # its tensor-core rule.  B = 2, 5, 12: each of the kernel's three sample-tile sizes with samples
    # missing from the last group of four; N = 516, 1028, 2052, 644: a last column strip of one or
    # five float4; N = 4096, B = 16: several 256-row blocks per CTA; N = 8: fewer rows than warps.
    cfg = dict(L=L, N=N, B=B, k=k)
    t = _inputs(L, N, B, y="onehot", seed=7 * N + B)
    out, stats = gpu_pass(cfg, t, gw_math=lf.LF_GW_MATH_FP32, delta_math=lf.LF_DELTA_MATH_FP32)
    assert stats["delta_math"] == lf.LF_DELTA_MATH_FP32 and stats["device_status"] == 0
    ref = oracle_pass(t, want_gw=True)
    compare_all(cfg, out, ref)
    # twice in a row through one context: the strip counters reset themselves
    out2, _ = gpu_pass(cfg, t, gw_math=lf.LF_GW_MATH_FP32, delta_math=lf.LF_DELTA_MATH_FP32, repeat=3)
    assert torch.equal(out2["delta"], out["delta"])
    # the library's own choice: fp32 up to 8 samples, and up to 16 from a width of 2048
    _, auto = gpu_pass(cfg, t, gw_math=lf.LF_GW_MATH_FP32)
    want = lf.LF_DELTA_MATH_FP32 if (B <= 8 or N >= 2048) else lf.LF_DELTA_MATH_3XTF32
    assert auto["delta_math"] == want


@pytest.mark.parametrize("variant", VARIANTS)
def test_result_does_not_depend_on_k(variant):
    # Theorem 1 on the GPU: every schedule writes every layer once, and because the delta
    # reduction order is fixed the results are bitwise the same for every k.
    L, N = 7, 516
    t = _inputs(L, N, 1, seed=5)
    base, _ = gpu_pass(dict(L=L, N=N, B=1, k=1), t, variant=variant)
    for k in (2, 3, 7, 12):
        out, stats = gpu_pass(dict(L=L, N=N, B=1, k=k), t, variant=variant)
        assert stats["k_effective"] == min(k, L)
        for name in ("delta", "gw", "gb"):
            assert torch.equal(out[name], base[name]), (name, k)


def test_variants_agree_bitwise_on_delta_and_gw():
    L, N = 6, 1028
    t = _inputs(L, N, 1, seed=9)
    cfg = dict(L=L, N=N, B=1, k=3)
    outs = [gpu_pass(cfg, t, variant=v)[0] for v in VARIANTS]
    for o in outs[1:]:
        # gw is one rounding of delta_j * a_k in every variant
        assert torch.equal(o["gw"], torch.einsum("lj,lk->ljk", o["delta"][:, 0], o["a"][:-1, 0]))


def test_repeated_calls_and_graph_replay_are_stable():
    cfg = dict(L=5, N=516, B=1, k=2)
    t = _inputs(5, 516, 1, seed=3)
    once, _ = gpu_pass(cfg, t, variant=lf.LF_VARIANT_STREAMS, use_graph=False)
    many, stats = gpu_pass(cfg, t, variant=lf.LF_VARIANT_STREAMS, use_graph=True, repeat=4)
    for name in ("delta", "gw", "gb"):
        assert torch.equal(once[name], many[name])
    assert stats["launches_backward"] == 2 * 5


def test_config1_parity():
    cfg, cpu = lf_inputs.make_config(1)
    t = {k: v.cuda() for k, v in cpu.items()}
    ref = oracle_pass(t)
    for variant in VARIANTS:
        out, _ = gpu_pass(cfg, t, variant=variant)
        compare_all(cfg, out, ref)


def test_config2_parity():
    cfg, cpu = lf_inputs.make_config(2)
    t = {k: v.cuda() for k, v in cpu.items()}
    ref = oracle_pass(t)
    for variant in VARIANTS:
        out, _ = gpu_pass(cfg, t, variant=variant)
        worst = compare_all(cfg, out, ref)
        print("config2 variant", variant, worst)


def test_config3_parity_long_chain():
    # L = 64, N = 4096: 4 GiB of weights, 4 GiB of gradients; the deepest delta are fp32
    # denormals (the gate's absolute floor covers them).  Inputs are drawn on the GPU and
    # copied to the host for the oracle; gw is checked layer by layer without keeping it.
    cfg, t = lf_inputs.make_config(3, device="cuda")
    ref = oracle_pass(t)                       # gw formed per layer on the fly
    out, stats = gpu_pass(cfg, t)              # AUTO: the fused persistent kernel
    assert stats["variant"] == lf.LF_VARIANT_FUSED and stats["device_status"] == 0
    worst = compare_all(cfg, out, ref)
    print("config3", worst)
    del out
    torch.cuda.empty_cache()
    out, stats = gpu_pass(cfg, t, variant=lf.LF_VARIANT_PERSISTENT)
    assert stats["variant"] == lf.LF_VARIANT_PERSISTENT and stats["worker_ctas"] > 0
    for name in ("delta", "gb"):
        g = out[name].cpu().numpy()
        for l in range(cfg["L"]):
            from lf_testlib import assert_layer_close
            assert_layer_close(name, l, g[l], ref[name][l], n_terms=cfg["N"])
    # leapfrog CTA groups write the same gw as the fused pass: one rounding of delta_j * a_k
    for l in (0, 17, 63):
        assert torch.equal(out["gw"][l], torch.outer(out["delta"][l, 0], out["a"][l, 0]))


@pytest.mark.parametrize("tiling", [lf.LF_TC_TILING_ONE_SM, lf.LF_TC_TILING_TWO_SM])
@pytest.mark.parametrize("L,N,B,k", [(2, 256, 32, 1), (3, 512, 256, 2), (2, 388, 70, 2), (2, 132, 16, 1),
                                     (2, 1028, 129, 3), (2, 64, 8, 1), (2, 2308, 96, 2),
                                     (2, 772, 300, 2), (2, 1284, 515, 1), (2, 516, 1024, 2)])
def test_minibatch_tf32_weight_gradient(L, N, B, k, tiling):
    # Eq. bp4 on the tensor cores: relative Frobenius error per layer <= 5e-3 against the
    # float64 oracle; everything else on the path stays fp32 and keeps the 1e-5 gate.  Both
    # tilings: one CTA per tile, and CTA pairs with the delta operand resident (N = 2308 gives
    # pairs runs of several tiles that cross a row-block boundary, with ragged last tiles) or, for
    # more than 256 samples, with both operands streaming (B = 300: a ragged last stage; B = 515:
    # more stages than the ring holds; B = 1024: the ring goes round six times per tile).
    cfg = dict(L=L, N=N, B=B, k=k)
    t = _inputs(L, N, B, y="onehot", seed=3 * N + B)
    out, stats = gpu_pass(cfg, t, gw_math=lf.LF_GW_MATH_TF32, tc_tiling=tiling)
    assert stats["gw_math"] == lf.LF_GW_MATH_TF32 and stats["device_status"] == 0
    assert stats["gw_tiling"] == tiling
    ref = oracle_pass(t, want_gw=True)
    worst = compare_all(cfg, out, ref, gw_tf32=True)
    # and against the fp32 CUDA-core contraction of the same delta and a
    out32, _ = gpu_pass(cfg, t, gw_math=lf.LF_GW_MATH_FP32)
    num = (out["gw"].double() - out32["gw"].double()).flatten(1).norm(dim=1)
    den = out32["gw"].double().flatten(1).norm(dim=1)
    assert float((num / den).max()) <= 5e-3
    print("tf32", (L, N, B), worst["gw"], float((num / den).max()))


def test_tf32_pair_kernel_long_runs():
    # N = 6148, B = 64: about eight 256 x 256 tiles per CTA pair, so every accumulator in tensor
    # memory and every barrier is reused several times and every run crosses row blocks.  One
    # layer; the oracle's Eq. bp4 is applied to the GPU's own delta and activations.
    from oracle import lf_oracle as orc
    from lf_testlib import rel_frobenius, TF32_TOL
    L, N, B = 1, 6148, 64
    cfg = dict(L=L, N=N, B=B, k=1)
    t = _inputs(L, N, B, y="onehot", seed=77)
    passes = {}
    for tiling in (lf.LF_TC_TILING_TWO_SM, lf.LF_TC_TILING_ONE_SM):
        out, stats = gpu_pass(cfg, t, gw_math=lf.LF_GW_MATH_TF32, tc_tiling=tiling, repeat=2)
        assert stats["gw_math"] == lf.LF_GW_MATH_TF32 and stats["device_status"] == 0
        assert stats["gw_tiling"] == tiling
        g = out["gw"][0].cpu().numpy()
        ref = orc.grad_w(out["delta"][0].cpu().numpy().astype(np.float64),
                         out["a"][0].cpu().numpy().astype(np.float64))
        assert np.all(np.isfinite(g))
        e = rel_frobenius(g, ref)
        assert e <= TF32_TOL, (tiling, e)
        passes[tiling] = out
    # on one delta and one a (the forward pass of so wide a layer depends on the tiling in its last
    # bits) the two tilings multiply the same truncated operands and add the samples in the same order
    d, a = passes[lf.LF_TC_TILING_TWO_SM]["delta"][0].contiguous(), passes[lf.LF_TC_TILING_TWO_SM]["a"][0].contiguous()
    outs = {}
    for tiling in (lf.LF_TC_TILING_TWO_SM, lf.LF_TC_TILING_ONE_SM):
        gw = torch.full((N, N), float("nan"), device="cuda")
        with lf.Leapfrog(1, N, B, 1) as ctx:
            ctx.set_option(lf.LF_OPT_GW_MATH, lf.LF_GW_MATH_TF32)
            ctx.set_option(lf.LF_OPT_TC_TILING, tiling)
            ctx.grad_w(d, a, gw)
            ctx.sync()
            assert ctx.stats()["gw_tiling"] == tiling and ctx.stats()["device_status"] == 0
        outs[tiling] = gw
    assert torch.equal(outs[lf.LF_TC_TILING_TWO_SM], outs[lf.LF_TC_TILING_ONE_SM])


def test_tf32_tilings_agree_bitwise_beyond_256_samples():
    # more than 256 samples: the CTA pairs stream both operands; they multiply the same truncated
    # operands and add the samples in the same order as the one-SM kernel.  Eq. bp4 alone
    # (lf_grad_w) on one delta and one a, so that nothing else depends on the tiling.
    for N, B in ((1540, 300), (772, 1024)):
        g = torch.Generator(device="cuda"); g.manual_seed(N + B)
        d = torch.empty((B, N), device="cuda").normal_(0.0, 1.0, generator=g)
        a = torch.empty((B, N), device="cuda").uniform_(0.0, 1.0, generator=g)
        outs = {}
        for tiling in (lf.LF_TC_TILING_TWO_SM, lf.LF_TC_TILING_ONE_SM):
            gw = torch.full((N, N), float("nan"), device="cuda")
            with lf.Leapfrog(1, N, B, 1) as ctx:
                ctx.set_option(lf.LF_OPT_GW_MATH, lf.LF_GW_MATH_TF32)
                ctx.set_option(lf.LF_OPT_TC_TILING, tiling)
                for _ in range(2):
                    ctx.grad_w(d, a, gw)
                ctx.sync()
                assert ctx.stats()["gw_tiling"] == tiling and ctx.stats()["device_status"] == 0
            outs[tiling] = gw
        assert torch.equal(outs[lf.LF_TC_TILING_TWO_SM], outs[lf.LF_TC_TILING_ONE_SM]), (N, B)
        ref = d.double().t() @ a.double()      # (a library product only as a second opinion on the size of the error)
        err = float((outs[lf.LF_TC_TILING_TWO_SM].double() - ref).norm() / ref.norm())
        assert err <= 5e-3, err


def test_config4_minibatch_full_size_sampled():
    # L = 16, N = 4096, B = 256, TF32 weight gradients.  The full oracle pass would take minutes,
    # so: (i) the whole chain is checked for a few samples -- samples never mix before Eq.
    # bp3/bp4, so the oracle runs the chain on just those columns; (ii) gb and gw, which sum
    # over all samples, are checked against the oracle's Eq. bp3/bp4 applied to the GPU's own
    # delta and a: gb and two whole layers of gw (Frobenius gate) plus sampled entries elsewhere.
    from oracle import lf_oracle as orc
    from lf_testlib import assert_layer_close, rel_frobenius, TF32_TOL
    cfg, t = lf_inputs.make_config(4, device="cuda")
    L, N, B = cfg["L"], cfg["N"], cfg["B"]
    out, stats = gpu_pass(cfg, t)
    assert stats["gw_math"] == lf.LF_GW_MATH_TF32 and stats["device_status"] == 0
    sel = [0, 101, 255]
    w = t["w"].cpu().numpy()
    sub = {k: t[k][sel].cpu().numpy() for k in ("x", "y")}
    z, a = orc.forward(w, t["b"].cpu().numpy(), sub["x"])
    delta, _, _ = orc.backward_sequential(w, z, a, sub["y"], want_gw=False)
    for name, ref in (("z", z), ("a", a), ("delta", delta)):
        g = out[name][:, sel].cpu().numpy()
        for l in range(ref.shape[0]):
            assert_layer_close(name, l, g[l], ref[l], n_terms=N)
    d_gpu = out["delta"].cpu().numpy().astype(np.float64)
    a_gpu = out["a"].cpu().numpy().astype(np.float64)
    rng = np.random.default_rng(4)
    for l in range(L):
        assert_layer_close("gb", l, out["gb"][l].cpu().numpy(), orc.grad_b(d_gpu[l]), n_terms=B)
        g = out["gw"][l].cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(g))
        if l in (0, L - 1):
            e = rel_frobenius(g, orc.grad_w(d_gpu[l], a_gpu[l]))
            assert e <= TF32_TOL, (l, e)
        else:
            rms = np.sqrt(np.mean(g * g))
            for _ in range(48):
                j, k = int(rng.integers(N)), int(rng.integers(N))
                ref = orc.grad_w_entry(d_gpu[l], a_gpu[l], j, k)
                assert abs(g[j, k] - ref) <= TF32_TOL * max(abs(ref), rms), (l, j, k, g[j, k], ref)


@pytest.mark.parametrize("L,N,B,gw_math", [(3, 516, 1, lf.LF_GW_MATH_AUTO), (2, 388, 70, lf.LF_GW_MATH_FP32),
                                           (3, 772, 256, lf.LF_GW_MATH_TF32), (2, 1028, 300, lf.LF_GW_MATH_TF32)])
def test_grad_w_alone_is_the_layer_slab_of_backward(L, N, B, gw_math):
    # lf_grad_w (Eq. bp4 of one layer as a call of its own) must give bitwise what lf_backward
    # writes for that layer, and so inherits its parity with the oracle.
    cfg = dict(L=L, N=N, B=B, k=2)
    t = _inputs(L, N, B, y="uniform" if B == 1 else "onehot", seed=17 * N + B)
    out, stats = gpu_pass(cfg, t, variant=lf.LF_VARIANT_STREAMS, gw_math=gw_math)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with lf.Leapfrog(L, N, B, 2, stream=st.cuda_stream) as ctx:
        ctx.set_option(lf.LF_OPT_GW_MATH, gw_math)
        for l in range(L):
            g = torch.full((N, N), float("nan"), device="cuda")
            ctx.grad_w(out["delta"][l], out["a"][l], g)
            ctx.sync()
            assert torch.equal(g, out["gw"][l]), l
        assert ctx.stats()["gw_math"] == stats["gw_math"]


@pytest.mark.parametrize("N,k,want", [(512, 2, lf.LF_VARIANT_FUSED), (640, 8, lf.LF_VARIANT_FUSED), (768, 2, lf.LF_VARIANT_PERSISTENT),
                                      (768, 8, lf.LF_VARIANT_FUSED), (1024, 8, lf.LF_VARIANT_PERSISTENT),
                                      (2048, 4, lf.LF_VARIANT_PERSISTENT), (2052, 2, lf.LF_VARIANT_FUSED)])
def test_auto_variant_follows_the_measured_table(N, k, want):
    # LF_VARIANT_AUTO for one sample: the fused pass with whole columns per CTA up to N = 640,
    # leapfrog CTA groups at the widths (and worker counts) where they were measured faster than the
    # fused pass, the fused pass elsewhere; the result passes parity either way.
    cfg = dict(L=9, N=N, B=1, k=k)
    t = _inputs(9, N, 1, seed=N)
    out, stats = gpu_pass(cfg, t)
    assert stats["variant"] == want and stats["device_status"] == 0
    compare_all(cfg, out, oracle_pass(t))


def test_width_beyond_the_persistent_kernels_falls_back_to_streams():
    # N = 16388 is wider than any strip plan of the persistent kernel (and past its documented
    # limit of 16384): AUTO, and an explicit request for the fused pass, must run the stream
    # variant instead, say so in the stats, and still pass parity.
    L, N = 2, 16388
    cfg = dict(L=L, N=N, B=1, k=2)
    t = _inputs(L, N, 1, seed=4)
    ref = oracle_pass(t)
    for variant in (lf.LF_VARIANT_AUTO, lf.LF_VARIANT_FUSED):
        out, stats = gpu_pass(cfg, t, variant=variant)
        assert stats["variant"] == lf.LF_VARIANT_STREAMS and stats["device_status"] == 0
        compare_all(cfg, out, ref)
        del out
        torch.cuda.empty_cache()
