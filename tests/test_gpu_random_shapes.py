"""Seeded random shapes through the per-layer-width and the layer-sharded paths, each compared with the
oracle: widths (multiples of 4 up to 1600, hidden runs included), batch, workers, variant, arithmetic
and tiling are drawn from a fixed seed, so a failure names a reproducible case."""
import random

import numpy as np
import pytest

import paper_1801_04928_b200 as lf
import test_gpu_shard as ts
import test_gpu_widths as tw
from lf_testlib import assert_layer_close
from oracle import lf_oracle as orc

pytestmark = pytest.mark.gpu


def _width_cases(seed, count):
    rng = random.Random(seed)
    cases = []
    for i in range(count):
        L = rng.randint(1, 6)
        if rng.random() < 0.5 and L >= 3:
            h = 4 * rng.randint(1, 300)
            widths = [4 * rng.randint(1, 300)] + [h] * (L - 1) + [4 * rng.randint(1, 300)]
        else:
            widths = [4 * rng.randint(1, 400) for _ in range(L + 1)]
        B = rng.choice([1, 1, 1, 2, 7, 33, 129, 257])
        cases.append((i, widths, B, rng.randint(1, 5), rng.choice(["fp32", "tc"]), rng.choice([0, 1, 2, 3]),
                      rng.choice([0, 1, 2])))
    return cases


@pytest.mark.parametrize("case,widths,B,k,mode,variant,tiling", _width_cases(20260114, 32),
                         ids=lambda v: "-".join(map(str, v)) if isinstance(v, list) else str(v))
def test_random_widths(case, widths, B, k, mode, variant, tiling):
    if B == 1:
        n, cpu, out, stats = tw._run_variant(widths, k, variant, seed=300 + case)
        tw._compare(n, 1, cpu, out)
    elif mode == "fp32":
        n, L, cpu, out, stats = tw._run(widths, B, k, y="onehot", seed=300 + case)
        tw._compare(n, B, cpu, out)
    else:
        n, L, cpu, out, stats = tw._run(widths, B, k, y="onehot", seed=300 + case, gw_math=lf.LF_GW_MATH_AUTO,
                                        delta_math=lf.LF_DELTA_MATH_AUTO, tiling=tiling)
        tw._compare(n, B, cpu, out, tf32=True)
    assert stats["device_status"] == 0


def _shard_cases(seed, count):
    rng = random.Random(seed)
    return [(i, rng.randint(1, 9), 4 * rng.randint(1, 320), rng.randint(1, 5), rng.randint(1, 5),
             rng.choice([0, 1, 2, 3]), rng.choice([None, None, 0.2])) for i in range(count)]


@pytest.mark.parametrize("case,L,N,k,S,variant,eta", _shard_cases(20260115, 16))
def test_random_shards(case, L, N, k, S, variant, eta):
    cpu, t = ts._inputs(L, N, 1, seed=400 + case)
    w, z, a, y = ts._oracle(cpu)
    for r in range(S):
        bufs, stats, owners = ts._shard_pass(L, N, 1, k, S, r, t, variant, sgd_eta=eta)
        assert stats["device_status"] == 0
        d_ref, gw_ref, gb_ref, wrote = orc.backward_shard(w, z, a, y, S, r)
        gw = bufs["gw"].cpu().numpy(); d = bufs["delta"].cpu().numpy()
        for l in range(1, L + 1):
            assert_layer_close("delta", l - 1, d[l - 1], d_ref[l - 1], n_terms=N + 1)
            if not wrote[l - 1]:
                assert np.all(np.isnan(gw[l - 1]))
            elif eta is None:
                assert_layer_close("gw", l - 1, gw[l - 1], gw_ref[l - 1], n_terms=N + 1)
            else:
                want = w[l - 1].astype(np.float64) - eta * gw_ref[l - 1]
                bound = eta * 1e-5 * np.max(np.abs(gw_ref[l - 1])) + 2.0 ** -23 * np.max(np.abs(want))
                assert np.max(np.abs(gw[l - 1] - want)) <= bound


def _uniform_cases(seed, count):
    rng = random.Random(seed)
    cases = []
    for i in range(count):
        B = rng.choice([1, 1, 1, 2, 5, 31, 128, 130, 256, 300])
        cases.append((i, rng.randint(1, 10), 4 * rng.randint(1, 400), B, rng.randint(1, 12),
                      rng.choice([0, 1, 2, 3]) if B == 1 else 0, rng.choice([0, 1, 2]), rng.choice([0, 1, 2]),
                      rng.choice([0, 1, 2]), rng.random() < 0.3))
    return cases


@pytest.mark.parametrize("case,L,N,B,k,variant,gw_math,delta_math,tiling,cross_entropy", _uniform_cases(20260116, 24))
def test_random_uniform_networks(case, L, N, B, k, variant, gw_math, delta_math, tiling, cross_entropy):
    import lf_inputs
    from lf_testlib import compare_all, gpu_pass, oracle_pass
    cpu = lf_inputs.make_inputs(L, N, B, "uniform" if B == 1 else "onehot", lf_inputs.SEED_BASE + 5000 + case, "cpu")
    t = {name: v.cuda() for name, v in cpu.items()}
    cfg = dict(L=L, N=N, B=B, k=k)
    out, stats = gpu_pass(cfg, t, variant=variant, gw_math=gw_math, delta_math=delta_math, tc_tiling=tiling,
                          cost=lf.LF_COST_CROSS_ENTROPY if cross_entropy else lf.LF_COST_QUADRATIC, repeat=2)
    assert stats["device_status"] == 0
    ref = oracle_pass(t, want_gw=False, cross_entropy=cross_entropy)
    compare_all(cfg, out, ref, gw_tf32=(stats["gw_math"] == lf.LF_GW_MATH_TF32))
