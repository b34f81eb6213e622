"""Pins for the float64 CPU oracle (no GPU needed).

The paper (arXiv 1801.04928) prints no worked numbers, so the oracle is tied to what the
mathematics fixes: the gradient is the derivative of the cost (central finite differences
of C, which only needs the forward pass), closed forms of special networks, the structure
Eq. bp3/bp4 impose, and Theorem 1 (every layer saved exactly once) together with a hand
trace of Algorithm 1.  Each test names the mistake it is there to catch.
"""
import os

import numpy as np
import pytest

from oracle import lf_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _net(L, N, B, seed, y_kind="uniform"):
    r = np.random.default_rng(seed)
    w = r.normal(0.0, 1.0 / np.sqrt(N), size=(L, N, N))
    b = r.normal(0.0, 1.0, size=(L, N))
    x = r.uniform(0.0, 1.0, size=(B, N))
    if y_kind == "uniform":
        y = r.uniform(0.0, 1.0, size=(B, N))
    else:
        y = np.zeros((B, N))
        y[np.arange(B), r.integers(0, N, size=B)] = 1.0
    return w, b, x, y


def _cost(w, b, x, y):
    _, a = orc.forward(w, b, x)
    return orc.cost(a, y)


# ---- sigma ---------------------------------------------------------------------------------

def test_sigmoid_values_and_symmetry():
    # sigma(0) = 1/2, sigma(ln 3) = 3/4, sigma(-t) = 1 - sigma(t); no overflow far out.
    assert orc.sigma(0.0) == 0.5
    assert abs(orc.sigma(np.log(3.0)) - 0.75) < 1e-15
    for t in (0.3, 2.0, 17.0, 700.0, 800.0):
        assert abs(orc.sigma(-t) - (1.0 - orc.sigma(t))) < 1e-15
        assert np.isfinite(orc.sigma(t)) and np.isfinite(orc.sigma(-t))
    assert orc.sigma(800.0) == 1.0 and orc.sigma(-800.0) == 0.0
    # sigma' peaks at 1/4 in 0 and matches a central difference of sigma elsewhere.
    assert orc.sigma_prime(0.0) == 0.25
    for t in (-3.0, -0.7, 0.4, 2.5):
        h = 1e-6
        fd = (orc.sigma(t + h) - orc.sigma(t - h)) / (2 * h)
        assert abs(fd - orc.sigma_prime(t)) < 1e-9


# ---- forward: closed forms -----------------------------------------------------------------

def test_forward_zero_weights_gives_half_activations():
    L, N, B = 3, 4, 2
    w = np.zeros((L, N, N)); b = np.zeros((L, N))
    x = np.random.default_rng(0).uniform(size=(B, N))
    z, a = orc.forward(w, b, x)
    assert np.array_equal(a[0], x)                    # Eq. x
    assert np.all(z == 0.0) and np.all(a[1:] == 0.5)


def test_forward_row_column_orientation():
    # One non-zero weight w[j=2][k=0]: only neuron 2 sees input 0.  A transposed index
    # would light up neuron 0 from input 2 instead.
    N = 4
    w = np.zeros((1, N, N)); w[0, 2, 0] = 3.0
    b = np.zeros((1, N))
    x = np.array([[1.0, 0.0, 5.0, 0.0]])
    z, a = orc.forward(w, b, x)
    assert np.array_equal(z[0, 0], np.array([0.0, 0.0, 3.0, 0.0]))
    # bias is ADDED to the weighted input (the reading of Eq. z)
    b[0, 1] = -2.0
    z, _ = orc.forward(w, b, x)
    assert np.array_equal(z[0, 0], np.array([0.0, -2.0, 3.0, 0.0]))


def test_cost_definition():
    a = np.zeros((2, 2, 3)); a[1] = [[1.0, 2.0, 3.0], [0.0, 0.0, 1.0]]
    y = np.array([[0.0, 2.0, 1.0], [1.0, 0.0, 1.0]])
    # 1/2 (1 + 0 + 4) + 1/2 (1 + 0 + 0) = 3: summed over samples, no 1/B.
    assert orc.cost(a, y) == 3.0


# ---- the gradient is the derivative of the cost --------------------------------------------

@pytest.mark.parametrize("L,N,B,y_kind", [(1, 3, 1, "uniform"), (2, 4, 1, "onehot"),
                                          (3, 5, 3, "uniform"), (4, 8, 1, "uniform"),
                                          (4, 6, 3, "onehot")])
def test_gradients_match_central_differences(L, N, B, y_kind):
    # Catches: dropped term, wrong sign, transposed w in bp2, a^{l} used for a^{l-1} in
    # bp4, sigma' taken at the wrong layer, a 1/B factor, missing bias.
    w, b, x, y = _net(L, N, B, seed=100 * L + 10 * N + B, y_kind=y_kind)
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y)
    h = 1e-5
    fd_w = np.empty_like(w)
    for idx in np.ndindex(*w.shape):
        wp = w.copy(); wp[idx] += h
        wm = w.copy(); wm[idx] -= h
        fd_w[idx] = (_cost(wp, b, x, y) - _cost(wm, b, x, y)) / (2 * h)
    fd_b = np.empty_like(b)
    for idx in np.ndindex(*b.shape):
        bp = b.copy(); bp[idx] += h
        bm = b.copy(); bm[idx] -= h
        fd_b[idx] = (_cost(w, bp, x, y) - _cost(w, bm, x, y)) / (2 * h)
    for l in range(L):  # per layer: deep layers have much smaller gradients
        sw = np.max(np.abs(fd_w[l])); sb = np.max(np.abs(fd_b[l]))
        assert np.max(np.abs(gw[l] - fd_w[l])) <= 2e-7 * sw + 1e-12
        assert np.max(np.abs(gb[l] - fd_b[l])) <= 2e-7 * sb + 1e-12


def test_delta_is_dC_dz_per_sample():
    # delta^l_b = dC/dz^l_b: perturbing b^l shifts z^l of every sample, so a single-sample
    # run's gb is that sample's delta.  The batch run must reproduce each sample's chain.
    L, N, B = 3, 5, 4
    w, b, x, y = _net(L, N, B, seed=7)
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y)
    gw_sum = np.zeros_like(gw)
    for s in range(B):
        zs, as_ = orc.forward(w, b, x[s:s + 1])
        ds, gws, gbs = orc.backward_sequential(w, zs, as_, y[s:s + 1])
        assert np.array_equal(zs[:, 0], z[:, s]) and np.array_equal(as_[:, 0], a[:, s])
        assert np.array_equal(ds[:, 0], delta[:, s])
        assert np.array_equal(gbs, ds[:, 0])          # Eq. bp3, B = 1
        gw_sum += gws
    assert np.allclose(gw, gw_sum, rtol=1e-14, atol=0)
    assert np.allclose(gb, delta.sum(axis=1), rtol=1e-14, atol=0)


# ---- structure imposed by Eq. bp3 / bp4 for a single sample --------------------------------

def test_single_sample_invariants_rank_one():
    L, N = 4, 7
    w, b, x, y = _net(L, N, 1, seed=3)
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y)
    assert np.array_equal(gb, delta[:, 0, :])                       # Eq. bp3
    for l in range(L):
        g = gw[l]
        assert np.linalg.matrix_rank(g, tol=1e-13 * np.max(np.abs(g))) == 1
        # all 2x2 minors vanish
        j0, k0 = np.unravel_index(np.argmax(np.abs(g)), g.shape)
        minors = g * g[j0, k0] - np.outer(g[:, k0], g[j0, :])
        assert np.max(np.abs(minors)) <= 1e-15 * np.max(np.abs(g)) ** 2 + 1e-300
        # row sums: sum_k gw_jk = delta_j * sum_k a^{l-1}_k ; column sums likewise.  The
        # row factor must be delta^l and the column factor a^{l-1} (NOT a^l).
        assert np.allclose(g.sum(axis=1), delta[l, 0] * a[l, 0].sum(), rtol=1e-12, atol=0)
        assert np.allclose(g.sum(axis=0), a[l, 0] * delta[l, 0].sum(), rtol=1e-12, atol=0)


# ---- closed forms of the backward pass -----------------------------------------------------

def test_single_layer_textbook_gradient():
    # L = 1: dC/dw = ((sigma(wx+b) - y) sigma'(wx+b)) x^T, written here with numpy.
    N = 6
    w, b, x, y = _net(1, N, 1, seed=11)
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y)
    zz = w[0] @ x[0] + b[0]
    s = 1.0 / (1.0 + np.exp(-zz))
    d = (s - y[0]) * s * (1.0 - s)
    assert np.allclose(z[0, 0], zz, rtol=1e-14)
    assert np.allclose(delta[0, 0], d, rtol=1e-13)
    assert np.allclose(gw[0], np.outer(d, x[0]), rtol=1e-13)
    assert np.allclose(gb[0], d, rtol=1e-13)


def test_zero_weights_closed_form():
    # w = 0, b = 0: a^l = 1/2, sigma' = 1/4, delta^L = (1/2 - y)/4, delta^l = 0 below,
    # gw^L = delta^L (a^{L-1})^T with a^{L-1} = 1/2 (or x when L = 1), gw^l = 0 below.
    L, N = 3, 4
    w = np.zeros((L, N, N)); b = np.zeros((L, N))
    x = np.array([[0.1, 0.2, 0.3, 0.4]]); y = np.array([[1.0, 0.0, 0.25, 0.5]])
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y)
    dL = (0.5 - y[0]) / 4.0
    assert np.array_equal(delta[L - 1, 0], dL)
    assert np.all(delta[:L - 1] == 0.0) and np.all(gw[:L - 1] == 0.0)
    assert np.array_equal(gw[L - 1], np.outer(dL, np.full(N, 0.5)))


def test_identity_weights_decouple_into_scalar_chains():
    # w = I: neuron i only talks to neuron i; delta^l_i = delta^L_i prod_{m=l}^{L-1} sigma'(z^m_i).
    L, N = 4, 5
    r = np.random.default_rng(5)
    w = np.stack([np.eye(N)] * L); b = r.normal(size=(L, N))
    x = r.uniform(size=(1, N)); y = r.uniform(size=(1, N))
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y)
    sp = a[1:, 0] * (1.0 - a[1:, 0])                                 # sigma'(z^l) via a^l
    expect = (a[L, 0] - y[0]) * sp[L - 1]
    assert np.allclose(delta[L - 1, 0], expect, rtol=1e-13)
    for l in range(L - 1, 0, -1):
        expect = expect * sp[l - 1]
        assert np.allclose(delta[l - 1, 0], expect, rtol=1e-12)


def test_bp2_uses_the_transpose():
    # A single off-diagonal weight w^{2}[j=1][k=3] routes delta^2_1 to neuron 3 of layer 1
    # (and to nobody else).  Using w instead of w^T would route delta^2_3 to neuron 1.
    N = 4
    w_up = np.zeros((N, N)); w_up[1, 3] = 2.0
    d_up = np.array([[10.0, 20.0, 30.0, 40.0]])
    z_l = np.zeros((1, N))                                           # sigma'(0) = 1/4
    d = orc.delta_step(w_up, d_up, z_l)
    assert np.array_equal(d[0], np.array([0.0, 0.0, 0.0, 2.0 * 20.0 * 0.25]))


def test_scalar_network_product_chain():
    # N = 1: everything is a scalar recurrence.
    L = 5
    r = np.random.default_rng(9)
    w = r.normal(size=(L, 1, 1)); b = r.normal(size=(L, 1))
    x = np.array([[0.7]]); y = np.array([[0.2]])
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y)
    act = [0.7]
    for l in range(L):
        act.append(1.0 / (1.0 + np.exp(-(w[l, 0, 0] * act[-1] + b[l, 0]))))
    d = (act[L] - 0.2) * act[L] * (1 - act[L])
    for l in range(L, 0, -1):
        assert np.isclose(delta[l - 1, 0, 0], d, rtol=1e-12)
        assert np.isclose(gw[l - 1, 0, 0], d * act[l - 1], rtol=1e-12)
        if l > 1:
            d = d * w[l - 1, 0, 0] * act[l - 1] * (1 - act[l - 1])


def test_step_functions_agree_with_full_backward():
    L, N, B = 3, 6, 2
    w, b, x, y = _net(L, N, B, seed=21)
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y)
    assert np.array_equal(orc.output_error(a[L], y, z[L - 1]), delta[L - 1])
    assert np.array_equal(orc.delta_step(w[2], delta[2], z[1]), delta[1])
    assert np.array_equal(orc.grad_b(delta[1]), gb[1])
    assert np.array_equal(orc.grad_w(delta[1], a[1]), gw[1])
    assert orc.grad_w_entry(delta[1], a[1], 4, 2) == gw[1, 4, 2]


def test_float_weight_flavour_promotes_exactly():
    L, N, B = 3, 8, 2
    w, b, x, y = _net(L, N, B, seed=2)
    w32 = w.astype(np.float32)
    z64, a64 = orc.forward(w32.astype(np.float64), b, x)
    z32, a32 = orc.forward(w32, b, x)
    assert np.array_equal(z64, z32) and np.array_equal(a64, a32)
    r64 = orc.backward_sequential(w32.astype(np.float64), z64, a64, y)
    r32 = orc.backward_sequential(w32, z32, a32, y)
    for u, v in zip(r64, r32):
        assert np.array_equal(u, v)


# ---- Algorithm 1: coverage, ownership, schedule invariance ---------------------------------

def _simulate_algorithm1_paper_numbering(Lp, k):
    """Integer-only walk of the printed pseudocode in the paper's own layer numbering
    (layers 1..Lp, layer 1 = input).  Returns {paper layer: saver}, parent = -1."""
    saver = {}
    for i in range(Lp - 1, Lp - k, -1):          # i = L-1 ... L-k+1
        if i >= 2:
            saver[i] = -1
    for t in range(k):
        j = t
        while j < Lp - k - 1:
            i = 0
            while i < k:
                l = Lp - 1 - j - i
                if i == k - 1:
                    assert l not in saver
                    saver[l] = t
                i += 1
            j += k
    return saver


def test_hand_trace_fixture_matches_pseudocode_walk():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "algorithm1_trace_L8_k3.txt"))
            if ln.strip() and not ln.startswith("#")]
    golden = {int(p): int(s) for p, s in rows}
    sim = _simulate_algorithm1_paper_numbering(8, 3)
    assert {p: s for p, s in golden.items() if s != -9} == sim
    # and the oracle's literal run (library L = 7 weight layers) names the same savers
    L, N, k = 7, 3, 3
    w, b, x, y = _net(L, N, 1, seed=1)
    z, a = orc.forward(w, b, x)
    _, _, _, writer, writes, _ = orc.backward_leapfrog(w, z, a, y, k)
    for p, s in golden.items():
        l = p - 1
        assert writer[l - 1] == (-1 if s == -9 else s)   # the top layer: parent (reading)
    assert np.all(writes == 1)


@pytest.mark.parametrize("threads", [True, False])
def test_leapfrog_is_bitwise_the_sequential_result_for_every_k(threads):
    L, N, B = 9, 5, 2
    w, b, x, y = _net(L, N, B, seed=77)
    z, a = orc.forward(w, b, x)
    ref = orc.backward_sequential(w, z, a, y)
    for k in range(1, L + 3):
        delta, gw, gb, writer, writes, bp2 = orc.backward_leapfrog(w, z, a, y, k,
                                                                   threads=threads)
        assert np.array_equal(delta, ref[0]) and np.array_equal(gw, ref[1])
        assert np.array_equal(gb, ref[2])
        assert np.all(writes == 1)                                   # Theorem 1
        ke = min(k, L)
        for l in range(1, L + 1):
            if l >= L - ke + 1:
                assert writer[l - 1] == -1                           # parent's layers
            else:
                assert writer[l - 1] == (L - l) % ke                 # owner residue class


def test_leapfrog_ownership_matches_pseudocode_for_many_sizes():
    N = 2
    for Lp in range(2, 22):
        L = Lp - 1
        w, b, x, y = _net(L, N, 1, seed=Lp)
        z, a = orc.forward(w, b, x)
        for k in range(1, Lp + 1):
            sim = _simulate_algorithm1_paper_numbering(Lp, min(k, L))
            _, _, _, writer, writes, _ = orc.backward_leapfrog(w, z, a, y, k, want_gw=False,
                                                               threads=False)
            assert np.all(writes == 1)
            for p in range(2, Lp):                                   # below the top layer
                assert sim[p] == writer[p - 2], (Lp, k, p)
            assert writer[L - 1] == -1


def test_leapfrog_recomputes_the_chain_in_every_thread():
    # Every thread applies bp2 at every layer from its start down to its last save: the
    # redundant work the cost model f' = f1 + f2 + f3/k leaves out.  Count it.
    L, N, k = 12, 2, 4
    w, b, x, y = _net(L, N, 1, seed=4)
    z, a = orc.forward(w, b, x)
    *_, bp2 = orc.backward_leapfrog(w, z, a, y, k, want_gw=False)
    expect = k - 1                                                   # parent
    for j in range(k):
        jj = j
        while jj < L - k:
            expect += k
            jj += k
    assert bp2 == expect and bp2 > L - 1


# ---- the gradient-descent step that consumes Eq. bp4 (not in the paper) -------------------------
def test_sgd_step_lowers_the_cost_by_eta_times_gradient_norm():
    # First-order check of sign and scale, against the cost itself: for a small step
    # C(w - eta g) - C(w) = -eta |g|^2 + O(eta^2).  A wrong sign gives +eta |g|^2, a missing
    # eta or a step along something other than dC/dw changes the ratio.
    L, N, B = 3, 6, 2
    w, b, x, y = _net(L, N, B, seed=21)
    z, a = orc.forward(w, b, x)
    _, gw, _ = orc.backward_sequential(w, z, a, y)
    c0 = orc.cost(a, y)
    g2 = float(np.sum(gw * gw))
    for eta in (1e-3, 1e-4):
        w1 = orc.sgd_step(w, gw, eta)
        _, a1 = orc.forward(w1, b, x)
        drop = orc.cost(a1, y) - c0
        assert drop < 0
        assert abs(drop / (-eta * g2) - 1.0) < 50 * eta      # second-order remainder shrinks with eta


def test_sgd_step_is_affine_in_eta_and_leaves_w_alone_at_zero():
    L, N = 2, 5
    w, b, x, y = _net(L, N, 1, seed=22)
    z, a = orc.forward(w, b, x)
    _, gw, _ = orc.backward_sequential(w, z, a, y)
    assert np.array_equal(orc.sgd_step(w, gw, 0.0), w)
    s1 = orc.sgd_step(w, gw, 0.25) - w
    s2 = orc.sgd_step(w, gw, 0.5) - w
    np.testing.assert_allclose(s2, 2.0 * s1, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(s1, -0.25 * gw, rtol=1e-12, atol=1e-15)


def test_sgd_step_closed_form_on_the_zero_network():
    # w = 0, b = 0: a = 1/2 everywhere, delta^L = (1/2 - y)/4 and the lower deltas vanish, so
    # only the top matrix moves: w_new^L[j][k] = -eta (1/2 - y_j) / 8.
    L, N, eta = 3, 4, 0.7
    w = np.zeros((L, N, N)); b = np.zeros((L, N))
    x = np.linspace(0.1, 0.9, N)[None, :]
    y = np.array([[1.0, 0.0, 0.25, 0.5]])
    z, a = orc.forward(w, b, x)
    _, gw, _ = orc.backward_sequential(w, z, a, y)
    w1 = orc.sgd_step(w, gw, eta)
    assert np.all(w1[: L - 1] == 0.0)
    want = np.repeat((-eta * (0.5 - y[0]) / 8.0)[:, None], N, axis=1)
    np.testing.assert_allclose(w1[L - 1], want, rtol=1e-13, atol=1e-16)


def test_sgd_step_float_weight_flavour_promotes_exactly():
    rng = np.random.default_rng(23)
    w32 = rng.standard_normal((2, 4, 4)).astype(np.float32)
    gw = rng.standard_normal((2, 4, 4))
    assert np.array_equal(orc.sgd_step(w32, gw, 0.3), orc.sgd_step(w32.astype(np.float64), gw, 0.3))


# ---- the second cost function: cross-entropy of the sigmoid outputs -----------------------------
def _cost_ce(w, b, x, y):
    _, a = orc.forward(w, b, x)
    return orc.cost(a, y, cross_entropy=True)


def test_cross_entropy_cost_definition():
    # one layer, zero weights and biases: a = 1/2, so C = N ln 2 per sample whatever y is
    N = 5
    w = np.zeros((1, N, N)); b = np.zeros((1, N))
    x = np.full((2, N), 0.3); y = np.array([[1, 0, 0.25, 0.5, 0.75], [0, 1, 1, 0, 0.1]], dtype=float)
    _, a = orc.forward(w, b, x)
    assert abs(orc.cost(a, y, cross_entropy=True) - 2 * N * np.log(2.0)) < 1e-13
    # and against the formula written out with numpy on a random net
    w, b, x, y = _net(2, 4, 3, seed=31)
    _, a = orc.forward(w, b, x)
    want = -np.sum(y * np.log(a[-1]) + (1 - y) * np.log(1 - a[-1]))
    assert abs(orc.cost(a, y, cross_entropy=True) - want) < 1e-12 * abs(want)


@pytest.mark.parametrize("L,N,B,y_kind", [(1, 3, 1, "uniform"), (3, 5, 3, "uniform"), (4, 6, 2, "onehot")])
def test_cross_entropy_gradients_match_central_differences(L, N, B, y_kind):
    # Eq. bp1 with grad_a C of the cross-entropy, then the same bp2-bp4: every dC/dw and dC/db
    # against central differences of the cross-entropy cost itself.
    w, b, x, y = _net(L, N, B, seed=500 + 100 * L + 10 * N + B, y_kind=y_kind)
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y, cross_entropy=True)
    h = 1e-5
    for l in range(L):
        fd_w = np.empty((N, N)); fd_b = np.empty((N,))
        for j in range(N):
            for k in range(N):
                wp = w.copy(); wp[l, j, k] += h
                wm = w.copy(); wm[l, j, k] -= h
                fd_w[j, k] = (_cost_ce(wp, b, x, y) - _cost_ce(wm, b, x, y)) / (2 * h)
            bp = b.copy(); bp[l, j] += h
            bm = b.copy(); bm[l, j] -= h
            fd_b[j] = (_cost_ce(w, bp, x, y) - _cost_ce(w, bm, x, y)) / (2 * h)
        assert np.max(np.abs(gw[l] - fd_w)) <= 2e-7 * np.max(np.abs(fd_w)) + 1e-12
        assert np.max(np.abs(gb[l] - fd_b)) <= 2e-7 * np.max(np.abs(fd_b)) + 1e-12


def test_cross_entropy_output_error_collapses_to_a_minus_y():
    # grad_a C (.) sigma'(z) = (a - y)/(a(1-a)) * a(1-a) = a - y: the closed form an implementation
    # may use; below the top layer the two costs share Eq. bp2-bp4, so their deltas differ exactly
    # by what the top deltas differ.
    w, b, x, y = _net(3, 6, 2, seed=33)
    z, a = orc.forward(w, b, x)
    d_top = orc.output_error(a[-1], y, z[-1], cross_entropy=True)
    np.testing.assert_allclose(d_top, a[-1] - y, rtol=1e-12, atol=1e-15)
    d_ce, _, _ = orc.backward_sequential(w, z, a, y, cross_entropy=True)
    np.testing.assert_allclose(d_ce[1], orc.delta_step(w[2], d_top, z[1]), rtol=1e-13, atol=0)


# ---- other activation functions (the paper's equations are stated for a general sigma) ---------
@pytest.mark.parametrize("act", ["tanh", "relu"])
@pytest.mark.parametrize("L,N,B", [(1, 3, 1), (3, 5, 3), (4, 6, 2)])
def test_other_activations_match_central_differences(act, L, N, B):
    # The same finite-difference pin as for the sigmoid.  The rectifier is not differentiable where
    # z = 0; with these seeds no pre-activation comes within 1e-3 of it (checked), so a step of
    # 1e-5 never crosses the kink.
    w, b, x, y = _net(L, N, B, seed=700 + 100 * L + 10 * N + B)
    with orc.activation(act):
        z, a = orc.forward(w, b, x)
        if act == "relu":
            assert np.min(np.abs(z)) > 1e-3
        delta, gw, gb = orc.backward_sequential(w, z, a, y)
        h = 1e-5
        for l in range(L):
            fd_w = np.empty((N, N)); fd_b = np.empty((N,))
            for j in range(N):
                for k in range(N):
                    wp = w.copy(); wp[l, j, k] += h
                    wm = w.copy(); wm[l, j, k] -= h
                    fd_w[j, k] = (_cost(wp, b, x, y) - _cost(wm, b, x, y)) / (2 * h)
                bp = b.copy(); bp[l, j] += h
                bm = b.copy(); bm[l, j] -= h
                fd_b[j] = (_cost(w, bp, x, y) - _cost(w, bm, x, y)) / (2 * h)
            assert np.max(np.abs(gw[l] - fd_w)) <= 2e-7 * max(np.max(np.abs(fd_w)), 1e-3) + 1e-12
            assert np.max(np.abs(gb[l] - fd_b)) <= 2e-7 * max(np.max(np.abs(fd_b)), 1e-3) + 1e-12
    # and the setting does not leak
    assert abs(orc.forward(np.zeros((1, 2, 2)), np.zeros((1, 2)), np.ones((1, 2)))[1][1, 0, 0] - 0.5) < 1e-15


def test_activation_values_and_closed_forms():
    w = np.zeros((1, 3, 3)); b = np.array([[-2.0, 0.0, 1.5]]); x = np.ones((1, 3)); y = np.zeros((1, 3))
    with orc.activation("tanh"):
        z, a = orc.forward(w, b, x)
        np.testing.assert_allclose(a[1, 0], np.tanh(b[0]), rtol=1e-15)
        d, _, _ = orc.backward_sequential(w, z, a, y)
        np.testing.assert_allclose(d[0, 0], np.tanh(b[0]) * (1 - np.tanh(b[0]) ** 2), rtol=1e-14)
    with orc.activation("relu"):
        z, a = orc.forward(w, b, x)
        assert np.array_equal(a[1, 0], [0.0, 0.0, 1.5])
        d, _, _ = orc.backward_sequential(w, z, a, y)
        assert np.array_equal(d[0, 0], [0.0, 0.0, 1.5])           # (a - y) * [z > 0], 0 at z = 0
    with pytest.raises(KeyError):
        orc.set_activation("softplus")


# ---- layers of different widths ------------------------------------------------------------------
def _net_widths(widths, B, seed):
    r = np.random.default_rng(seed)
    sz = orc.sizes_widths(widths, B)
    w = np.concatenate([r.normal(0.0, 1.0 / np.sqrt(widths[l - 1]), size=widths[l] * widths[l - 1])
                        for l in range(1, len(widths))])
    b = r.normal(0.0, 1.0, size=sz["b"])
    x = r.uniform(0.0, 1.0, size=sz["x"])
    y = r.uniform(0.0, 1.0, size=sz["y"])
    return w, b, x, y


def _cost_widths(widths, w, b, x, y, B, cross_entropy=False):
    _, a = orc.forward_widths(widths, w, b, x)
    aL = orc.split(a, widths, "a", B)[-1]
    return orc.cost(aL[None], y.reshape(B, -1), cross_entropy=cross_entropy)


@pytest.mark.parametrize("act,cross_entropy", [("sigmoid", False), ("sigmoid", True), ("tanh", False)])
@pytest.mark.parametrize("widths,B", [([3, 5, 2], 1), ([4, 2, 6, 3], 3), ([2, 7, 7, 1, 5], 2)])
def test_widths_gradients_match_central_differences(widths, B, act, cross_entropy):
    # Every dC/dw and dC/db of a network whose layers differ in width, against central differences
    # of the cost (forward pass only).  Catches a block offset or a row length taken from the wrong
    # layer: with n_l != n_{l-1} either one reads another layer's numbers.
    w, b, x, y = _net_widths(widths, B, seed=900 + sum(widths) + B)
    with orc.activation(act):
        z, a = orc.forward_widths(widths, w, b, x)
        delta, gw, gb = orc.backward_widths(widths, w, z, a, y, cross_entropy=cross_entropy)
        h = 1e-5
        fd_w = np.empty_like(w); fd_b = np.empty_like(b)
        for i in range(w.size):
            wp = w.copy(); wp[i] += h
            wm = w.copy(); wm[i] -= h
            fd_w[i] = (_cost_widths(widths, wp, b, x, y, B, cross_entropy) -
                       _cost_widths(widths, wm, b, x, y, B, cross_entropy)) / (2 * h)
        for i in range(b.size):
            bp = b.copy(); bp[i] += h
            bm = b.copy(); bm[i] -= h
            fd_b[i] = (_cost_widths(widths, w, bp, x, y, B, cross_entropy) -
                       _cost_widths(widths, w, bm, x, y, B, cross_entropy)) / (2 * h)
    for g, f in zip(orc.split(gw, widths, "w"), orc.split(fd_w, widths, "w")):
        assert np.max(np.abs(g - f)) <= 3e-7 * np.max(np.abs(f)) + 1e-12
    for g, f in zip(orc.split(gb, widths, "b"), orc.split(fd_b, widths, "b")):
        assert np.max(np.abs(g - f)) <= 3e-7 * np.max(np.abs(f)) + 1e-12
    # Eq. bp3 for one sample: gb is delta itself
    if B == 1:
        assert np.array_equal(gb, delta)


def test_widths_with_one_common_width_is_the_uniform_oracle_bitwise():
    L, N, B = 4, 6, 3
    w, b, x, y = _net(L, N, B, seed=77)
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y)
    widths = [N] * (L + 1)
    z2, a2 = orc.forward_widths(widths, w.ravel(), b.ravel(), x.ravel())
    d2, gw2, gb2 = orc.backward_widths(widths, w.ravel(), z2, a2, y.ravel())
    assert np.array_equal(z2, z.ravel()) and np.array_equal(a2, a.ravel())
    assert np.array_equal(d2, delta.ravel()) and np.array_equal(gw2, gw.ravel()) and np.array_equal(gb2, gb.ravel())
    dce, _, _ = orc.backward_sequential(w, z, a, y, cross_entropy=True)
    d3, _, _ = orc.backward_widths(widths, w.ravel(), z2, a2, y.ravel(), cross_entropy=True)
    assert np.array_equal(d3, dce.ravel())


def test_widths_network_is_the_zero_padded_uniform_network():
    # Embed widths [4, 7, 3, 5] into the uniform network of width 7 with zero weights to and from the
    # padding neurons.  The padding neurons fire (sigma(b) != 0) but nothing reads them, and adding
    # exact zeros changes no sum: the real entries must come out bitwise equal, the gradients by the
    # padding weights that leave real neurons (rows of padding neurons) need not vanish, those into
    # padding columns of layer 1 multiply x-padding = 0.
    widths, B = [4, 7, 3, 5], 2
    L, N = len(widths) - 1, max(widths)
    w, b, x, y = _net_widths(widths, B, seed=5)
    W = np.zeros((L, N, N)); Bv = np.zeros((L, N)); X = np.zeros((B, N)); Y = np.zeros((B, N))
    for l, (wl, bl) in enumerate(zip(orc.split(w, widths, "w"), orc.split(b, widths, "b")), start=1):
        W[l - 1, :widths[l], :widths[l - 1]] = wl
        Bv[l - 1, :widths[l]] = bl
    X[:, :widths[0]] = x.reshape(B, -1)
    Y[:, :widths[-1]] = y.reshape(B, -1)
    Z, A = orc.forward(W, Bv, X)
    # the padded outputs must not contribute to delta^L: give them the target they already hit
    Y[:, widths[-1]:] = A[-1][:, widths[-1]:]
    D, GW, GB = orc.backward_sequential(W, Z, A, Y)
    z, a = orc.forward_widths(widths, w, b, x)
    d, gw, gb = orc.backward_widths(widths, w, z, a, y)
    for l, (zl, dl, gwl, gbl) in enumerate(zip(orc.split(z, widths, "z", B), orc.split(d, widths, "z", B),
                                               orc.split(gw, widths, "w"), orc.split(gb, widths, "b")), start=1):
        assert np.array_equal(zl, Z[l - 1][:, :widths[l]])
        assert np.array_equal(dl, D[l - 1][:, :widths[l]])
        assert np.array_equal(gwl, GW[l - 1][:widths[l], :widths[l - 1]])
        assert np.array_equal(gbl, GB[l - 1][:widths[l]])
    for l, al in enumerate(orc.split(a, widths, "a", B)):
        assert np.array_equal(al, A[l][:, :widths[l]])


# ---- the schedule on S GPUs ---------------------------------------------------------------------
def test_shards_cover_every_layer_once_and_add_up_to_the_sequential_pass():
    # Catches: a layer no GPU owns or two GPUs own, a GPU that starts its chain from the wrong delta,
    # gradients emitted before the chain reached the layer.
    L, N, B = 7, 5, 2
    w, b, x, y = _net(L, N, B, seed=404)
    z, a = orc.forward(w, b, x)
    delta, gw, gb = orc.backward_sequential(w, z, a, y)
    for S in range(1, L + 3):
        count = np.zeros(L, dtype=int)
        for r in range(S):
            d, g, v, wrote = orc.backward_shard(w, z, a, y, S, r)
            assert np.array_equal(d, delta)                      # every GPU has the whole chain
            for l in range(1, L + 1):
                mine = (L - l) % S == r
                assert bool(wrote[l - 1]) == mine
                if mine:
                    assert np.array_equal(g[l - 1], gw[l - 1]) and np.array_equal(v[l - 1], gb[l - 1])
                else:
                    assert np.all(np.isnan(g[l - 1])) and np.all(np.isnan(v[l - 1]))
            count += wrote
        assert np.all(count == 1)


def test_shard_classes_are_the_thread_classes_of_algorithm_1():
    # With k GPUs for k threads: all layers one thread of Algorithm 1 saves lie in one shard, and
    # different threads' layers lie in different shards (the parent's top layers aside, which the
    # pseudocode handles before it constructs the threads).
    L, N, B = 11, 3, 1
    w, b, x, y = _net(L, N, B, seed=405)
    z, a = orc.forward(w, b, x)
    for k in range(1, L + 1):
        _, _, _, writer, writes, _ = orc.backward_leapfrog(w, z, a, y, k, threads=False)
        cls = {}
        for l in range(1, L + 1):
            j = int(writer[l - 1])
            if j >= 0:
                cls.setdefault(j, set()).add((L - l) % k)
        assert all(len(v) == 1 for v in cls.values())
        residues = [next(iter(v)) for v in cls.values()]
        assert len(set(residues)) == len(residues)


def test_shard_rejects_bad_rank():
    w, b, x, y = _net(2, 3, 1, seed=1)
    z, a = orc.forward(w, b, x)
    with pytest.raises(ValueError):
        orc.backward_shard(w, z, a, y, 2, 2)
