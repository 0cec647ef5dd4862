"""Pins for the float64 oracle: each test checks it against something fixed by the paper
or by mathematics that is NOT a re-typing of the oracle's own formula -- closed forms,
invariants, finite differences and brute force on tiny problems, and a hand-worked
rational example.  Mutation tests at the end show that plausible mistakes fail a pin."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import adacons_oracle as oc

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hand_worked_two_steps.txt")
rng = np.random.default_rng(12345)


def rand_G(N, d, seed=0, noise=0.5):
    r = np.random.default_rng(seed)
    return r.standard_normal(d)[None, :] + noise * r.standard_normal((N, d))


def single_step(G, **kw):
    o = oc.AdaConsOracle(G.shape[0], G.shape[1], **kw)
    return o.step(G), o


# ---- P1: identical gradients reduce to that gradient (text after Eq. 8) --------------
@pytest.mark.parametrize("N", [1, 2, 5, 16])
def test_identical_gradients_return_the_gradient_even_with_history(N):
    d = 37
    o = oc.AdaConsOracle(N, d)
    for t in range(4):                      # build some momentum history first
        o.step(rand_G(N, d, seed=t))
    g = np.random.default_rng(9).standard_normal(d)
    r = o.step(np.tile(g, (N, 1)))
    np.testing.assert_allclose(r["psi"], g, rtol=1e-13, atol=1e-15)


# ---- P2: one worker is the identity -----------------------------------------------------
def test_single_worker_is_identity():
    g = np.random.default_rng(1).standard_normal((1, 11))
    r, _ = single_step(g)
    assert r["gamma"].shape == (1, 1) and r["gamma"][0, 0] == 1.0
    np.testing.assert_array_equal(r["psi"], g[0])


# ---- P3: weights sum to one (text before Eq. 12) ---------------------------------------
def test_weights_sum_to_one_over_many_steps():
    N, d = 9, 50
    o = oc.AdaConsOracle(N, d)
    for t in range(30):
        r = o.step(rand_G(N, d, seed=100 + t, noise=2.0))
        assert abs(r["gamma"].sum() - 1.0) < 1e-14


# ---- P4: worker order does not matter (purpose of the sort in Eq. 11) ------------------
def test_worker_permutation_invariance_with_momentum():
    N, d, T = 7, 40, 6
    Gs = [rand_G(N, d, seed=200 + t, noise=1.0) for t in range(T)]
    o1, o2 = oc.AdaConsOracle(N, d), oc.AdaConsOracle(N, d)
    r = np.random.default_rng(3)
    for t in range(T):
        perm = r.permutation(N)             # a different shuffle every step
        r1, r2 = o1.step(Gs[t]), o2.step(Gs[t][perm])
        np.testing.assert_allclose(r2["gamma"][0], r1["gamma"][0][perm], rtol=1e-12)
        np.testing.assert_allclose(r2["psi"], r1["psi"], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(r2["m"], r1["m"], rtol=1e-12)


def test_index_ema_is_not_permutation_invariant():
    """Eq. 10 couples a coefficient to the worker index; Eq. 11 was introduced to remove
    exactly this.  The sort=False variant must therefore fail the invariance."""
    N, d = 5, 30
    G0, G1 = rand_G(N, d, seed=1, noise=1.0), rand_G(N, d, seed=2, noise=1.0)
    perm = np.array([3, 0, 4, 1, 2])
    o1 = oc.AdaConsOracle(N, d, sort=False, beta=0.5)
    o2 = oc.AdaConsOracle(N, d, sort=False, beta=0.5)
    o1.step(G0); o2.step(G0)
    r1, r2 = o1.step(G1), o2.step(G1[perm])
    assert np.max(np.abs(r1["psi"] - r2["psi"])) > 1e-6


# ---- P5: preconditioner form psi = lambda P P^T gbar (Eq. 9) ---------------------------
def test_direction_is_PPt_gbar():
    N, d = 6, 23
    G = rand_G(N, d, seed=5, noise=1.5)
    r, _ = single_step(G)
    P = (G / np.linalg.norm(G, axis=1, keepdims=True)).T          # d x N, unit columns
    gbar = G.mean(axis=0)
    v = P @ (P.T @ gbar)
    # explicit rank-one sum of Eq. 9, written independently of the oracle
    M = sum(np.outer(g, g) / (g @ g) for g in G)
    np.testing.assert_allclose(M @ gbar, v, rtol=1e-12)
    psi = r["psi"]
    cos = psi @ v / np.linalg.norm(psi) / np.linalg.norm(v)
    assert abs(cos - 1.0) < 1e-14
    # the scale is fixed by sum(gamma) = 1:  psi = P P^T gbar / sum_i (P^T gbar)_i/||g_i||
    lam = 1.0 / np.sum((P.T @ gbar) / np.linalg.norm(G, axis=1))
    np.testing.assert_allclose(psi, lam * v, rtol=1e-12)


# ---- P6: subspace objective on tiny quadratics (Eq. 5, Eq. 6) --------------------------
def _quadratic(N, d, seed, isotropic=None):
    r = np.random.default_rng(seed)
    centers = r.standard_normal((N, d))
    if isotropic is None:
        B = r.standard_normal((d, d))
        A = B @ B.T + d * np.eye(d)
    else:
        A = isotropic * np.eye(d)
    w = r.standard_normal(d)

    def f(x):
        diffs = x[None, :] - centers
        return 0.5 * np.mean(np.einsum("nd,de,ne->n", diffs, A, diffs))

    G = (w[None, :] - centers) @ A          # g_i = grad f_i(w); their mean is grad f(w)
    return f, w, G, A


def test_first_order_coefficients_are_the_subspace_gradient_by_finite_differences():
    N, d = 4, 6
    f, w, G, _ = _quadratic(N, d, seed=7)
    P = (G / np.linalg.norm(G, axis=1, keepdims=True)).T
    h, eps = (lambda al: f(w + P @ al)), 1e-6
    fd = np.array([(h(eps * e) - h(-eps * e)) / (2 * eps) for e in np.eye(N)])
    r, _ = single_step(G)
    np.testing.assert_allclose(r["a"][0], fd, rtol=1e-7, atol=1e-9)


def test_aggregate_is_a_descent_direction():
    for seed in range(5):
        f, w, G, _ = _quadratic(5, 8, seed=20 + seed)
        r, _ = single_step(G)
        assert r["Z"][0] > 0
        assert f(w - 1e-4 * r["psi"]) < f(w)


def test_exact_subspace_minimiser_matches_first_order_when_subspace_hessian_is_isotropic():
    """With A = kappa I and mutually orthogonal g_i, P^T A P = kappa I, so the exact
    minimiser of Eq. 5 is the first-order step of Eq. 6 with lambda = 1/kappa.  Brute
    force: exact N x N solve and a grid search over alpha."""
    N, d, kappa = 2, 3, 2.5
    # orthogonal gradients g_i = kappa (w - c_i): pick centers accordingly
    w = np.array([0.3, -0.2, 0.1])
    D = np.array([[1.0, 2.0, 0.0], [-2.0, 1.0, 3.0]])            # rows orthogonal
    assert abs(D[0] @ D[1]) < 1e-15
    centers = w[None, :] - D / kappa
    f = lambda x: 0.5 * kappa * np.mean(np.sum((x[None, :] - centers) ** 2, axis=1))
    G = kappa * (w[None, :] - centers)
    P = (G / np.linalg.norm(G, axis=1, keepdims=True)).T
    gbar = G.mean(axis=0)
    alpha_exact = -np.linalg.solve(P.T @ (kappa * np.eye(d)) @ P, P.T @ gbar)
    # grid search for the minimiser of f(w + P alpha)
    grid = np.linspace(-2, 2, 401)
    vals = np.array([[f(w + P @ np.array([x, y])) for y in grid] for x in grid])
    ix, iy = np.unravel_index(np.argmin(vals), vals.shape)
    np.testing.assert_allclose([grid[ix], grid[iy]], alpha_exact, atol=0.011)
    r, _ = single_step(G)
    np.testing.assert_allclose(-r["a"][0] / kappa, alpha_exact, rtol=1e-12)
    # weights on the raw gradients are alpha_i/||g_i|| normalised; orthogonal => 1/N (P8)
    wts = alpha_exact / np.linalg.norm(G, axis=1)
    np.testing.assert_allclose(r["gamma"][0], wts / wts.sum(), rtol=1e-12)


def test_first_order_is_not_the_exact_minimiser_in_general():
    f, w, G, A = _quadratic(3, 5, seed=31)
    P = (G / np.linalg.norm(G, axis=1, keepdims=True)).T
    alpha_exact = -np.linalg.solve(P.T @ A @ P, P.T @ G.mean(axis=0))
    r, _ = single_step(G)
    a = r["a"][0]
    cos = (-a) @ alpha_exact / np.linalg.norm(a) / np.linalg.norm(alpha_exact)
    assert cos < 1 - 1e-6


# ---- P7: collinear gradients, closed form ----------------------------------------------
def test_collinear_gradients_give_harmonic_weights():
    x = np.random.default_rng(4).standard_normal(19)
    k = np.array([1.0, 1.0, 1.0, 20.0])
    r, _ = single_step(k[:, None] * x[None, :])
    np.testing.assert_allclose(r["gamma"][0], (1 / k) / np.sum(1 / k), rtol=1e-13)
    np.testing.assert_allclose(r["gamma"][0], [20 / 61, 20 / 61, 20 / 61, 1 / 61], rtol=1e-13)
    np.testing.assert_allclose(r["psi"], len(k) / np.sum(1 / k) * x, rtol=1e-13)
    # a sign-flipped collinear worker gets a negative weight and still helps
    k2 = np.array([2.0, -4.0, 5.0])
    r2, _ = single_step(k2[:, None] * x[None, :])
    np.testing.assert_allclose(r2["gamma"][0], (1 / k2) / np.sum(1 / k2), rtol=1e-13)


# ---- P8: orthogonal gradients get equal weights ----------------------------------------
def test_orthogonal_gradients_get_uniform_weights():
    Q, _ = np.linalg.qr(np.random.default_rng(8).standard_normal((12, 5)))
    G = (Q * np.array([0.1, 1.0, 7.0, 30.0, 2.0])).T
    r, _ = single_step(G)
    np.testing.assert_allclose(r["gamma"][0], np.full(5, 0.2), rtol=1e-12)


# ---- P9: homogeneity; first step after reset does not depend on beta -------------------
def test_scale_homogeneity_and_first_step_beta_independence():
    G = rand_G(6, 25, seed=11, noise=1.0)
    base, _ = single_step(G, beta=0.0)
    for beta in (0.3, 0.99):
        r, _ = single_step(G, beta=beta)
        np.testing.assert_allclose(r["gamma"], base["gamma"], rtol=1e-12)
    r, _ = single_step(1e-3 * G)
    np.testing.assert_allclose(r["gamma"], base["gamma"], rtol=1e-12)
    np.testing.assert_allclose(r["psi"], 1e-3 * base["psi"], rtol=1e-12)
    # single step, no momentum: gamma_i = c_i / sum c_j with c_i = <g_i,gbar>/||g_i||^2
    gbar = G.mean(0)
    c = np.array([g @ gbar / (g @ g) for g in G])
    np.testing.assert_allclose(base["gamma"][0], c / c.sum(), rtol=1e-12)


# ---- P10: sum_i N p_i = || sum_j g_j ||^2 ---------------------------------------------
def test_statistics_identity_and_slabs():
    G = rand_G(7, 101, seed=13, noise=3.0)
    p, q = oc.consensus_statistics(G)
    assert abs(G.shape[0] * p.sum() - np.sum(G.sum(0) ** 2)) < 1e-9 * np.sum(G.sum(0) ** 2)
    np.testing.assert_allclose(q, np.linalg.norm(G, axis=1) ** 2, rtol=1e-13)
    # Gram form of Eq. 7, line 3: p_i = (1/N) sum_j <g_i, g_j>
    np.testing.assert_allclose(p, (G @ G.T).sum(axis=1) / G.shape[0], rtol=1e-12)
    ps, qs = oc.consensus_statistics_slabs([G[:, :40], G[:, 40:41], G[:, 41:]])
    np.testing.assert_allclose(ps, p, rtol=1e-13)
    np.testing.assert_allclose(qs, q, rtol=1e-13)


# ---- P11: hand-worked rational example (tests/golden) ----------------------------------
def _load_gold():
    vals = {}
    with open(GOLD) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            vals[k] = np.array([float(Fraction(t)) for t in v])
    return vals


def test_hand_worked_two_step_example():
    g = _load_gold()
    o = oc.AdaConsOracle(3, 2, beta=float(g["beta"][0]))
    for s in ("step1", "step2"):
        r = o.step(g[f"{s}.G"].reshape(3, 2))
        for key in ("p", "q", "a", "gamma"):
            np.testing.assert_allclose(r[key][0], g[f"{s}.{key}"], rtol=1e-14, err_msg=f"{s}.{key}")
        np.testing.assert_allclose(r["m"][0], g[f"{s}.m"], rtol=1e-14)
        np.testing.assert_allclose(r["psi"], g[f"{s}.psi"], rtol=1e-14)


# ---- momentum: independent brute-force restatement via order statistics -----------------
def test_momentum_state_is_the_ema_of_order_statistics():
    """Slot k of the state must equal the EMA over time of the k-th smallest coefficient
    (Eq. 11) -- checked with sorted() on Python lists, bias-corrected closed form."""
    N, d, T, beta = 6, 30, 12, 0.9
    o = oc.AdaConsOracle(N, d, beta=beta)
    hist = []
    for t in range(T):
        G = rand_G(N, d, seed=300 + t, noise=2.0)
        r = o.step(G)
        gbar = G.mean(0)
        hist.append(sorted(float(g @ gbar / np.sqrt(g @ g)) for g in G))
        want = [sum((1 - beta) * beta ** (t - s) * hist[s][k] for s in range(t + 1)) for k in range(N)]
        np.testing.assert_allclose(r["m"][0], want, rtol=1e-12)
        # each worker gets back the slot of its own rank
        ranks = np.argsort(np.argsort(r["a"][0], kind="stable"), kind="stable")
        np.testing.assert_allclose(r["a_tilde"][0], np.array(want)[ranks], rtol=1e-12)


def test_second_worked_example_three_betas():
    """An independently computed example with irrational norms (tests/golden/): both steps for
    beta = 0, 0.5 and 0.99, to the digits the example was given with."""
    g = {}
    with open(os.path.join(os.path.dirname(GOLD), "second_worked_example.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                k, *v = line.split()
                g[k] = np.array([float(t) for t in v])
    tol = dict(rtol=5e-6, atol=0)          # half a unit of the sixth significant digit
    for beta, tag in ((0.0, "beta0"), (0.5, "beta0.5"), (0.99, "beta0.99")):
        o = oc.AdaConsOracle(3, 2, beta=beta)
        r1 = o.step(g["step1.G"].reshape(3, 2))
        r2 = o.step(g["step2.G"].reshape(3, 2))
        for r, s in ((r1, "step1"), (r2, "step2")):
            for key in ("p", "q", "a"):
                np.testing.assert_allclose(r[key][0], g[f"{s}.{key}"], err_msg=f"{tag} {s}.{key}", **tol)
            order = np.argsort(r["a"][0], kind="stable")
            np.testing.assert_array_equal(order, g[f"{s}.pi"].astype(int))
        np.testing.assert_allclose(r1["gamma"][0], g["step1.gamma"], **tol)
        np.testing.assert_allclose(r1["psi"], g["step1.psi"], **tol)
        np.testing.assert_allclose(r2["gamma"][0], g[f"{tag}.step2.gamma"], **tol)
        np.testing.assert_allclose(r2["psi"], g[f"{tag}.step2.psi"], **tol)
        if f"{tag}.step2.m" in g:
            np.testing.assert_allclose(r2["m"][0], g[f"{tag}.step2.m"], **tol)


def test_normalised_weights_closed_forms():
    """normalised_weights alone (Eq. 8, Eq. 12-13): with a~_i = c ||g_i|| every u_i is c and the
    weights are 1/N; in general gamma_i = (a~_i/||g_i||)/sum_j(a~_j/||g_j||), checked in exact
    rationals with integer norms; lambda = 1 keeps Eq. 8's 1/N; the flags of the degenerate cases."""
    q = np.array([4.0, 9.0, 25.0, 1.0])
    u, Z, gamma, flags = oc.normalised_weights(0.7 * np.sqrt(q), q)
    np.testing.assert_allclose(u, 0.7, rtol=1e-15)
    np.testing.assert_allclose(gamma, 0.25, rtol=1e-15)
    assert flags == 0 and abs(Z - 2.8) < 1e-14
    at = [Fraction(3), Fraction(-1, 2), Fraction(5, 4), Fraction(2)]
    norms = [2, 3, 5, 1]
    uf = [x / n for x, n in zip(at, norms)]
    want = [float(x / sum(uf)) for x in uf]
    u, Z, gamma, flags = oc.normalised_weights(np.array([float(x) for x in at]), q)
    np.testing.assert_allclose(gamma, want, rtol=1e-15)
    assert abs(gamma.sum() - 1.0) < 1e-15 and flags == 0
    _, _, g_un, _ = oc.normalised_weights(np.array([float(x) for x in at]), q, normalize=False)
    np.testing.assert_allclose(g_un, [float(x) / 4 for x in uf], rtol=1e-15)
    _, Z, gamma, flags = oc.normalised_weights(np.array([1.0, -1.0]), np.array([1.0, 1.0]))
    assert flags == oc.FLAG_DEGENERATE_Z and np.all(gamma == 0.5) and Z == 0.0
    _, Z, gamma, flags = oc.normalised_weights(np.array([1.0, -3.0]), np.array([1.0, 1.0]))
    assert flags == oc.FLAG_NEG_Z and Z == -2.0
    np.testing.assert_allclose(gamma, [-0.5, 1.5], rtol=1e-15)
    u, _, gamma, _ = oc.normalised_weights(np.array([1.0, 5.0]), np.array([4.0, 0.0]))
    assert u[1] == 0.0 and gamma[1] == 0.0 and gamma[0] == 1.0          # a zero gradient gets no weight


# ---- variants (Table 2) ------------------------------------------------------------------
def test_unnormalised_variant_matches_eq8():
    G = rand_G(5, 17, seed=17, noise=1.0)
    r, _ = single_step(G, normalize=False, momentum=False)
    N = G.shape[0]
    want = sum(sum(G[i] @ G[j] for j in range(N)) / (G[i] @ G[i]) * G[i] for i in range(N)) / N**2
    np.testing.assert_allclose(r["psi"], want, rtol=1e-12)
    # identical gradients still reduce to averaging without the normalisation
    g = np.arange(1.0, 6.0)
    r2, _ = single_step(np.tile(g, (4, 1)), normalize=False, momentum=False)
    np.testing.assert_allclose(r2["psi"], g, rtol=1e-14)


def test_momentum_off_leaves_state_untouched():
    o = oc.AdaConsOracle(4, 10, momentum=False)
    r = o.step(rand_G(4, 10, seed=1))
    assert np.all(r["m"] == 0)
    np.testing.assert_array_equal(r["a"], r["a_tilde"])


# ---- per-segment ("layer-wise") mode ----------------------------------------------------
def test_per_segment_mode_is_the_global_rule_on_each_slice():
    N, d = 5, 60
    off = [0, 7, 7, 31, 60]                      # includes an empty segment
    o = oc.AdaConsOracle(N, d, seg_offsets=off, per_segment=True, beta=0.8)
    subs = [oc.AdaConsOracle(N, off[s + 1] - off[s], beta=0.8) for s in range(4)]
    for t in range(3):
        G = rand_G(N, d, seed=400 + t, noise=1.0)
        r = o.step(G)
        for s in range(4):
            if off[s + 1] == off[s]:                 # no columns: no layer, no flag, state untouched
                assert r["flags"][s] == 0 and not r["m"][s].any()
                continue
            rs = subs[s].step(G[:, off[s]:off[s + 1]])
            np.testing.assert_allclose(r["psi"][off[s]:off[s + 1]], rs["psi"], rtol=1e-13)
            np.testing.assert_allclose(r["gamma"][s], rs["gamma"][0], rtol=1e-13)
    # offsets without per_segment only describe the layout
    og = oc.AdaConsOracle(N, d, seg_offsets=off, per_segment=False)
    assert og.S == 1


# ---- degenerate inputs --------------------------------------------------------------------
def test_zero_row_and_all_zero_and_nonfinite():
    G = rand_G(4, 12, seed=3)
    G[2] = 0
    r, _ = single_step(G)
    assert r["flags"][0] & oc.FLAG_ZERO_ROW and r["gamma"][0, 2] == 0
    assert abs(r["gamma"].sum() - 1) < 1e-14
    r, _ = single_step(np.zeros((3, 5)))
    assert r["flags"][0] & oc.FLAG_DEGENERATE_Z
    np.testing.assert_array_equal(r["gamma"][0], np.full(3, 1 / 3))
    np.testing.assert_array_equal(r["psi"], np.zeros(5))
    G = rand_G(3, 8, seed=4)
    o = oc.AdaConsOracle(3, 8)
    o.step(G)
    m_before = o.m.copy()
    G[1, 3] = np.inf
    r = o.step(G)
    assert r["flags"][0] & oc.FLAG_NONFINITE
    np.testing.assert_array_equal(r["gamma"][0], np.full(3, 1 / 3))
    np.testing.assert_array_equal(o.m, m_before)


def test_negative_normaliser_is_flagged():
    x = np.array([1.0, 2.0, -1.0])
    r, _ = single_step(np.stack([10 * x, -x]))
    assert r["flags"][0] & oc.FLAG_NEG_Z
    assert abs(r["gamma"].sum() - 1) < 1e-14


# ---- storage rounding ------------------------------------------------------------------
def test_bf16_rounding_matches_torch():
    import torch
    r = np.random.default_rng(0)
    x = np.concatenate([r.standard_normal(5000) * 10.0 ** r.integers(-30, 30, 5000),
                        [0.0, 1.0, 1.00390625, 1.01171875, -3.0e-40, 1e-45, 3.38e38, 3.4e38]])
    x32 = x.astype(np.float32).astype(np.float64)       # values where one rounding suffices
    want = torch.from_numpy(x32.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    got = oc.round_to_storage(x32, "bf16")
    np.testing.assert_array_equal(got, want)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert oc.round_to_storage(np.array([1.00390625]), "bf16")[0] == 1.0
    assert oc.round_to_storage(np.array([1.01171875]), "bf16")[0] == 1.015625
    np.testing.assert_array_equal(oc.round_to_storage(x, "f32"), x.astype(np.float32).astype(np.float64))


# ---- mutation tests: a plausible mistake in the oracle must fail a pin ----------------
def test_mutant_single_norm_power_fails_eq9_pin():
    """Dividing by the norm once instead of twice (weights proportional to a~_i) still sums
    to one and still returns identical gradients, but is not parallel to P P^T gbar."""
    G = rand_G(5, 14, seed=23, noise=2.0)
    P = (G / np.linalg.norm(G, axis=1, keepdims=True)).T
    v = P @ (P.T @ G.mean(0))
    c = oc.coefficients(*oc.consensus_statistics(G), np.zeros(5), 0.99)
    wrong = c["a_tilde"] / c["a_tilde"].sum()
    psi = oc.combine(G, wrong)
    cos = psi @ v / np.linalg.norm(psi) / np.linalg.norm(v)
    assert abs(cos - 1) > 1e-6


def test_mutant_unsorted_momentum_fails_hand_example():
    g = _load_gold()
    o = oc.AdaConsOracle(3, 2, beta=0.5, sort=False)
    o.step(g["step1.G"].reshape(3, 2))
    r = o.step(g["step2.G"].reshape(3, 2))
    assert np.max(np.abs(r["gamma"][0] - g["step2.gamma"])) > 1e-3


def test_sort_direction_is_immaterial():
    """Sorting descending mirrors the slots of the state and changes nothing else, so the
    paper's silence on the direction of S does not affect the result."""
    g = _load_gold()
    m = 0.5 * np.sort(g["step1.a"])[::-1]
    m = 0.5 * m + 0.5 * np.sort(g["step2.a"])[::-1]
    np.testing.assert_allclose(m[::-1], g["step2.m"], rtol=1e-14)


def test_mutant_transposed_operand_fails_statistics_identity():
    G = rand_G(6, 6, seed=29, noise=2.0)                 # square so the transpose type-checks
    p, _ = oc.consensus_statistics(G.T)
    assert abs(6 * p.sum() - np.sum(G.sum(0) ** 2)) > 1e-6
