"""Randomised property checks of the oracle (hypothesis): the invariants the paper fixes must hold
for arbitrary shapes, scales and histories, not only for the hand-picked cases of the pin tests."""
import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import adacons_oracle as oc


def matrices(draw, n_max=9, d_max=24):
    n = draw(st.integers(1, n_max))
    d = draw(st.integers(1, d_max))
    seed = draw(st.integers(0, 2**31 - 1))
    scale = 10.0 ** draw(st.integers(-6, 6))
    noise = draw(st.sampled_from([0.0, 0.1, 1.0, 10.0]))
    r = np.random.default_rng(seed)
    return scale * (r.standard_normal(d)[None, :] + noise * r.standard_normal((n, d)))


mat = st.composite(matrices)()


@settings(max_examples=150, deadline=None, derandomize=True)
@given(mat, st.floats(0.0, 0.999), st.integers(0, 3))
def test_weights_sum_to_one_and_result_is_in_the_span(G, beta, history):
    n, d = G.shape
    o = oc.AdaConsOracle(n, d, beta=beta)
    r0 = np.random.default_rng(1)
    for _ in range(history):
        o.step(r0.standard_normal((n, d)))
    r = o.step(G)
    assert abs(r["gamma"].sum() - 1.0) < 1e-9
    np.testing.assert_allclose(r["psi"], r["gamma"][0] @ G, rtol=1e-9, atol=1e-300)
    assert np.all(np.diff(np.sort(r["a"][0])) >= 0)


@settings(max_examples=100, deadline=None, derandomize=True)
@given(mat, st.integers(0, 2**31 - 1))
def test_first_step_is_permutation_and_scale_equivariant(G, seed):
    n, d = G.shape
    perm = np.random.default_rng(seed).permutation(n)
    r1 = oc.AdaConsOracle(n, d).step(G)
    if r1["flags"][0] & (oc.FLAG_DEGENERATE_Z | oc.FLAG_NONFINITE):
        return
    a = np.sort(r1["a"][0])
    if n > 1 and np.min(np.diff(a)) < 1e-9 * max(1.0, np.abs(a).max()):
        return                                       # (near-)ties: the slot assignment is not unique
    if abs(r1["Z"][0]) < 1e-6 * np.abs(r1["u"][0]).sum():
        return                                       # ill-conditioned normaliser
    r2 = oc.AdaConsOracle(n, d).step(G[perm])
    np.testing.assert_allclose(r2["gamma"][0], r1["gamma"][0][perm], rtol=1e-7)
    r3 = oc.AdaConsOracle(n, d).step(3.5 * G)
    np.testing.assert_allclose(r3["gamma"][0], r1["gamma"][0], rtol=1e-7)
    np.testing.assert_allclose(r3["psi"], 3.5 * r1["psi"], rtol=1e-7, atol=1e-300)


@settings(max_examples=60, deadline=None, derandomize=True)
@given(st.integers(1, 8), st.integers(1, 16), st.integers(0, 2**31 - 1), st.floats(0.0, 0.99))
def test_identical_gradients_after_any_history(n, d, seed, beta):
    r = np.random.default_rng(seed)
    o = oc.AdaConsOracle(n, d, beta=beta)
    for _ in range(3):
        o.step(r.standard_normal((n, d)))
    g = r.standard_normal(d) + 0.1
    res = o.step(np.tile(g, (n, 1)))
    if res["flags"][0] & oc.FLAG_DEGENERATE_Z:
        return
    np.testing.assert_allclose(res["psi"], g, rtol=1e-8, atol=1e-12)
