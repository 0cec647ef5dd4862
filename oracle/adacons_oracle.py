"""Float64 CPU oracle for Adaptive Consensus (AdaCons) gradient aggregation.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
aggregation computes.  It exists so that the CUDA library can be checked against
something that was written from the paper alone; it shares no code with the CUDA
path, never imports it, and must never be used as a fallback by the product.
Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import it.

Every function cites the passage of the paper (arXiv 2411.03742) it follows.
All arithmetic is IEEE float64 (numpy); inputs are the stored gradient values
(fp32 or bf16) converted exactly to float64 by the caller.

Notation (paper, Section 3):
    G        N x d matrix, row i = worker gradient g_i(w_t)
    gbar     mean gradient, (1/N) sum_i g_i                       (text before Eq. 7)
    p_i      <g_i, gbar>                                           (Eq. 7)
    q_i      ||g_i||^2
    a_i      first-order subspace coefficient <g_i, gbar>/||g_i||  (Eq. 7, lambda = 1,
             sign chosen so that the result is subtracted by the optimiser, Eq. 4)
    S        sorting operator, ascending, stable                   (Eq. 11)
    m        EMA of the *sorted* coefficients, slot k = k-th order statistic (Eq. 11)
    a_tilde  S^{-1}(m): smoothed coefficient handed back to its worker (Eq. 11)
    u_i      a_tilde_i / ||g_i||: weight on the raw (un-normalised) g_i, because the
             subspace matrix P has unit columns g_i/||g_i||           (Eq. 8, Eq. 9)
    gamma_i  u_i / sum_j u_j: weights constrained to sum to one     (Eq. 12, Eq. 13)
    psi      sum_i gamma_i g_i                                       (Eq. 12)

Pins (tests/test_oracle_pins.py): identical gradients return that gradient, N=1 is
the identity, sum(gamma)=1, worker-permutation invariance, psi parallel to P P^T gbar
(Eq. 9), finite-difference subspace gradient and exact subspace minimiser on tiny
quadratics (Eq. 5-6), closed forms for collinear and orthogonal gradients, a
hand-worked two-step rational example (tests/golden/), homogeneity, and the identity
sum_i N p_i = ||sum_j g_j||^2.  No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

# Status flags reported next to the coefficients (numerical degeneracies are not errors).
FLAG_ZERO_ROW = 1       # some ||g_i|| = 0: that worker gets a_i = u_i = gamma_i = 0
FLAG_DEGENERATE_Z = 2   # sum_i u_i is zero / negligible / non-finite: fall back to 1/N
FLAG_NONFINITE = 4      # a non-finite statistic was seen: fall back to 1/N, state kept
FLAG_NEG_Z = 8          # sum_i u_i < 0: computed as defined, reported

DEFAULT_BETA = 0.99     # the value used in the paper's ablation (Table 2 caption)
DEGENERATE_REL = 1e-12  # |Z| <= DEGENERATE_REL * sum|u_i| counts as Z = 0


def mean_gradient(G: np.ndarray) -> np.ndarray:
    """gbar_k = (1/N) sum_j g_jk  -- Monte-Carlo estimate of the full gradient
    (sentence before Eq. 7)."""
    G = np.asarray(G, dtype=np.float64)
    return G.sum(axis=0) / G.shape[0]


def consensus_statistics(G: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """p_i = <g_i, gbar>, q_i = ||g_i||^2 for every worker (Eq. 7, numerator and the
    squared denominator)."""
    G = np.asarray(G, dtype=np.float64)
    gbar = mean_gradient(G)
    p = np.sum(G * gbar[None, :], axis=1)
    q = np.sum(G * G, axis=1)
    return p, q


def consensus_statistics_slabs(slabs) -> tuple[np.ndarray, np.ndarray]:
    """Same as consensus_statistics for a matrix delivered as column slabs
    (an iterable of N x d_j arrays).  Both sums of Eq. 7 are sums over columns, and
    gbar is defined column by column, so the slabs simply add."""
    p = q = None
    for slab in slabs:
        ps, qs = consensus_statistics(slab)
        p = ps if p is None else p + ps
        q = qs if q is None else q + qs
    return p, q


def first_order_coefficients(p: np.ndarray, q: np.ndarray) -> np.ndarray:
    """a_i = <g_i, gbar> / ||g_i||  (Eq. 7 with lambda = 1; Algorithm 1, step 2).
    A zero gradient has no direction: its coefficient is 0."""
    p = np.asarray(p, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    a = np.zeros_like(p)
    nz = q > 0
    a[nz] = p[nz] / np.sqrt(q[nz])
    return a


def subspace_momentum(a: np.ndarray, m_prev: np.ndarray, beta: float,
                      sort: bool = True) -> tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Sorted subspace momentum (Eq. 11):
        m_t      = beta m_{t-1} + (1-beta) S(a)
        a_tilde  = S^{-1}(m_t)
    S sorts ascending and is stable (ties keep worker order).  With sort=False this is
    the index-coupled EMA of Eq. 10.  Returns (m_t, a_tilde, pi) where pi[k] is the
    worker whose coefficient occupies sorted slot k."""
    a = np.asarray(a, dtype=np.float64)
    n = a.shape[0]
    pi = np.argsort(a, kind="stable") if sort else np.arange(n)
    m = beta * np.asarray(m_prev, dtype=np.float64) + (1.0 - beta) * a[pi]
    a_tilde = np.empty(n, dtype=np.float64)
    a_tilde[pi] = m
    return m, a_tilde, pi


def normalised_weights(a_tilde, q, *, normalize: bool = True):
    """From the (smoothed) subspace coefficients to the weights on the raw gradients
    (Eq. 8 and the text before Eq. 12, Eq. 13): returns (u, Z, gamma, flags).

    normalize=False keeps lambda = 1 and the 1/N of Eq. 8: gamma_i = u_i / N."""
    a_tilde = np.asarray(a_tilde, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    n = a_tilde.shape[0]
    flags = 0
    uniform = np.full(n, 1.0 / n)
    # P has unit columns, psi = P alpha  =>  weight on g_i is alpha_i / ||g_i||  (Eq. 8)
    u = np.zeros(n, dtype=np.float64)
    nz = q > 0
    u[nz] = a_tilde[nz] / np.sqrt(q[nz])
    Z = float(np.sum(u))
    if normalize:
        # the weights are rescaled so that they add up to one  (text before Eq. 12, Eq. 13)
        if (not np.isfinite(Z)) or abs(Z) <= DEGENERATE_REL * float(np.sum(np.abs(u))):
            gamma = uniform
            flags |= FLAG_DEGENERATE_Z
        else:
            gamma = u / Z
            if Z < 0:
                flags |= FLAG_NEG_Z
    else:
        gamma = u / n
    return u, Z, gamma, flags


def coefficients(p, q, m_prev, beta: float = DEFAULT_BETA, *, momentum: bool = True,
                 sort: bool = True, normalize: bool = True) -> dict:
    """Algorithm 1 steps 2-3: from the 2N statistics to the N weights gamma.

    momentum=False skips Eq. 11 (a_tilde = a, state untouched); sort=False uses Eq. 10;
    normalize=False keeps lambda = 1 and the 1/N of Eq. 8: gamma_i = u_i / N
    (which gives plain averaging for identical gradients, as the text after Eq. 8 says).
    """
    p = np.asarray(p, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    m_prev = np.asarray(m_prev, dtype=np.float64)
    n = p.shape[0]
    flags = 0
    if np.any(q == 0):
        flags |= FLAG_ZERO_ROW
    uniform = np.full(n, 1.0 / n)
    if not (np.all(np.isfinite(p)) and np.all(np.isfinite(q))):
        a = np.full(n, np.nan)
        # a non-finite statistic: plain mean, momentum state left as it was
        return dict(p=p, q=q, a=a, a_tilde=a.copy(), u=np.full(n, np.nan), Z=np.nan,
                    gamma=uniform, m=m_prev.copy(), pi=np.arange(n),
                    flags=flags | FLAG_NONFINITE)
    a = first_order_coefficients(p, q)
    if momentum:
        m, a_tilde, pi = subspace_momentum(a, m_prev, beta, sort=sort)
    else:
        m, a_tilde, pi = m_prev.copy(), a.copy(), np.arange(n)
    u, Z, gamma, wflags = normalised_weights(a_tilde, q, normalize=normalize)
    return dict(p=p, q=q, a=a, a_tilde=a_tilde, u=u, Z=Z, gamma=gamma, m=m, pi=pi,
                flags=flags | wflags)


def combine(G: np.ndarray, gamma: np.ndarray) -> np.ndarray:
    """psi_k = sum_i gamma_i g_ik  (Eq. 12)."""
    G = np.asarray(G, dtype=np.float64)
    return np.sum(np.asarray(gamma, dtype=np.float64)[:, None] * G, axis=0)


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round float64 values to the storage format of the output ("f32" or "bf16"),
    round-to-nearest-even, and return them as float64.  The paper is silent on the
    output type; the library writes the input's type with one rounding at the end."""
    x = np.asarray(x, dtype=np.float64)
    if dtype == "f32":
        with np.errstate(over="ignore"):
            return x.astype(np.float32).astype(np.float64)
    if dtype == "bf16":
        # bf16: 8 significant bits (1 implicit + 7 stored), fp32's exponent range.
        out = x.copy()
        fin = np.isfinite(x) & (x != 0)
        _, e = np.frexp(x[fin])                     # x = f * 2^e, 0.5 <= |f| < 1
        quantum = np.ldexp(1.0, np.maximum(e, -125) - 8)
        r = np.rint(x[fin] / quantum) * quantum     # rint rounds half to even
        r[np.abs(r) > 3.3895313892515355e38] = np.inf * np.sign(r[np.abs(r) > 3.3895313892515355e38])
        out[fin] = r
        return out
    raise ValueError(f"unknown storage dtype {dtype!r}")


class AdaConsOracle:
    """Stateful aggregation psi_t = AdaCons({g_i}, t)  (Eq. 12), global ("model-wise")
    or per segment ("layer-wise", Section 4, first paragraph on the experimental setup:
    the same rule applied to each layer's slice with its own momentum state).

    seg_offsets: None for one global segment, else S+1 ascending column offsets with
    seg_offsets[0] = 0 and seg_offsets[S] = d.  per_segment=False ignores the offsets
    for the arithmetic (they only describe the layout)."""

    def __init__(self, N: int, d: int, *, beta: float = DEFAULT_BETA,
                 seg_offsets=None, per_segment: bool = False, momentum: bool = True,
                 sort: bool = True, normalize: bool = True):
        self.N, self.d = int(N), int(d)
        self.beta = float(beta)
        self.momentum, self.sort, self.normalize = momentum, sort, normalize
        if per_segment and seg_offsets is not None:
            off = np.asarray(seg_offsets, dtype=np.int64)
            assert off[0] == 0 and off[-1] == d and np.all(np.diff(off) >= 0)
            self.offsets = off
        else:
            self.offsets = np.array([0, d], dtype=np.int64)
        self.S = len(self.offsets) - 1
        self.reset()

    def reset(self) -> None:
        """alpha^m_0 = 0 and t = 0 (the paper does not give an initial value; zero needs
        no bias correction because the sum-to-one normalisation cancels any common
        scale of m)."""
        self.m = np.zeros((self.S, self.N), dtype=np.float64)
        self.t = 0

    def step(self, G: np.ndarray, storage: str | None = None) -> dict:
        """One aggregation.  Returns per-segment arrays (S x N) of p, q, a, a_tilde,
        gamma, the new state m, flags (S,), psi (d,) and, if `storage` is given, `out`
        = psi rounded to that format."""
        G = np.asarray(G, dtype=np.float64)
        assert G.shape == (self.N, self.d)
        keys = ("p", "q", "a", "a_tilde", "u", "gamma")
        res = {k: np.zeros((self.S, self.N)) for k in keys}
        res["Z"] = np.zeros(self.S)
        res["flags"] = np.zeros(self.S, dtype=np.int64)
        psi = np.zeros(self.d, dtype=np.float64)
        for s in range(self.S):
            lo, hi = int(self.offsets[s]), int(self.offsets[s + 1])
            Gs = G[:, lo:hi]
            p, q = consensus_statistics(Gs)
            c = coefficients(p, q, self.m[s], self.beta, momentum=self.momentum,
                             sort=self.sort, normalize=self.normalize)
            self.m[s] = c["m"]
            for k in keys:
                res[k][s] = c[k]
            res["Z"][s] = c["Z"]
            # a segment without columns is no layer (Section 4, layer-wise aggregation): its
            # all-zero statistics are not a degenerate gradient and raise no flag
            res["flags"][s] = c["flags"] if hi > lo else 0
            psi[lo:hi] = combine(Gs, c["gamma"])
        self.t += 1
        res["m"] = self.m.copy()
        res["psi"] = psi
        if storage is not None:
            res["out"] = round_to_storage(psi, storage)
        return res
