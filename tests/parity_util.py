"""Shared pieces of the GPU parity tests: tolerances, comparisons and the near-tie rule.

Tolerances
  coefficients (p, q, a, a~, gamma, state m): 1e-5 relative, with the floor
      |x_gpu - x_or| <= 1e-5 * max(|x_or_i|, 1e-3 * max_j |x_or_j|)
  output: |out_gpu - psi_or| <= 1e-5 * max|g|  (fp32 storage)  or  4e-3 * max|g|  (bf16 storage),
  and additionally the tighter element-wise bound that follows from the coefficient tolerance:
      |out_gpu - psi_or| <= 1e-5 * sum_i |gamma_i g_ik| + one rounding to the storage format.

Near-ties.  Eq. 11 sorts the coefficients, and a sort is discontinuous: the sorted values (hence
the state m) depend continuously on a, but two workers whose coefficients agree to within the
kernel's fp32 accumulation error may legitimately come out in the other order.  The oracle is
never told about the kernel's order.  When the two orders differ, the test itself checks that the
kernel's order is a valid answer -- it sorts the ORACLE's coefficients to within twice the
coefficient tolerance -- and then forms the expectation for the later stages from the oracle's own
state by an index operation, a~_i = m_oracle[kernel's slot of worker i], followed by the oracle's
own normalisation and combination.  Every such worker is counted; the counts are printed in the
terminal summary, and tests on recipes whose coefficients are well separated demand zero.
"""
import numpy as np
import torch

from oracle import adacons_oracle as oc

COEFF_RTOL = 1e-5
OUT_TOL = {"f32": 1e-5, "bf16": 4e-3}
ULP = {"f32": 2.0 ** -23, "bf16": 2.0 ** -8}

# test name -> [steps compared, coefficient sets compared, workers that took a swapped slot]
SLOT_TALLY = {}


def tally(what, sets, swapped):
    t = SLOT_TALLY.setdefault(what, [0, 0, 0])
    t[0] += 1
    t[1] += int(sets)
    t[2] += int(swapped)


def to_f64(G: torch.Tensor) -> np.ndarray:
    return G.detach().cpu().to(torch.float64).numpy()


def assert_coeffs(got, want, what, floor_frac=1e-3):
    got, want = np.asarray(got, dtype=np.float64).ravel(), np.asarray(want, dtype=np.float64).ravel()
    floor = floor_frac * np.max(np.abs(want)) if want.size else 0.0
    tol = COEFF_RTOL * np.maximum(np.abs(want), floor)
    bad = np.abs(got - want) > tol
    assert not bad.any(), f"{what}: max rel err {np.max(np.abs(got - want) / np.maximum(np.abs(want), floor)):.3e}"


def assert_coeffs_by_set(got, want, what):
    for s in range(want.shape[0]):
        assert_coeffs(got[s], want[s], f"{what} set {s}")


def assert_output(out_t, res, G64, dtype, what, offsets=None):
    got = to_f64(out_t)
    psi = res["psi"]
    gmax = float(np.max(np.abs(G64))) if G64.size else 0.0
    err = np.abs(got - psi)
    S = res["gamma"].shape[0]
    # The 1e-5 * max|g| bound presumes weights of total mass sum|gamma_i| ~ 1.  A segment of a few
    # columns can have sum_i u_i close to zero and hence huge weights of both signs; there the bound
    # scales with the mass of the weights (their own 1e-5 relative error times |g|).
    if S == 1:
        mass = (np.abs(res["gamma"][0])[:, None] * np.abs(G64)).sum(axis=0)
        wsum = np.full(G64.shape[1], np.abs(res["gamma"][0]).sum())
    else:
        mass, wsum = np.zeros(G64.shape[1]), np.ones(G64.shape[1])
        for s in range(S):
            lo, hi = offsets[s], offsets[s + 1]
            mass[lo:hi] = (np.abs(res["gamma"][s])[:, None] * np.abs(G64[:, lo:hi])).sum(axis=0)
            wsum[lo:hi] = np.abs(res["gamma"][s]).sum()
    loose = OUT_TOL[dtype] * gmax * np.maximum(1.0, wsum) + 1e-300
    assert np.all(err <= loose), f"{what}: max err {err.max():.3e} vs max|g| {gmax:.3e}"
    tight = 1e-5 * mass + ULP[dtype] * np.abs(psi) + 1e-45
    assert np.all(err <= tight), f"{what}: tight bound violated by {np.max(err / tight):.3f}x"


def ranks_of(a):
    """Stable ascending rank of every worker, per set (rows of a 2-D array)."""
    order = np.argsort(a, axis=1, kind="stable")
    r = np.empty_like(order)
    np.put_along_axis(r, order, np.broadcast_to(np.arange(a.shape[1]), a.shape), axis=1)
    return r


def with_kernel_slot_order(c, r_gpu, *, normalize=True, what=""):
    """c: the oracle's own result for ONE coefficient set (dict from oracle.coefficients or a row
    of AdaConsOracle.step: a, m, q, flags, ...).  r_gpu[i]: the slot the kernel gave worker i.
    Returns (expectation, number of workers whose slot differs from the oracle's).

    Equal orders: the oracle's result, untouched.  Otherwise the kernel's order must sort the
    oracle's a to within 2 * COEFF_RTOL (relative, with the usual floor); the expectation is then
    a~ = m_oracle[r_gpu] (an index operation) pushed through the oracle's own normalisation."""
    r_or = ranks_of(np.asarray(c["a"])[None, :])[0]
    swapped = int(np.count_nonzero(r_or != r_gpu))
    if swapped == 0:
        return c, 0
    a = np.asarray(c["a"])
    sorted_by_gpu = a[np.argsort(r_gpu, kind="stable")]
    slack = 2 * COEFF_RTOL * np.maximum(np.abs(a).max() * 1e-3, np.abs(sorted_by_gpu[:-1]))
    assert np.all(np.diff(sorted_by_gpu) >= -slack), f"{what}: the kernel's slot order does not sort the oracle's coefficients"
    a_tilde = np.asarray(c["m"])[r_gpu]
    u, Z, gamma, wflags = oc.normalised_weights(a_tilde, c["q"], normalize=normalize)
    keep = int(c["flags"]) & (oc.FLAG_ZERO_ROW | oc.FLAG_NONFINITE)
    out = dict(c)
    out.update(a_tilde=a_tilde, u=u, Z=Z, gamma=gamma, flags=keep | wflags)
    return out, swapped


def oracle_step(orc, G64, dtype, a_gpu, *, what, sort=True, momentum=True, normalize=True, allow_swaps=True):
    """One step of the (pure) oracle, with the near-tie rule applied set by set where the kernel's
    slot order differs.  a_gpu: the kernel's first-order coefficients (sets x N), used only for
    their ORDER.  Returns the dict of AdaConsOracle.step."""
    res = orc.step(G64, storage=dtype)
    S = res["a"].shape[0]
    if not (sort and momentum):
        tally(what, S, 0)
        return res
    r_gpu = ranks_of(np.asarray(a_gpu))
    total = 0
    for s in range(S):
        c = {k: res[k][s] for k in ("a", "q", "a_tilde", "u", "gamma")}
        c.update(m=res["m"][s], Z=res["Z"][s], flags=res["flags"][s])
        c2, n = with_kernel_slot_order(c, r_gpu[s], normalize=normalize, what=f"{what} set {s}")
        if n == 0:
            continue
        total += n
        for k in ("a_tilde", "u", "gamma"):
            res[k][s] = c2[k]
        res["Z"][s], res["flags"][s] = c2["Z"], c2["flags"]
        lo, hi = int(orc.offsets[s]), int(orc.offsets[s + 1])
        res["psi"][lo:hi] = oc.combine(G64[:, lo:hi], c2["gamma"])
    if total:
        res["out"] = oc.round_to_storage(res["psi"], dtype)
    tally(what, S, total)
    assert allow_swaps or total == 0, f"{what}: {total} workers took a swapped slot on a recipe with well-separated coefficients"
    return res


def streamed_statistics(G, slab=2_000_000, threads=8):
    """p, q of the oracle over ALL columns of a device matrix: column slabs are copied to the host
    and handed to oracle.consensus_statistics by a few threads; the slab results are added in slab
    order (both statistics are sums over columns)."""
    from concurrent.futures import ThreadPoolExecutor
    N, d = G.shape
    starts = list(range(0, d, slab))

    def one(c0):
        return oc.consensus_statistics(to_f64(G[:, c0:min(d, c0 + slab)]))

    with ThreadPoolExecutor(max_workers=threads) as ex:
        parts = list(ex.map(one, starts))
    return sum(p for p, _ in parts), sum(q for _, q in parts)


def shifted_pass1_applies(N, d, dtype, pitch=None):
    """Whether pass 1 takes the per-class tensor maps (ADACONS_INFO_LAST_PATH 10) for rows `pitch` elements apart
    that the staged kernels cannot take: up to 64 workers, a body of at least one 16-byte group, and classes of
    rows thick enough (bf16 always; fp32 from 4 rows per class on, k = 16 / gcd(pitch in bytes, 16) classes)."""
    eb = 4 if dtype == "f32" else 2
    rem = ((pitch or d) * eb) % 16
    k = 1 if rem == 0 else 16 // (rem & -rem)
    return N <= 64 and d >= 4 * (16 // eb) and (dtype == "bf16" or N >= 4 * k)
