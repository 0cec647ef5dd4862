"""Measured parity margins per benchmark configuration (not a test: a report).

    python tests/parity_report.py            # needs a B200 and the built library

For each configuration: the largest relative error of the coefficients (p, q, a, gamma, state m)
against the float64 oracle and the largest output error relative to max|g|, over the steps run.
Configurations 3-5 use the oracle's statistics over all columns (streamed through the host) and
the output on 200k sampled columns; configurations 1-2 are compared element by element.
"""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from oracle import adacons_oracle as oc                         # noqa: E402
from paper_2411_03742_b200 import binding as ac, workloads as wl  # noqa: E402
import test_parity_gpu as tp                                      # noqa: E402


def rel(got, want):
    got, want = np.asarray(got, float).ravel(), np.asarray(want, float).ravel()
    floor = 1e-3 * np.abs(want).max()
    return float(np.max(np.abs(got - want) / np.maximum(np.abs(want), floor)))


def report(name, steps, per_segment=False, full_oracle=True):
    w = wl.WORKLOADS[name]
    dev = torch.device("cuda:0")
    off = wl.segment_offsets(w)
    h = ac.AdaCons(w.N, w.d, w.dtype, seg_offsets=off)
    if per_segment:
        h.set_option(ac.OPT_PER_SEGMENT, 1)
    S = h.info(ac.INFO_COEFF_SETS)
    bounds = off if per_segment else [0, w.d]
    out = torch.empty(w.d, dtype=w.torch_dtype, device=dev)
    m = np.zeros((S, w.N))
    worst = dict(p=0.0, q=0.0, a=0.0, gamma=0.0, m=0.0, out=0.0)
    gen = torch.Generator().manual_seed(0)
    G = None
    for t in range(steps):
        G = wl.generate(w, t, dev, out=G)
        h.aggregate(G, out)
        torch.cuda.synchronize()
        a_gpu = h.coeffs(ac.COEFF_A)
        ranks = tp.ranks_of(a_gpu)
        gam = np.zeros((S, w.N))
        for s_ in range(S):
            lo, hi = bounds[s_], bounds[s_ + 1]
            p, q = tp.streamed_statistics(G[:, lo:hi]) if hi - lo > 4_000_000 else oc.consensus_statistics(tp.to_f64(G[:, lo:hi]))
            c = oc.coefficients(p, q, m[s_], 0.99)
            if not np.array_equal(tp.ranks_of(c["a"][None, :])[0], ranks[s_]):
                c = oc.coefficients(p, q, m[s_], 0.99, assign=ranks[s_])
            m[s_] = c["m"]
            gam[s_] = c["gamma"]
            for k, code in (("p", ac.COEFF_P), ("q", ac.COEFF_Q), ("a", ac.COEFF_A), ("gamma", ac.COEFF_GAMMA)):
                worst[k] = max(worst[k], rel(h.coeffs(code)[s_], c[k]))
            worst["m"] = max(worst["m"], rel(h.state()[0][s_], c["m"]))
        cols = torch.randint(0, w.d, (200_000,), generator=gen) if w.N * w.d > 5e8 else torch.arange(w.d)
        seg = np.searchsorted(np.asarray(bounds), cols.numpy(), side="right") - 1
        Gs = tp.to_f64(G[:, cols.to(dev)])
        psi = np.sum(gam[seg].T * Gs, axis=0)
        got = tp.to_f64(out[cols.to(dev)])
        gmax = float(G.abs().max())
        worst["out"] = max(worst["out"], float(np.abs(got - psi).max()) / gmax)
    mode = "per segment" if per_segment else "model-wise"
    print(f"| {name} ({w.dtype}, N={w.N}, d={w.d}, {mode}) | {steps} | " +
          " | ".join(f"{worst[k]:.1e}" for k in ("p", "q", "a", "gamma", "m", "out")) + " |", flush=True)
    h.close()


if __name__ == "__main__":
    print("| configuration | steps | p | q | a | gamma | m | output / max\\|g\\| |")
    print("|---|---|---|---|---|---|---|---|")
    report("small4", 1)
    report("resnet8", 5)
    report("mixed16", 3)
    report("bert64", 2)
    report("ragged32", 2)
    report("ragged32", 2, per_segment=True)
