"""Stochastic linear regression with N simulated workers, aggregated through the library.

The objective is the one of the paper's first experiment (Section 4.1, Eq. 14):
    min_w  E_{zeta ~ U[0,1]^d} [ (w^T zeta)^2 / 2 ],   d = 1000,
each worker drawing its own mini-batch per step; the workers' gradients are stacked as an N x d
matrix on the GPU and aggregated either by the plain mean or by AdaCons (`adacons_aggregate`).
Both runs use the same step size and the same random batches.  The paper tunes the step size
analytically per method but prints neither the rule nor numbers (its curves are figures), so this
driver only supports a qualitative comparison (final loss of the two aggregation rules).

    python -m paper_2411_03742_b200.examples.linear_regression --workers 32 --batch 16 --steps 200
"""
from __future__ import annotations

import argparse

import torch

from .. import binding


def expected_loss(w: torch.Tensor) -> float:
    """E (w^T zeta)^2 / 2 for zeta ~ U[0,1]^d:  E[zeta zeta^T] = I/12 + 11^T/4."""
    w = w.double()
    return float(0.5 * ((w * w).sum() / 12.0 + w.sum() ** 2 / 4.0))


def worker_gradients(w: torch.Tensor, N: int, batch: int, gen: torch.Generator) -> torch.Tensor:
    """g_i = mean over the worker's batch of (w^T zeta) zeta  ->  N x d."""
    d = w.numel()
    zeta = torch.rand((N, batch, d), generator=gen, device=w.device)
    r = zeta @ w                                  # N x batch
    return (r.unsqueeze(-1) * zeta).mean(dim=1).contiguous()


def run(N: int = 32, batch: int = 16, steps: int = 200, d: int = 1000, lr: float = 0.0, seed: int = 0,
        device: str = "cuda:0"):
    """Returns (losses_mean, losses_adacons), one value per step."""
    dev = torch.device(device)
    if lr <= 0.0:
        lr = 1.0 / (d / 4.0 + 1.0 / 12.0)          # 1 / largest eigenvalue of E[zeta zeta^T]
    w0 = torch.randn(d, generator=torch.Generator().manual_seed(seed)).to(dev)
    results = []
    for rule in ("mean", "adacons"):
        gen = torch.Generator(device=dev).manual_seed(seed + 1)
        w = w0.clone()
        agg = binding.AdaCons(N, d, "f32") if rule == "adacons" else None
        psi = torch.empty(d, device=dev)
        losses = []
        for _ in range(steps):
            G = worker_gradients(w, N, batch, gen)
            if agg is None:
                psi = G.mean(dim=0)
            else:
                agg.aggregate(G, psi)
            w = w - lr * psi
            losses.append(expected_loss(w))
        if agg is not None:
            agg.close()
        results.append(losses)
    return results[0], results[1]


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workers", type=int, default=32)
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--lr", type=float, default=0.0)
    a = ap.parse_args(argv)
    lm, la = run(a.workers, a.batch, a.steps, lr=a.lr)
    print(f"N={a.workers} batch={a.batch} steps={a.steps}: final loss  mean {lm[-1]:.6e}   adacons {la[-1]:.6e}")


if __name__ == "__main__":
    main()
