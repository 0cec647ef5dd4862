"""Seeded input generators: shapes, reproducibility and the statistics the recipes promise."""
import math

import torch

from paper_2411_03742_b200 import workloads as wl


def test_registry_matches_the_benchmark_configurations():
    w = wl.WORKLOADS
    assert (w["small4"].N, w["small4"].d, w["small4"].dtype) == (4, 100_000, "f32")
    assert (w["resnet8"].N, w["resnet8"].d, w["resnet8"].steps) == (8, 25_600_000, 50)
    assert (w["mixed16"].N, w["mixed16"].d, w["mixed16"].dtype) == (16, 110_000_000, "bf16")
    assert (w["bert64"].N, w["bert64"].d, w["bert64"].dtype) == (64, 340_000_000, "bf16")
    assert (w["ragged32"].N, w["ragged32"].d, w["ragged32"].num_segments) == (32, 340_000_000, 390)


def test_generation_is_reproducible_and_step_dependent():
    w = wl.WORKLOADS["small4"].scaled(5000)
    a, b, c = wl.generate(w, 0), wl.generate(w, 0), wl.generate(w, 1)
    assert torch.equal(a, b) and not torch.equal(a, c)
    assert a.shape == (4, 5000) and a.dtype == torch.float32


def test_recipes_have_the_stated_structure():
    w = wl.WORKLOADS["resnet8"].scaled(200_000)
    G = wl.generate(w, 0).double()
    norms = G.norm(dim=1)
    assert 15 < float(norms[0] / norms[1:].mean()) < 25          # the x20 outlier
    w = wl.WORKLOADS["bert64"].scaled(50_000)
    G = wl.generate(w, 0).double()
    mean_rest = G[2:].mean(0)
    assert float((G[0] * mean_rest).sum()) < 0 and float((G[1] * mean_rest).sum()) < 0
    assert float((G[2] * mean_rest).sum()) > 0
    assert G.dtype == torch.float64 and wl.generate(w, 0).dtype == torch.bfloat16
    assert float(G.abs().max()) > 20                              # heavy tails
    w = wl.WORKLOADS["mixed16"].scaled(100_000)
    G = wl.generate(w, 3).double()
    sd = G.std(dim=1)
    assert float(sd.max() / sd.min()) > 5
    assert 5e-5 < float(sd.min()) and float(sd.max()) < 2e-2


def test_segment_offsets_are_ragged_and_cover_d():
    w = wl.WORKLOADS["ragged32"]
    off = wl.segment_offsets(w)
    assert len(off) == 391 and off[0] == 0 and off[-1] == w.d
    sizes = [b - a for a, b in zip(off, off[1:])]
    assert min(sizes) > 0
    assert sum(1 for o in off[1:-1] if o % 4) > 100               # boundaries not vector-aligned
    assert max(sizes) / min(sizes) > 100
    assert wl.segment_offsets(wl.WORKLOADS["small4"]) is None
    small = w.scaled(1_000_000)
    off = wl.segment_offsets(small)
    assert off[-1] == 1_000_000 and all(b >= a for a, b in zip(off, off[1:]))
