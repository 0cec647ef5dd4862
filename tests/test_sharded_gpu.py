"""The step in two halves (adacons_pass1 / adacons_finish) for a matrix whose columns are spread over
several devices, against the float64 oracle of the WHOLE matrix.  The shards are emulated on one
GPU: one context per shard, the shards' kernels run one after the other (none waits for another),
and the records that an all-gather would deliver are written side by side in one buffer."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import adacons_oracle as oc
from paper_2411_03742_b200 import workloads as wl
from paper_2411_03742_b200.sharded import ColumnSharded, clip_segments, column_ranges
from parity_util import assert_coeffs_by_set, assert_output, oracle_step, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ac():
    from paper_2411_03742_b200 import binding
    binding.load_library()
    return binding


def sharded_step(ctxs, shards_G, outs, stats_all):
    """What R ranks do in a step: pass 1 each into its slot, (all-gather), finish each."""
    n = ctxs[0].stats_doubles
    for r, (h, G) in enumerate(zip(ctxs, shards_G)):
        h.pass1(G, stats_all[r * n:(r + 1) * n])
    for h, G, o in zip(ctxs, shards_G, outs):
        h.finish(G, o, stats_all, len(ctxs))
    torch.cuda.synchronize()


def run_sharded(ac, w, ranges, steps, *, offsets=None, beta=0.9, expect_paths=None, what=None):
    dev = torch.device("cuda:0")
    what = what or f"sharded {w.name} x{len(ranges)}"
    per_segment = offsets is not None
    ctxs = []
    for lo, hi in ranges:
        h = ac.AdaCons(w.N, hi - lo, w.dtype, seg_offsets=clip_segments(offsets, lo, hi) if per_segment else None)
        if per_segment:
            h.set_option(ac.OPT_PER_SEGMENT, 1)
        h.set_option(ac.OPT_BETA, beta)
        ctxs.append(h)
    kw = dict(seg_offsets=offsets, per_segment=True) if per_segment else {}
    orc = oc.AdaConsOracle(w.N, w.d, beta=beta, **kw)
    n = ctxs[0].stats_doubles
    assert all(h.stats_doubles == n for h in ctxs)
    stats_all = torch.full((len(ranges) * n,), float("nan"), dtype=torch.float64, device=dev)
    outs = [torch.empty(hi - lo, dtype=w.torch_dtype, device=dev) for lo, hi in ranges]
    flags = 0
    for t in range(steps):
        G = wl.generate(w, t, dev)
        shards_G = [G[:, lo:hi].contiguous() for lo, hi in ranges]
        sharded_step(ctxs, shards_G, outs, stats_all)
        G64 = to_f64(G)
        res = oracle_step(orc, G64, w.dtype, ctxs[0].coeffs(ac.COEFF_A), what=what)
        # every shard holds the same coefficients and state, bit for bit
        for kind in (ac.COEFF_P, ac.COEFF_Q, ac.COEFF_A, ac.COEFF_A_TILDE, ac.COEFF_GAMMA):
            ref = ctxs[0].coeffs(kind)
            for h in ctxs[1:]:
                assert np.array_equal(h.coeffs(kind), ref, equal_nan=True), f"{what}: shards disagree on coefficient kind {kind}"
        m0, step0 = ctxs[0].state()
        for h in ctxs[1:]:
            m, step = h.state()
            assert step == step0 == t + 1 and np.array_equal(m, m0)
        h = ctxs[0]
        assert_coeffs_by_set(h.coeffs(ac.COEFF_P), res["p"], f"{what} step {t} p")
        assert_coeffs_by_set(h.coeffs(ac.COEFF_Q), res["q"], f"{what} step {t} q")
        assert_coeffs_by_set(h.coeffs(ac.COEFF_A), res["a"], f"{what} step {t} a")
        assert_coeffs_by_set(h.coeffs(ac.COEFF_A_TILDE), res["a_tilde"], f"{what} step {t} a~")
        assert_coeffs_by_set(h.coeffs(ac.COEFF_GAMMA), res["gamma"], f"{what} step {t} gamma")
        assert_coeffs_by_set(m0, res["m"], f"{what} step {t} m")
        assert_output(torch.cat(outs), res, G64, w.dtype, f"{what} step {t}", offsets)
        flags |= int(np.bitwise_or.reduce(res["flags"]))
        for h in ctxs:
            assert h.status() == flags
        if expect_paths is not None:
            assert [h.info(ac.INFO_LAST_PATH) for h in ctxs] == expect_paths
    for h in ctxs:
        h.close()


@pytest.mark.parametrize("N,d,dtype", [(8, 400_000, "f32"), (16, 300_008, "bf16"), (5, 70_001, "f32")])
def test_one_shard_gives_the_bits_of_the_three_kernel_path(ac, N, d, dtype):
    dev = torch.device("cuda:0")
    w = wl.Workload("one-shard", N, d, dtype, 3, "gauss", seed=11)
    a, b = ac.AdaCons(N, d, dtype), ac.AdaCons(N, d, dtype)
    for h in (a, b):
        h.set_option(ac.OPT_FUSED_SMALL, 0)
        h.set_option(ac.OPT_ONE_LAUNCH, 0)
    stats = torch.empty(b.stats_doubles, dtype=torch.float64, device=dev)
    oa, ob = (torch.empty(d, dtype=w.torch_dtype, device=dev) for _ in range(2))
    for t in range(3):
        G = wl.generate(w, t, dev)
        a.aggregate(G, oa)
        b.pass1(G, stats)
        assert b.state()[1] == t                     # the first half changes no state
        b.finish(G, ob, stats, 1)
        torch.cuda.synchronize()
        assert torch.equal(oa.view(torch.uint8), ob.view(torch.uint8))
        for kind in range(5):
            assert np.array_equal(a.coeffs(kind), b.coeffs(kind))
        assert np.array_equal(a.state()[0], b.state()[0]) and a.state()[1] == b.state()[1] == t + 1
        assert float(stats[-1]) == d                 # the record's last entry: the set's columns on this shard
    a.close(); b.close()


@pytest.mark.parametrize("shards", [2, 3, 5])
@pytest.mark.parametrize("N,d,dtype,recipe", [(8, 1_000_000, "f32", "gauss_outlier"), (16, 700_040, "bf16", "loguniform"),
                                              (64, 200_000, "bf16", "student_flip")])
def test_aligned_shards_against_the_oracle(ac, shards, N, d, dtype, recipe):
    w = wl.Workload(f"{recipe}{N}", N, d, dtype, 4, recipe, seed=3 * N + shards)
    run_sharded(ac, w, column_ranges(d, shards, 16), 4, expect_paths=[1] * shards)


def test_ragged_shards(ac):
    """Shards of any width: rows that are not a multiple of 16 bytes long arrive through one tensor map per class of equally offset rows, a
    one-column shard runs on the scalar kernels."""
    w = wl.Workload("ragged-shards", 16, 300_001, "f32", 3, "gauss", seed=21)
    run_sharded(ac, w, [(0, 100_003), (100_003, 100_004), (100_004, 250_000), (250_000, 300_001)], 3,
                expect_paths=[10, 2, 1, 10])


@pytest.mark.parametrize("N,paths", [(100, [7, 7]), (200, [7, 7]), (300, [4, 4])])
def test_more_than_64_workers_sharded(ac, N, paths):
    w = wl.Workload(f"sharded{N}", N, 120_000, "bf16", 2, "student_flip", seed=N)
    run_sharded(ac, w, column_ranges(120_000, 2, 16), 2, expect_paths=paths)


def test_per_segment_sharded(ac):
    """Every shard gets all segments clipped to its columns: some are empty on one shard, some straddle
    a boundary, one is empty everywhere (no flag)."""
    N, d = 8, 600_000
    rng = np.random.default_rng(5)
    cuts = np.sort(rng.integers(0, d // 8, size=22)) * 8
    offsets = [0] + [int(c) for c in cuts] + [int(cuts[-1])] + [d]            # a repeated offset: an empty segment
    w = wl.Workload("seg-sharded", N, d, "f32", 3, "gauss", seed=8)
    run_sharded(ac, w, column_ranges(d, 3, 16), 3, offsets=offsets)


def test_plumbing_class_with_one_shard(ac):
    dev = torch.device("cuda:0")
    w = wl.Workload("plumbing", 8, 100_000, "f32", 2, "gauss", seed=2)
    a, b = ac.AdaCons(8, 100_000, "f32"), ac.AdaCons(8, 100_000, "f32")
    a.set_option(ac.OPT_FUSED_SMALL, 0); a.set_option(ac.OPT_ONE_LAUNCH, 0)
    sh = ColumnSharded(b, 0, 1, device=dev)
    oa, ob = (torch.empty(100_000, dtype=torch.float32, device=dev) for _ in range(2))
    for t in range(2):
        G = wl.generate(w, t, dev)
        a.aggregate(G, oa)
        sh.aggregate(G, ob)
        torch.cuda.synchronize()
        assert torch.equal(oa, ob)
    a.close(); b.close()


def test_bad_arguments_are_refused(ac):
    dev = torch.device("cuda:0")
    h = ac.AdaCons(4, 1000, "f32")
    G = torch.randn(4, 1000, device=dev)
    out = torch.empty(1000, device=dev)
    stats = torch.empty(h.stats_doubles, dtype=torch.float64, device=dev)
    lib = ac.load_library()
    st = torch.cuda.current_stream().cuda_stream
    assert lib.adacons_pass1(h._ctx, G.data_ptr(), None, st) == ac.EINVAL
    assert lib.adacons_pass1(h._ctx, G.data_ptr(), stats.data_ptr() + 4, st) == ac.EINVAL
    assert lib.adacons_finish(h._ctx, G.data_ptr(), out.data_ptr(), None, 1, st) == ac.EINVAL
    assert lib.adacons_finish(h._ctx, G.data_ptr(), out.data_ptr(), stats.data_ptr(), 0, st) == ac.EINVAL
    assert lib.adacons_finish(h._ctx, G.data_ptr(), None, stats.data_ptr(), 1, st) == ac.EINVAL
    with pytest.raises(ValueError):
        h.pass1(G, stats[:-1])
    with pytest.raises(ValueError):
        h.pass1(G, stats.float())
    with pytest.raises(ValueError):
        h.finish(G, out, stats, 2)
    with pytest.raises(ValueError):
        h.finish(G, out, stats, 0)
    assert h.state()[1] == 0
    h.close()


def test_two_halves_replayed_from_a_cuda_graph(ac):
    """Both halves only enqueue kernels: a whole two-range step can be captured once and replayed."""
    from parity_util import assert_coeffs
    dev = torch.device("cuda:0")
    w = wl.Workload("sharded-graph", 16, 600_000, "bf16", 3, "gauss", seed=31)
    ranges = column_ranges(w.d, 2, 16)
    ctxs = [ac.AdaCons(w.N, hi - lo, "bf16") for lo, hi in ranges]
    n = ctxs[0].stats_doubles
    stats_all = torch.zeros(2 * n, dtype=torch.float64, device=dev)
    static = [torch.empty(w.N, hi - lo, dtype=torch.bfloat16, device=dev) for lo, hi in ranges]
    outs = [torch.empty(hi - lo, dtype=torch.bfloat16, device=dev) for lo, hi in ranges]

    def step():
        for r in range(2):
            ctxs[r].pass1(static[r], stats_all[r * n:(r + 1) * n])
        for r in range(2):
            ctxs[r].finish(static[r], outs[r], stats_all, 2)

    G = wl.generate(w, 0, dev)
    for r, (lo, hi) in enumerate(ranges):
        static[r].copy_(G[:, lo:hi])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                                         # warm-up outside the capture (encodes the tensor maps)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    for h in ctxs:
        h.reset()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    orc = oc.AdaConsOracle(w.N, w.d)
    for t in range(3):
        G = wl.generate(w, t, dev)
        for r, (lo, hi) in enumerate(ranges):
            static[r].copy_(G[:, lo:hi])
        graph.replay()
        torch.cuda.synchronize()
        G64 = to_f64(G)
        res = oracle_step(orc, G64, "bf16", ctxs[0].coeffs(ac.COEFF_A), what="sharded graph replay")
        for h in ctxs:
            assert_coeffs(h.coeffs(), res["gamma"], f"gamma replay {t}")
            assert_coeffs(h.state()[0], res["m"], f"m replay {t}")
        assert_output(torch.cat(outs), res, G64, "bf16", f"sharded replay {t}")
    assert all(h.state()[1] == 3 and h.status() == 0 for h in ctxs)
    for h in ctxs:
        h.close()


def test_finish_with_non_finite_statistics_falls_back_to_the_mean(ac):
    """A record that carries NaN (a shard that overflowed) is a non-finite statistic like any other:
    plain mean on every shard, state left as it was, NONFINITE raised; the next clean step recovers."""
    dev = torch.device("cuda:0")
    N, d = 6, 50_000
    w = wl.Workload("nan-record", N, d, "f32", 2, "gauss", seed=4)
    h = ac.AdaCons(N, d, "f32")
    h.set_option(ac.OPT_BETA, 0.5)
    n = h.stats_doubles
    stats = torch.empty(2 * n, dtype=torch.float64, device=dev)
    out = torch.empty(d, device=dev)
    G = wl.generate(w, 0, dev)
    h.pass1(G, stats[:n])
    stats[n:] = 0.0
    h.finish(G, out, stats, 2)                               # a clean first step (the second record adds nothing)
    torch.cuda.synchronize()
    m_before, step_before = h.state()
    assert step_before == 1 and h.status() == 0
    G = wl.generate(w, 1, dev)
    h.pass1(G, stats[:n])
    stats[n + 2] = float("nan")
    h.finish(G, out, stats, 2)
    torch.cuda.synchronize()
    assert h.status() == ac.FLAG_NONFINITE
    np.testing.assert_array_equal(h.coeffs(ac.COEFF_GAMMA)[0], np.full(N, 1.0 / N))
    m_after, step_after = h.state()
    np.testing.assert_array_equal(m_after, m_before)
    assert step_after == 2
    mean = to_f64(G).mean(axis=0)
    assert np.max(np.abs(to_f64(out) - mean)) <= 1e-5 * float(G.abs().max())
    h.close()
