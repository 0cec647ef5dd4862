"""The allocation-free entry point (adacons_stats_noalloc) against the ordinary one.

Some callers cannot allocate device memory at the moment they need the aggregation's statistics
-- typically a gradient hook running inside a training framework whose caching allocator has
already taken the device's memory, where a raw cudaMalloc can fail and stalls the device.  For
them the library keeps pass 1's scratch in a fixed array of its own device image.  This test
calls that entry point through the C ABI twice in a row (different shapes, so that anything left
in the shared scratch by the first call would show) and checks p_i and q_i both against what
adacons_aggregate + adacons_get_coeffs report for the same input and against the float64 oracle's
consensus_statistics, within the coefficient tolerance of the parity tests; it also checks that
the device's free memory is the same before and after the calls.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from oracle import adacons_oracle as oc
from paper_2411_03742_b200 import workloads as wl
from parity_util import assert_coeffs, streamed_statistics, to_f64

pytestmark = pytest.mark.gpu
COEFF_RTOL = 1e-5


def _reference(ac, G):
    N, d = G.shape
    h = ac.AdaCons(N, d, "f32" if G.dtype == torch.float32 else "bf16")
    out = torch.empty(d, dtype=G.dtype, device=G.device)
    h.aggregate(G, out)
    torch.cuda.synchronize()
    p, q = h.coeffs(ac.COEFF_P)[0].copy(), h.coeffs(ac.COEFF_Q)[0].copy()
    h.close()
    return p, q


def test_noalloc_matches_the_allocating_entry_point_twice_in_a_row():
    from paper_2411_03742_b200 import binding as ac
    dev = torch.device("cuda:0")
    cases = [wl.Workload("na64", 64, 300_008, "bf16", 1, "student_flip", seed=5),
             wl.Workload("na7", 7, 123_456, "f32", 1, "gauss_outlier", seed=6),
             wl.Workload("na5odd", 5, 10_001, "bf16", 1, "gauss", seed=7)]       # generic (unaligned) path
    pq = torch.full((128,), float("nan"), dtype=torch.float64, device=dev)
    ac.stats_noalloc(wl.generate(cases[2], 0, dev), pq)      # the first call on a device looks the scratch up
    for w in cases:
        G = wl.generate(w, 0, dev)
        torch.cuda.synchronize()
        pq.fill_(float("nan"))
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        ac.stats_noalloc(G, pq)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before, "the allocation-free entry point changed the device's free memory"
        got = pq.cpu().numpy()
        p, q = _reference(ac, G)
        np.testing.assert_allclose(got[:w.N], p, rtol=COEFF_RTOL, atol=COEFF_RTOL * 1e-3 * np.abs(p).max())
        np.testing.assert_allclose(got[w.N:2 * w.N], q, rtol=COEFF_RTOL)
        p_or, q_or = oc.consensus_statistics(to_f64(G))                        # the float64 oracle
        assert_coeffs(got[:w.N], p_or, f"{w.name} p against the oracle")
        assert_coeffs(got[w.N:2 * w.N], q_or, f"{w.name} q against the oracle")
        assert np.all(np.isnan(got[2 * w.N:]))                                  # nothing written past 2N
        del G
    # same input again right after the others: the shared scratch holds stale partials by now
    w = cases[0]
    G = wl.generate(w, 0, dev)
    ac.stats_noalloc(G, pq)
    ac.stats_noalloc(G, pq)
    torch.cuda.synchronize()
    p, q = _reference(ac, G)
    got = pq.cpu().numpy()
    np.testing.assert_allclose(got[:w.N], p, rtol=COEFF_RTOL, atol=COEFF_RTOL * 1e-3 * np.abs(p).max())
    np.testing.assert_allclose(got[w.N:2 * w.N], q, rtol=COEFF_RTOL)
    p_or, q_or = oc.consensus_statistics(to_f64(G))
    assert_coeffs(got[:w.N], p_or, "second call in a row, p against the oracle")
    assert_coeffs(got[w.N:2 * w.N], q_or, "second call in a row, q against the oracle")


def test_noalloc_vector_longer_than_one_tma_chunk():
    """Beyond 2^30 columns pass 1 runs once per column chunk; the scratch then holds the partial
    sums of every chunk.  Same comparison as above, N = 2, d = 2^30 + 32,768 (4.3 GB)."""
    from paper_2411_03742_b200 import binding as ac
    dev = torch.device("cuda:0")
    free, _ = torch.cuda.mem_get_info()
    if free < 12e9:
        pytest.skip("needs 12 GB of free device memory")
    w = wl.Workload("nalong", 2, (1 << 30) + 32_768, "bf16", 1, "gauss", seed=12)
    G = wl.generate(w, 0, dev, row_block=64_000_000)
    pq = torch.zeros(4, dtype=torch.float64, device=dev)
    for _ in range(2):
        ac.stats_noalloc(G, pq)
    torch.cuda.synchronize()
    p, q = _reference(ac, G)
    got = pq.cpu().numpy()
    np.testing.assert_allclose(got[:2], p, rtol=COEFF_RTOL)
    np.testing.assert_allclose(got[2:], q, rtol=COEFF_RTOL)
    p_or, q_or = streamed_statistics(G, slab=64_000_000, threads=4)           # the float64 oracle, all columns
    assert_coeffs(got[:2], p_or, "long vector p against the oracle")
    assert_coeffs(got[2:], q_or, "long vector q against the oracle")


def test_noalloc_rejects_sizes_beyond_its_scratch():
    from paper_2411_03742_b200 import binding as ac
    G = torch.zeros(ac.NOALLOC_MAX_N + 1, 256, device="cuda:0")
    pq = torch.zeros(2 * (ac.NOALLOC_MAX_N + 1), dtype=torch.float64, device="cuda:0")
    with pytest.raises(ac.AdaConsError) as e:
        ac.stats_noalloc(G, pq)
    assert e.value.code == ac.ELIMIT and "scratch" in str(e.value)
