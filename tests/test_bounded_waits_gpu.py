"""Hang protection: a wait inside a kernel that can never be satisfied gives up after its limit,
reports ADACONS_FLAG_TIMEOUT and leaves the context (and the GPU) usable.  Nothing here faults,
traps or spins without bound: the self-test kernels wait on a barrier nobody arrives on, with the
same 2 s limit as the production kernels."""
import time

import numpy as np
import pytest
import torch

from oracle import adacons_oracle as oc
from paper_2411_03742_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("which", [0, 1, 2], ids=["mbarrier", "grid-barrier", "published-weights"])
def test_unsatisfiable_wait_times_out_and_context_survives(which):
    from paper_2411_03742_b200 import binding as ac
    w = wl.Workload("bw", 6, 40_000, "f32", 1, "gauss", seed=8)
    dev = "cuda:0"
    h = ac.AdaCons(w.N, w.d, "f32")
    G = wl.generate(w, 0, dev)
    out = torch.empty(w.d, device=dev)
    h.aggregate(G, out)
    torch.cuda.synchronize()
    assert h.status() == 0
    t0 = time.perf_counter()
    h.selftest_bounded_wait(which)
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert 1.5 < waited < 10.0, waited                      # gave up at the limit, not before, not never
    assert h.status() & ac.FLAG_TIMEOUT
    h.reset()
    assert h.status() == 0
    for fused, one_launch, path in ((1, 0, 3), (0, 2, 5), (0, 0, 1)):   # every path still works, incl. its waits
        h.set_option(ac.OPT_FUSED_SMALL, fused)
        h.set_option(ac.OPT_ONE_LAUNCH, one_launch)
        h.reset()
        h.aggregate(G, out)
        torch.cuda.synchronize()
        assert h.info(ac.INFO_LAST_PATH) == path
        res = oc.AdaConsOracle(w.N, w.d).step(G.cpu().double().numpy())
        np.testing.assert_allclose(h.coeffs()[0], res["gamma"][0], rtol=1e-5)
        assert h.status() == 0
