"""The N > 1 path of bench.py is "independent replicas": no data-path collective, only the
whole-job reduction (max over ranks of the time, sum of the units).  Two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    r, w, l = bench.dist_setup(world, use_cuda=False)
    assert (r, w, l) == (rank, world, rank)
    bench.barrier()
    ms, units = bench.reduce_over_ranks(10.0 + 5.0 * rank, 1000.0 * (rank + 1))
    q.put((rank, ms, units))
    bench.barrier()
    dist.destroy_process_group()


def test_two_replicas_reduce_to_max_time_and_total_units():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, units in got:
        assert ms == 15.0 and units == 3000.0


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(3.5, 7.0) == (3.5, 7.0)
    w = bench.parse_args([])
    assert (w.gpus, w.steps, w.warmup, w.workload) == (1, 10, 3, "bert64")
