"""The exchange step of the column-sharded form: every rank's statistics record lands in rank order
in every rank's gathered buffer, and finish is told the number of shards.  Two gloo ranks on the
CPU, with a stand-in for the context (the kernels need a GPU; the plumbing does not)."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2411_03742_b200.sharded import ColumnSharded, clip_segments, column_ranges  # noqa: E402


class FakeContext:
    """Records what the plumbing hands to the two halves of a step."""
    stats_doubles = 7

    def __init__(self, rank):
        self.rank, self.calls = rank, []

    def pass1(self, grads, stats, stream=None):
        assert stats.numel() == self.stats_doubles
        stats.copy_(torch.arange(self.stats_doubles, dtype=torch.float64) + 100.0 * (self.rank + 1) + float(grads))
        self.calls.append("pass1")

    def finish(self, grads, out, stats_all, shards, stream=None):
        self.calls.append(("finish", stats_all.clone(), shards))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group(backend="gloo", rank=rank, world_size=world)
    ctx = FakeContext(rank)
    sh = ColumnSharded(ctx, rank, world, device="cpu")
    for step in range(2):                       # a second step must not see the first one's records
        sh.aggregate(torch.tensor(float(step)), None)
    q.put((rank, [(c[1].tolist(), c[2]) for c in ctx.calls if c != "pass1"], [c for c in ctx.calls if c == "pass1"]))
    dist.barrier()
    dist.destroy_process_group()


def test_records_arrive_in_rank_order_on_every_rank():
    mpc = mp.get_context("spawn")
    q = mpc.Queue()
    port = _free_port()
    procs = [mpc.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, finishes, pass1s in got:
        assert len(pass1s) == 2 and len(finishes) == 2
        for step, (stats_all, shards) in enumerate(finishes):
            assert shards == 2
            want = [e + 100.0 * (r + 1) + step for r in range(2) for e in range(7)]
            assert stats_all == want, (rank, step)


def test_one_shard_needs_no_process_group():
    ctx = FakeContext(0)
    sh = ColumnSharded(ctx, 0, 1, device="cpu")
    sh.aggregate(torch.tensor(0.0), None)
    assert ctx.calls[0] == "pass1" and ctx.calls[1][2] == 1
    assert ctx.calls[1][1].tolist() == [100.0 + e for e in range(7)]
    with pytest.raises(ValueError):
        ColumnSharded(ctx, 1, 1, device="cpu")


@pytest.mark.parametrize("d,shards,multiple", [(1000, 3, 16), (340_000_000, 8, 16), (17, 4, 16), (0, 2, 8), (4096, 4, 8),
                                               (100_003, 7, 1)])
def test_column_ranges_tile_the_vector(d, shards, multiple):
    r = column_ranges(d, shards, multiple)
    assert len(r) == shards and r[0][0] == 0 and r[-1][1] == d
    for (lo, hi), (lo2, _) in zip(r, r[1:]):
        assert hi == lo2 and lo <= hi
    for lo, hi in r[:-1]:
        assert lo % multiple == 0 and hi % multiple == 0
    sizes = [hi - lo for lo, hi in r]
    assert max(sizes[:-1], default=0) - min(sizes[:-1], default=0) <= multiple
    assert sizes[-1] - min(sizes) < 2 * multiple + (d % multiple)


def test_clip_segments_keeps_every_column_once():
    off = [0, 5, 5, 40, 100, 100, 257]
    ranges = column_ranges(257, 3, 16)
    total = [0] * (len(off) - 1)
    for lo, hi in ranges:
        c = clip_segments(off, lo, hi)
        assert c[0] == 0 and c[-1] == hi - lo and all(a <= b for a, b in zip(c, c[1:]))
        for s in range(len(total)):
            total[s] += c[s + 1] - c[s]
    assert total == [b - a for a, b in zip(off, off[1:])]
