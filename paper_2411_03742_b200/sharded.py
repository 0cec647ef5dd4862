"""Column-sharded aggregation over several devices: plumbing around adacons_pass1 / adacons_finish.

Device r of R holds columns [c_r, c_{r+1}) of all N gradients.  A step is: pass 1 on the local
columns (kernel), an all-gather of the shards' statistics records (a few KB, torch.distributed),
the coefficient step on all records added in rank order and pass 2 on the local columns (kernels).
Nothing here computes: the sum over shards runs inside the coefficient kernel.
"""
from __future__ import annotations


def column_ranges(d: int, shards: int, multiple: int = 16):
    """Split [0, d) into `shards` consecutive ranges whose interior boundaries are multiples of
    `multiple` columns (so every shard starts 32-byte aligned for 2- and 4-byte elements); sizes
    differ by at most `multiple`, except that the last range takes the ragged end."""
    if shards < 1 or d < 0 or multiple < 1:
        raise ValueError("need shards >= 1, d >= 0, multiple >= 1")
    units = d // multiple
    cuts = [min(d, ((units * r) // shards) * multiple) for r in range(shards)] + [d]
    return [(cuts[r], cuts[r + 1]) for r in range(shards)]


def clip_segments(seg_offsets, lo: int, hi: int):
    """The segment offsets of the whole vector as seen by the shard that holds columns [lo, hi):
    every segment clipped to the range and shifted to start at 0; segments elsewhere become empty."""
    return [min(max(int(o), lo), hi) - lo for o in seg_offsets]


class ColumnSharded:
    """One rank's view of a column-sharded aggregation.

    ctx    the rank's aggregation context (anything with pass1, finish and stats_doubles), created
           for the rank's own number of columns and, in per-segment mode, with clip_segments(...).
    group  a torch.distributed process group (None: the default group); world size 1 needs none.
    """

    def __init__(self, ctx, rank: int, world: int, group=None, device=None):
        import torch
        if not 0 <= rank < world:
            raise ValueError("rank must lie in [0, world)")
        self.ctx, self.rank, self.world, self.group = ctx, int(rank), int(world), group
        n = int(ctx.stats_doubles)
        self._all = torch.zeros(self.world * n, dtype=torch.float64, device=device)
        self._mine = self._all[self.rank * n:(self.rank + 1) * n]     # pass 1 writes straight into its slot

    def aggregate(self, grads, out, stream=None) -> None:
        self.ctx.pass1(grads, self._mine, stream)
        if self.world > 1:
            import torch.distributed as dist
            # in place: rank r's slot of the gathered buffer is its own input
            dist.all_gather_into_tensor(self._all, self._mine, group=self.group)
        self.ctx.finish(grads, out, self._all, self.world, stream)
