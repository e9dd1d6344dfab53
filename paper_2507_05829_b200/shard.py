"""Band sharding over several devices: which rows each rank produces and the one exchange per plan.

Sec. IV-C (operation replication): bands that carry their halo are independent units, so rank ``r`` of ``W`` runs the
contiguous block of bands ``lop_plan_shard`` gives it on its own copy of the parameters, and the ranks then exchange
the output rows they produced -- one all-gather per plan, after which every rank holds the whole output tensor (the
next plan's input).  This module holds only that plumbing: the row bookkeeping and a ``torch.distributed`` all-gather
of unequal row blocks.  It works on whatever device the tensors live on (NCCL for CUDA tensors, gloo for CPU tensors).
"""
import torch
import torch.distributed as dist


def shard_table(plan, world):
    """[(band_lo, band_hi, row_lo, row_hi, in_lo, in_hi)] for every rank; the row blocks tile the output rows."""
    table = [plan.shard(r, world) for r in range(world)]
    rows = [(t[2], t[3]) for t in table if t[3] > t[2]]
    for (a0, a1), (b0, b1) in zip(rows, rows[1:]):
        if a1 != b0:
            raise ValueError("the ranks' row blocks do not tile the output: %r" % (rows,))
    return table


def all_gather_rows(out, table, rank, group=None):
    """Every rank has written rows [row_lo, row_hi) of ``out`` ([N, H, W, C]); afterwards every rank has all rows.

    The blocks differ in size, so each rank sends its block padded to the largest one and the receivers keep the
    valid part.  Bits are moved, never added up."""
    world = len(table)
    if world == 1:
        return out
    n_max = max(t[3] - t[2] for t in table)
    if n_max == 0:
        return out
    N, H, W, C = out.shape
    lo, hi = table[rank][2], table[rank][3]
    mine = torch.zeros((N, n_max, W, C), dtype=out.dtype, device=out.device)
    if hi > lo:
        mine[:, :hi - lo].copy_(out[:, lo:hi])
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine, group=group)
    for r, part in enumerate(parts):
        r_lo, r_hi = table[r][2], table[r][3]
        if r != rank and r_hi > r_lo:
            out[:, r_lo:r_hi].copy_(part[:, :r_hi - r_lo])
    return out


class ShardedChain:
    """A :class:`~.chain.DeviceChain` whose every plan runs only this rank's block of bands, with one all-gather of
    output rows behind each plan."""

    def __init__(self, device_chain, rank, world, group=None):
        self.dc = device_chain
        self.rank, self.world, self.group = rank, world, group
        self.tables = [shard_table(p, world) for p in device_chain.plans]

    def run(self, x_dev, stream=None):
        """Every plan's block of bands on ``stream`` (default: torch's current stream), each followed by the all-gather of
        its output rows.  torch orders a collective, and the copies around it, against its CURRENT stream, so the whole
        loop runs with ``stream`` made current: the gather then waits for this rank's launch, and the next plan's launch
        for the gathered rows."""
        dc = self.dc
        cur = torch.cuda.current_stream(dc.device) if stream is None else stream
        with torch.cuda.stream(cur):
            s = cur.cuda_stream
            for plan, ws, out, table in zip(dc.plans, dc.ws, dc.outs, self.tables):
                b_lo, b_hi = table[self.rank][0], table[self.rank][1]
                plan.run_shard(b_lo, b_hi, x_dev.data_ptr(), out.data_ptr(), ws.data_ptr(), s)
                all_gather_rows(out, table, self.rank, self.group)
                x_dev = out
        return dc.outs[-1]
