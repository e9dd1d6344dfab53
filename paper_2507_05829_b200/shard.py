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


# ---------------------------------------------------------------------------------------------------------------------
# Halo exchange: the other side of the paper's trade between replication and transmission (Sec. IV-C).  Instead of
# recomputing the halo rows of every intermediate tensor, each rank computes every row of every layer exactly ONCE and
# the ranks trade the few rows a neighbour's receptive field reaches into, layer by layer -- the per-layer loop of the
# paper's runtime (Sec. IV-D, Alg. 1 / 2: compute the layer's local operations, then Send / Receive along its edges).
#
# Who computes what: rank r owns the bands [b_lo, b_hi) of lop_plan_shard.  At layer i it computes the rows
# [new_lo of its first band, out_hi of its last band) of a reuse-halo plan -- what its bands need and no lower rank has
# produced -- so the ranks' rows tile every layer.  Its upper halo it computes itself (it is part of those rows); the
# rows below its own that its taps reach were computed by lower ranks and are received from them before the layer runs.
# ---------------------------------------------------------------------------------------------------------------------
def owned_rows(plan, layer, table, rank):
    """Rows [lo, hi) of ``layer``'s output (``-1``: the plan's input) that ``rank`` computes (for the input: holds)."""
    b_lo, b_hi = table[rank][0], table[rank][1]
    lo = hi = None
    for b in range(b_lo, b_hi):
        r = plan.get_range(b, layer)
        if r.out_hi <= r.out_lo:
            continue
        first = r.out_lo if layer == -1 else r.new_lo          # the chain input comes from the host, halo included
        lo = first if lo is None else min(lo, first)
        hi = r.out_hi if hi is None else max(hi, r.out_hi)
    return (0, 0) if lo is None else (lo, hi)


def rows_read(layer_desc, lo, hi, h_in):
    """Input rows the output rows [lo, hi) of a window operator reach (the analytic receptive range, cut to the tensor)."""
    if hi <= lo:
        return (0, 0)
    a = lo * layer_desc.sh - layer_desc.ph
    b = (hi - 1) * layer_desc.sh - layer_desc.ph + (layer_desc.kh - 1) * layer_desc.dh + 1
    a, b = max(a, 0), min(b, h_in)
    return (a, b) if a < b else (0, 0)


class MailboxTransport:
    """send / recv between ranks that live in one process and take turns (tests, one-GPU emulation)."""

    def __init__(self):
        self.box = {}
        self.bytes_sent = 0

    def send(self, src, dst, tag, tensor):
        self.box[(src, dst, tag)] = tensor.clone()
        self.bytes_sent += tensor.numel() * tensor.element_size()

    def recv(self, src, dst, tag, out):
        out.copy_(self.box.pop((src, dst, tag)))

    def flush(self):
        pass


class DistTransport:
    """send / recv over torch.distributed point-to-point calls (NCCL for CUDA tensors, gloo for CPU tensors)."""

    def __init__(self, group=None):
        self.group, self.pending, self.bytes_sent = group, [], 0

    def send(self, src, dst, tag, tensor):
        t = tensor.contiguous()
        self.pending.append((dist.isend(t, dst, group=self.group, tag=tag), t))
        self.bytes_sent += t.numel() * t.element_size()

    def recv(self, src, dst, tag, out):
        buf = torch.empty(out.shape, dtype=out.dtype, device=out.device)
        dist.recv(buf, src, group=self.group, tag=tag)
        out.copy_(buf)

    def flush(self):
        for work, _ in self.pending:
            work.wait()
        self.pending = []


class HaloExchangeRank:
    """One rank of the halo-exchange form of band sharding over one plan.

    ``plan``: a reuse-halo plan (binding.Plan); ``layers``: the plan's layer descriptions (fields of lop_layer);
    ``tensor(idx)``: the rank's full-size tensor of layer ``idx``'s output (``-1``: the plan's input) as a torch tensor
    [N, H, W, C]; ``compute(layer, lo, hi)``: runs rows [lo, hi) of a layer on this rank's tensors (lop_run_layer on a
    GPU; the oracle in CPU tests).  ``step(i)`` is split in two so that ranks sharing a process can take turns."""

    def __init__(self, plan, layers, table, rank, tensor, compute, transport):
        self.plan, self.layers, self.table, self.rank = plan, layers, table, rank
        self.world = len(table)
        self.tensor, self.compute, self.tr = tensor, compute, transport
        self.rows_computed = 0

    def _h_in(self, layer):
        src = self.layers[layer].input_from
        return self.tensor(src).shape[1]

    def _wanted_from(self, layer, reader, owner):
        """[(edge, source tensor, lo, hi)]: rows that rank ``reader`` reads at this layer -- through the layer's window from
        its main input (edge 0), one to one from its residual tensor (edge 1) -- and that rank ``owner`` (< reader) computed."""
        l = self.layers[layer]
        lo, hi = owned_rows(self.plan, layer, self.table, reader)
        out = []
        edges = [(0, l.input_from, rows_read(l, lo, hi, self._h_in(layer)))]
        if l.residual_from != -2:
            edges.append((1, l.residual_from, (lo, hi)))
        for edge, src, (a, b) in edges:
            if src < 0 or b <= a:
                continue                                       # the chain input arrives from the host with its halo
            own_lo, _ = owned_rows(self.plan, src, self.table, reader)
            o_lo, o_hi = owned_rows(self.plan, src, self.table, owner)
            lo2, hi2 = max(a, o_lo), min(min(b, own_lo), o_hi)
            if lo2 < hi2:
                out.append((edge, src, lo2, hi2))
        return out

    def post_sends(self, layer):
        for reader in range(self.rank + 1, self.world):
            for edge, src, lo, hi in self._wanted_from(layer, reader, self.rank):
                self.tr.send(self.rank, reader, 2 * layer + edge, self.tensor(src)[:, lo:hi])

    def receive_and_compute(self, layer):
        for owner in range(self.rank):
            for edge, src, lo, hi in self._wanted_from(layer, self.rank, owner):
                self.tr.recv(owner, self.rank, 2 * layer + edge, self.tensor(src)[:, lo:hi])
        lo, hi = owned_rows(self.plan, layer, self.table, self.rank)
        if hi > lo:
            self.compute(layer, lo, hi)
            self.rows_computed += hi - lo
        self.tr.flush()

    def run(self):
        """All layers, for ranks that each live in a process of their own."""
        for i in range(len(self.layers)):
            self.post_sends(i)
            self.receive_and_compute(i)
