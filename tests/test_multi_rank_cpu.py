"""The multi-process side of bench.py on CPU (gloo, world size 2): every rank runs an independent replica, the
job's time is the slowest rank's, rank 0 alone reports.  No GPU is touched."""
import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    try:
        slowest = bench.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow one
        out.put((rank, slowest, bench.job_images_per_s(8, world, slowest)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_job_time_is_the_slowest_rank_and_throughput_counts_every_replica():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    got = sorted(out.get() for _ in range(2))
    for rank, slowest, ips in got:
        assert slowest == 15.0
        assert abs(ips - 16 / 15.0e-3) < 1e-6


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.job_images_per_s(1, 1, 0.5) == 2000.0


def test_reference_arm_under_torchrun_prints_one_line_from_rank_0():
    env = dict(os.environ, OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--workload", "single_conv"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0


# ------------------------------------------------------------------------------------ band sharding (gloo, CPU tensors)
def _shard_rank(rank, world, port, out):
    """One rank of a band-sharded run on CPU: the library's planner and shard table, the package's row all-gather
    over gloo, and -- in place of the GPU kernels -- the oracle computing the rank's block of bands."""
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import lop_inputs as li
    import paper_2507_05829_b200 as lop
    from oracle import chain as ochain, planner as oplanner
    from paper_2507_05829_b200.shard import all_gather_rows, shard_table
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    try:
        wl = li.build("resnet18", H=48, W=16, width=8)
        x = wl.x
        for seg in wl.segments:
            reuse = True
            plan = lop.Plan(seg.layers, x.shape[0], x.shape[1], x.shape[2], x.shape[3], lop.LOP_BF16, seg.n_bands,
                            lop.LOP_FLAG_REUSE_HALO)
            table = shard_table(plan, world)
            oplan = oplanner.make_plan(seg.layers, x.shape[1], x.shape[2], x.shape[3], seg.n_bands, reuse)
            b0, b1, r0, r1, i0, i1 = table[rank]
            x_mine = np.full_like(x, np.inf)
            x_mine[:, i0:i1] = x[:, i0:i1]                           # the rank receives only the rows the table names
            got = ochain.run_band_block(seg.layers, x_mine, oplan, True, b0, b1, reuse)
            t = torch.from_numpy(np.where(np.isfinite(got), got, 0.0).astype(np.float32)).to(torch.bfloat16)
            assert np.isfinite(got[:, r0:r1]).all() and not np.isfinite(got[:, :r0]).any() and not np.isfinite(got[:, r1:]).any()
            all_gather_rows(t, table, rank)
            whole = ochain.run_whole(seg.layers, x, True)
            assert torch.equal(t, torch.from_numpy(whole).to(torch.bfloat16)), "rank %d: stitched rows differ" % rank
            x = whole
        out.put((rank, [list(r) for r in table]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_band_sharding_over_two_and_three_ranks_gives_the_whole_output_on_every_rank():
    ctx = mp.get_context("spawn")
    for world in (2, 3):
        out = ctx.SimpleQueue()
        port = _free_port()
        procs = [ctx.Process(target=_shard_rank, args=(r, world, port, out)) for r in range(world)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(300)
            assert p.exitcode == 0
        tables = [out.get()[1] for _ in range(world)]
        assert all(t == tables[0] for t in tables)                 # every rank derives the same table


def test_shard_table_is_the_floor_partition_of_the_bands():
    sys.path.insert(0, ROOT)
    import lop_inputs as li
    import paper_2507_05829_b200 as lop
    from oracle import planner as oplanner
    wl = li.build("vgg_block", with_data=False)
    seg = wl.segments[0]
    B = 8
    plan = lop.Plan(seg.layers, wl.N, wl.H, wl.W, wl.C, lop.LOP_BF16, B)
    oplan = oplanner.make_plan(seg.layers, wl.H, wl.W, wl.C, B)
    for world in (1, 2, 3, 5, 8, 11):
        covered = 0
        for rank in range(world):
            b0, b1, r0, r1, i0, i1 = plan.shard(rank, world)
            assert (b0, b1) == (rank * B // world, (rank + 1) * B // world)
            if b1 > b0:
                assert (r0, r1) == (oplan.ranges[b0][-1].out_lo, oplan.ranges[b1 - 1][-1].out_hi)
                assert (i0, i1) == (min(oplan.input_need[b][0] for b in range(b0, b1)), max(oplan.input_need[b][1] for b in range(b0, b1)))
                assert r0 == covered
                covered = r1
            else:
                assert (r0, r1, i0, i1) == (0, 0, 0, 0)
        assert covered == 112
    with __import__("pytest").raises(lop.LopError):
        plan.shard(2, 2)


# ------------------------------------------------------------------------------------ halo exchange (no recompute)
def _halo_setup(wl_seg_layers, x, n_bands, world, transport_of):
    """Per rank: poisoned tensors holding only the rank's input rows, the oracle as the compute step."""
    import numpy as np
    import torch
    import paper_2507_05829_b200 as lop
    from oracle import chain as ochain, planner as oplanner
    from paper_2507_05829_b200 import shard
    N, H, W, C = x.shape
    plan = lop.Plan(wl_seg_layers, N, H, W, C, lop.LOP_BF16, n_bands, lop.LOP_FLAG_REUSE_HALO)
    table = shard.shard_table(plan, world)
    shapes = oplanner.infer_shapes(wl_seg_layers, H, W, C)
    ranks = []
    for r in range(world):
        t = {-1: np.full(x.shape, np.inf, dtype=np.float32)}
        i0, i1 = table[r][4], table[r][5]
        t[-1][:, i0:i1] = x[:, i0:i1]
        for i, (h, w, c) in enumerate(shapes):
            t[i] = np.full((N, h, w, c), np.inf, dtype=np.float32)
        views = {k: torch.from_numpy(v) for k, v in t.items()}

        def compute(layer, lo, hi, t=t):
            l = wl_seg_layers[layer]
            res = t[l.residual_from] if l.residual_from != -2 else None
            ochain.run_layer(l, t[l.input_from], res, (lo, hi), True, t[layer])

        ranks.append((shard.HaloExchangeRank(plan, wl_seg_layers, table, r, lambda idx, v=views: v[idx], compute, transport_of(r)), t))
    return plan, table, ranks


def test_halo_exchange_computes_every_row_once_and_stitches_to_the_whole():
    """Ranks taking turns in one process (a mailbox carries the rows): no row is computed twice, every rank's rows are
    the whole-tensor result, and the rows traded are exactly the halo -- against the rows recomputed by the replication
    form (lop_run_shard) of the same sharding."""
    sys.path.insert(0, ROOT)
    import numpy as np
    import lop_inputs as li
    from oracle import chain as ochain
    from paper_2507_05829_b200 import shard
    for name, kw in (("vgg_block", dict(H=44, W=12, width=8)), ("resnet18", dict(H=48, W=16, width=8)), ("csp_stack", dict(H=128, W=32, base=8))):
        wl = li.build(name, **kw)
        x = wl.x
        for seg in wl.segments:
            whole = ochain.run_whole(seg.layers, x, True, keep_all=True)
            for world in (2, 3):
                box = shard.MailboxTransport()
                plan, table, ranks = _halo_setup(seg.layers, x, seg.n_bands, world, lambda r: box)
                for i in range(len(seg.layers)):
                    for hx, _ in ranks:
                        hx.post_sends(i)
                    for hx, _ in ranks:
                        hx.receive_and_compute(i)
                assert not box.box                                   # every row sent was wanted
                for i, want in enumerate(whole):
                    done = 0
                    for r, (hx, t) in enumerate(ranks):
                        lo, hi = shard.owned_rows(plan, i, table, r)
                        if hi > lo:
                            assert lo == done or done == 0           # the ranks' rows tile the layer
                            assert np.array_equal(t[i][:, lo:hi], want[:, lo:hi]), (name, world, i, r)
                            done = hi
                    assert sum(hx.rows_computed for hx, _ in ranks) >= done
                total = sum(hx.rows_computed for hx, _ in ranks)
                assert total == sum(w.shape[1] for w in whole)        # every row of every layer exactly once
            x = whole[-1]


def _halo_rank(rank, world, port, out):
    import numpy as np
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import lop_inputs as li
    from oracle import chain as ochain
    from paper_2507_05829_b200 import shard
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    try:
        wl = li.build("resnet18", H=48, W=16, width=8)
        x = wl.x
        sent = 0
        for seg in wl.segments:
            tr = shard.DistTransport()
            plan, table, ranks = _halo_setup(seg.layers, x, seg.n_bands, world, lambda r: tr)
            hx, t = ranks[rank]
            hx.run()
            whole = ochain.run_whole(seg.layers, x, True, keep_all=True)
            for i, want in enumerate(whole):
                lo, hi = shard.owned_rows(plan, i, table, rank)
                assert np.array_equal(t[i][:, lo:hi], want[:, lo:hi]), (rank, i)
            sent += tr.bytes_sent
            x = whole[-1]
        out.put((rank, sent))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_halo_exchange_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_halo_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(300)
        assert p.exitcode == 0
    got = dict(out.get() for _ in range(2))
    assert got[0] > 0 and got[1] == 0                              # rows only travel upwards: rank 0 sends, rank 1 receives
