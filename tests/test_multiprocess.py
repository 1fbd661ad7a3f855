"""The N > 1 path on CPU: two gloo ranks shard a workload by sequence, and the measurement is
aggregated as the benchmark does it (all units of all ranks over the slowest rank's time)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_00419_b200 import inputs as I
from paper_2509_00419_b200 import sharding as S


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        base = I.shrink(I.CFG1, n=64, T=16, C=64, planted=4)
        w = S.shard_workload(base, rank, world)
        assert (w.B, w.n, w.T, w.C) == (base.B, base.n, base.T, base.C)         # weak scaling: same shapes
        h = I.hidden_states(w).float()
        sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sums, h.double().sum().reshape(1))
        assert len({round(float(x), 6) for x in sums}) == world                 # every rank has its own sequences
        # the slowest rank sets the time; the value counts every rank's units
        ms_local = 2.0 + rank
        value, ms = S.aggregate_throughput(units_per_rank=1000, ms_local=ms_local, world=world)
        assert ms == 2.0 + (world - 1)
        assert abs(value - 1000 * world / (ms * 1e-3)) < 1e-6
        dist.barrier()
        out.put((rank, value, ms))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_by_sequence_and_aggregate():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    got = sorted(out.get(timeout=10) for _ in range(world))
    assert [g[0] for g in got] == [0, 1] and got[0][1:] == got[1][1:]          # both ranks report the same aggregate


def test_single_process_needs_no_group():
    assert S.shard_workload(I.CFG2, 0, 1) is I.CFG2
    assert S.max_over_ranks(3.5) == 3.5
    assert S.aggregate_throughput(10, 2.0, 1) == (5000.0, 2.0)
