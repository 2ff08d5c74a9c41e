"""The N > 1 leg of bench.py ("replicas only"): units add up over ranks, time is the slowest
rank's.  Run as two gloo ranks on CPU."""
import os
import socket
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, world, rank)
    # rank r moved (r+1) GB in (r+1)*2 ms: total 3 GB, slowest 4 ms -> 750 GB/s, 75k seq/s
    gbs, seqs, ms = bench.aggregate_replicas((rank + 1) * 1e9, 100 * (rank + 1), 2.0 * (rank + 1), torch.device("cpu"))
    ret[rank] = (gbs, seqs, ms)
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    ret = ctx.Manager().dict()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, ret)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    for r in range(2):
        gbs, seqs, ms = ret[r]
        assert ms == pytest.approx(4.0) and gbs == pytest.approx(750.0) and seqs == pytest.approx(75000.0)


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    gbs, seqs, ms = bench.aggregate_replicas(2e9, 64, 0.5, torch.device("cpu"))
    assert gbs == pytest.approx(4000.0) and seqs == pytest.approx(128000.0) and ms == 0.5
