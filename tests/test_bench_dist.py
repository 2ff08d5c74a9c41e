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


def test_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` needs no GPU: it times the oracle on the host cores and prints one JSON
    line with the keys the benchmark contract names."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--workload", "c1",
                          "--steps", "1", "--warmup", "1"], capture_output=True, text=True, timeout=600,
                         env={**os.environ, "CUDA_VISIBLE_DEVICES": ""})
    assert res.returncode == 0, res.stderr[-2000:]
    line = json.loads(res.stdout.strip().splitlines()[-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "GB/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0


def test_byte_accounting_of_the_workloads():
    """algorithmic_bytes counts every sequence's attended K/V rows (exact token counts, not pages);
    unique_kv_bytes counts a physical row once however many sequences share its page."""
    sys.path.insert(0, ROOT)
    import workloads
    row = 2 * 8 * 128 * 2                                   # K + V, 8 KV heads, 128 values, bf16
    shared = workloads.build_case("acct", [40, 50, 33], 16, 7, "cpu", shared_prefix_tokens=32)
    assert shared.unique_kv_bytes() == (32 + 8 + 18 + 1) * row
    per_seq = 48 * 128 * 2 + 48 * 128 * 4 + 48 * 4 + 4       # q, out, lse, seq_len
    pages = 3 + 4 + 3                                        # block-table entries touched
    assert shared.algorithmic_bytes(4) == (40 + 50 + 33) * row + 3 * per_seq + pages * 4
    windowed = workloads.build_case("acct", [40, 50, 33], 16, 7, "cpu", window=20)
    assert windowed.unique_kv_bytes() == 60 * row            # nothing shared: 20 rows each
    assert list(windowed.attended_tokens()) == [20, 20, 20]
