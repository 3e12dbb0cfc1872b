"""Host-side pieces of the benchmark that need no GPU: the algorithmic-byte formula and the
whole-job aggregation used when N replicas run (max time over ranks, sum of units), exercised with
two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402


def test_algorithmic_bytes_per_row():
    # bytes per row: the row in, packed codes and scales out
    assert bench.algorithmic_bytes(1, 4096, 4096, 3, 0, 2) == 9732
    assert bench.algorithmic_bytes(1, 4096, 4096, 4, 0, 2) == 10244
    assert bench.algorithmic_bytes(1, 3584, 3584, 3, 128, 2) == 8624
    assert bench.algorithmic_bytes(1, 18944, 20480, 4, 0, 2) == 48132
    assert bench.algorithmic_bytes(1, 128, 128, 3, 0, 2) == 308
    assert bench.algorithmic_bytes(4096, 4096, 4096, 3, 0, 2) == 4096 * 9732


def _rank_main(rank, world, port, results):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms, units = bench.aggregate(float(rank + 1), 10.0 * (rank + 1), True, None)
        results[rank] = (ms, units)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_replica_aggregation_with_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mgr = mp.Manager()
    results = mgr.dict()
    mp.spawn(_rank_main, args=(2, port, results), nprocs=2, join=True)
    assert results[0] == (2.0, 30.0) and results[1] == (2.0, 30.0)


def test_single_process_aggregation_is_identity():
    assert bench.aggregate(3.5, 7.0, False) == (3.5, 7.0)
