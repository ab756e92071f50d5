"""The N > 1 leg of bench.py on CPU: two gloo ranks, whole-job figure = units summed
over ranks divided by the slowest rank's time.  (The path itself has no exchange
between GPUs: every rank runs an independent replica.)"""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ms, units = bench.aggregate(10.0 + 5.0 * rank, 1000.0 * (rank + 1), world)
    out[rank] = (ms, units)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_over_gloo():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0] == out[1] == (15.0, 3000.0)          # max of the times, sum of the units


def test_single_rank_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(3.5, 42.0, 1) == (3.5, 42.0)


def test_algorithmic_bytes_formula():
    """Workload 3: rows + 3x IDs + 3x bag boundaries + output once is about 2.40 GB per step."""
    sys.path.insert(0, ROOT)
    import bench
    import bls_inputs as bi
    w = bi.workload(3)
    step, gather = bench.algorithmic_bytes(w, 8_519_243)
    assert abs(step - (8_519_243 * 256 + 3 * 8_519_243 * 4 + 3 * 425_984 * 4 + 425_984 * 64 * 4)) < 1
    assert 2.39e9 < step < 2.41e9 and gather < step
