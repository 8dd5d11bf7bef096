"""The N>1 benchmark path: replicas, timed as the max over ranks, units summed (world size 2, gloo, CPU)."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, results):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r "measured" (10 + 5 r) ms per step over (1000 + r) units
        ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000 + rank, world)
        results[rank] = (ms, units)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_aggregate_is_max_time_and_summed_units():
    world = 2
    port = _free_port()
    with mp.Manager() as m:
        results = m.dict()
        mp.spawn(_worker, args=(world, port, results), nprocs=world, join=True)
        got = dict(results)
    assert got[0] == got[1] == (15.0, 2001)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.0, 7, 1) == (3.0, 7)


def test_algorithmic_bytes_and_flops_of_the_768p_workload():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2609_20744_b200 import inputs
    w = inputs.CLIP_768P
    ab = bench.algorithmic_bytes(w)
    assert ab["total"] == 1 * 86 * 4080 * 40 * (4 * 128 * 2 + 4) == 14428185600
    assert ab["gram"] + ab["readout"] == ab["total"]
    assert bench.algorithmic_flops(w)["tensor"] == 6 * 86 * 4080 * 40 * 128 * 128
