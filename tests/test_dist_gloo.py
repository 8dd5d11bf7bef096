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


def test_plain_gpus_flag_launches_its_own_ranks():
    # `python bench.py --gpus 2` with no WORLD_SIZE in the environment starts two ranks itself (torch.distributed.run
    # on 127.0.0.1); with --launcher-selftest the ranks do no GPU work and aggregate made-up times through gloo, so
    # the whole launch path runs here on CPU.  Rank r reports (10 + 5 r) ms: the line must carry the slower one,
    # both ranks' tokens and n_gpus = 2.
    import json
    import subprocess
    from paper_2609_20744_b200 import inputs
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--launcher-selftest",
                          "--workload", "tiny"], capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    line = lines[0]
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 15.0
    assert line["value"] == 2 * inputs.TINY.tokens / 0.015
    assert line["config"]["parallelism"] == "2 independent replicas" and line["scaling"] == "weak"


def test_both_arms_print_the_same_config_object():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2609_20744_b200 import inputs
    win = dict(chunk=1, radius=0, anchors=False)
    a = bench.layer_config(inputs.CLIP_768P, 1, win)
    assert a == bench.layer_config(inputs.CLIP_768P, 1, dict(win))
    assert set(a) == {"workload", "B", "T", "F", "H", "d", "io_dtype", "seed", "parallelism", "l2", "window"}
    assert "model" not in a


def test_implementation_bytes_of_the_768p_workload():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2609_20744_b200 import inputs
    ib = bench.implementation_bytes(inputs.CLIP_768P)
    n, dd = 3440, 128 * 128
    assert ib["statistics"] == n * dd * 4 * 5 and ib["inverse_split"] == n * dd * 2 * 9 and ib["read_states"] == n * dd * 2 * 4
    assert ib["total"] == ib["statistics"] + ib["inverse_split"] + ib["read_states"]
    assert 2.4e9 < ib["total"] < 2.7e9


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
