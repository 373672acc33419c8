"""The multi-rank plumbing of bench.py (replicas, barrier, max over ranks) on CPU with gloo, world size 2."""
import json
import os
import socket
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import bench
    r, w, local = bench.dist_setup(world, backend="gloo")
    assert (r, w, local) == (rank, world, rank)
    bench.barrier()
    seconds = bench.max_over_ranks(1.0 + rank)  # rank 1 is the slower replica
    value = bench.aggregate_value(5120, 4, w, seconds)
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"seconds": seconds, "value": value}, f)
    bench.barrier()
    import torch.distributed as dist
    dist.destroy_process_group()


def test_two_ranks_take_the_max_time_and_sum_the_work(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"r{r}.json")) for r in range(world)]
    for r in res:
        assert r["seconds"] == 2.0  # max over ranks, seen by every rank
        assert r["value"] == pytest.approx(5120 * 4 * 2 / 2.0)


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    os.environ.pop("WORLD_SIZE", None)
    assert bench.dist_setup(1) == (0, 1, 0)
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.aggregate_value(100, 2, 1, 0.5) == 400.0


def test_algorithmic_work_matches_hand_count():
    sys.path.insert(0, ROOT)
    import numpy as np
    import bench
    from paper_2511_17560_b200 import workloads as W
    m, r = W.request_for("llama8b_10x512")
    p = 772
    rows = np.concatenate([np.arange(0, 5120, 5120 // p)[:p], np.arange(5120, 5152)])
    fl, by = bench.algorithmic_work(m, r, p, rows)
    M = p + 32
    per_row = 2 * (4096 * 6144 + 4096 * 4096 + 3 * 4096 * 14336)
    gemm = fl["gemm_qkv"] + fl["gemm_residual"] + fl["gemm_swiglu"]
    expect = per_row * (5152 + 31 * M) + 2 * 4096 * (5152 * 2048 + 32 * 4096)
    assert gemm == pytest.approx(expect)
    assert by["rerotate"] == 4 * 5120 * 1024 * 2 * 30
    assert 14e12 < gemm + fl["attention"] + fl["scores"] < 15.5e12
