"""The N > 1 path of the benchmark on CPU: two gloo ranks run the replica plumbing (distinct
seeds, barrier, maximum over ranks of the measured times, whole-job metric)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2508_12407_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local = [10.0 + rank, 3.0 - rank, 7.0 + 2 * rank]     # each rank measured different times
        replicas.barrier()
        got = replicas.max_over_ranks(local, torch.device("cpu"))
        seed = replicas.replica_seed(20250812, rank)
        with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
            f.write(" ".join(str(x) for x in got) + f" {seed}\n")
    finally:
        dist.destroy_process_group()


def test_two_rank_max_and_seeds(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    rows = [open(tmp_path / f"r{r}.txt").read().split() for r in range(world)]
    for r in rows:
        assert [float(x) for x in r[:3]] == [11.0, 3.0, 9.0]       # element-wise max over the ranks
    assert rows[0][3] != rows[1][3]                                # replicas draw different inputs


def test_single_process_is_identity():
    assert replicas.max_over_ranks([1.5, 2.5], torch.device("cpu")) == [1.5, 2.5]
    # 2 replicas x batch 1 x 256 steps in 100 ms -> 195.3 us per token of the whole job
    assert replicas.whole_job_us_per_token(100.0, 2, 1, 256) == pytest.approx(100e3 / 512)
