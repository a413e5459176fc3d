"""The N > 1 path is replicas plus a barrier and a max over ranks: exercised here with two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp

from paper_2605_16928_b200 import replicas


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, w, lr = replicas.env_rank_world()
    assert (r, w, lr) == (rank, world, rank)
    dist = replicas.init("gloo", w)
    replicas.barrier(dist, "cpu")
    ms = 100.0 + 50.0 * rank                      # rank 1 is the slow replica
    worst = replicas.max_over_ranks(dist, ms)
    rate = replicas.whole_job_rate(w, 131072, worst)
    replicas.barrier(dist, "cpu")
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
        f.write(f"{worst} {rate}")
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_replica(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    vals = [open(tmp_path / f"rank{r}.txt").read().split() for r in range(world)]
    for worst, rate in vals:
        assert float(worst) == 150.0                                   # max over ranks, on every rank
        assert float(rate) == pytest.approx(2 * 131072 / 0.150)        # whole-job rate: both replicas' tokens


def test_single_process_needs_no_group():
    assert replicas.init("gloo", 1) is None
    assert replicas.max_over_ranks(None, 12.5) == 12.5
    assert replicas.whole_job_rate(1, 1000, 500.0) == 2000.0
    replicas.barrier(None, "cpu")
