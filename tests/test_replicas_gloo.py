"""The N > 1 path of the benchmark (independent replicas) with two CPU processes over gloo:
rank-specific workloads, the max-over-ranks timing protocol and the whole-job metric."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2502_06282_b200 import replicas, synth


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = replicas.rank_workload(synth.WORKLOADS["tiny"], rank)
        u = synth.layer_hidden(w, 0, 1)
        dist.barrier()
        ms = replicas.max_over_ranks(2.0 + rank, "cpu")          # rank 1 is the slow one
        dist.barrier()
        np.save(os.path.join(out_dir, f"r{rank}.npy"),
                np.concatenate([[w.seed, ms, replicas.job_steps_per_s(world, ms)], u.reshape(-1)[:8]]))
    finally:
        dist.destroy_process_group()


def test_two_replicas_over_gloo(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r0, r1 = (np.load(tmp_path / f"r{r}.npy") for r in range(world))
    base = synth.WORKLOADS["tiny"].seed
    assert r0[0] == base and r1[0] == base + 17                  # every rank its own sequences
    assert not np.allclose(r0[3:], r1[3:])
    assert r0[1] == r1[1] == 3.0                                 # the slowest rank sets the time
    assert np.isclose(r0[2], 2 * 1000.0 / 3.0) and r0[2] == r1[2]


def test_single_process_needs_no_group():
    assert replicas.max_over_ranks(1.25, "cpu") == 1.25
    assert replicas.job_steps_per_s(1, 2.0) == 500.0
    assert replicas.rank_workload(synth.WORKLOADS["tiny"], 0).seed == synth.WORKLOADS["tiny"].seed
