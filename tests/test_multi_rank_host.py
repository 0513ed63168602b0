"""World-size-2 run of the multi-GPU host logic on CPU (gloo): replicas with their own seeds, timing reduced as
the max over ranks, no data-path collective."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2507_00715_b200 import replicas, workloads as wl


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = replicas.rank_workload(wl.CONFIGS["tiny"], rank)
        q, _, _ = wl.layer_qkv(w, 0, "cpu")
        mine = 0.010 * (rank + 1)                       # rank 1 is the slow replica
        slowest = replicas.max_over_ranks(mine, dist)
        tokens = int(wl.seqlens(w).sum())
        np.save(os.path.join(out_dir, f"r{rank}.npy"),
                np.array([w.seed, slowest, replicas.job_throughput(tokens, world, slowest), float(q.double().sum())]))
    finally:
        dist.destroy_process_group()


def test_two_replicas_reduce_only_their_timing(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0, r1 = (np.load(tmp_path / f"r{r}.npy") for r in range(2))
    base = wl.CONFIGS["tiny"]
    assert int(r0[0]) == base.seed and int(r1[0]) == base.seed + replicas.SEED_STRIDE
    assert r0[3] != r1[3]                                # different seeds -> different batches
    assert r0[1] == r1[1] == 0.020                       # both ranks see the slowest rank's time
    tokens = int(wl.seqlens(base).sum())
    assert np.isclose(r0[2], 2 * tokens / 0.020) and r0[2] == r1[2]


def test_single_process_needs_no_process_group():
    assert replicas.max_over_ranks(0.5) == 0.5
    assert replicas.rank_workload(wl.CONFIGS["7b"], 0) is wl.CONFIGS["7b"]
    assert replicas.job_throughput(100, 4, 2.0) == 200.0
