"""World-size-2 gloo run of the replica timing reduction (CPU only)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2512_10310_b200.replicas import aggregate_steps_per_s, max_over_ranks


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local = 10.0 + 5.0 * rank            # rank 1 is the slow replica
    out[rank] = max_over_ranks(local, dist)
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_world2():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0] == out[1] == 15.0
    assert aggregate_steps_per_s(out[0], world) == 2 / 15e-6


def test_identity_without_process_group():
    assert max_over_ranks(3.5) == 3.5
