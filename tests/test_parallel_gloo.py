"""World-size-2 gloo test of the multi-GPU plumbing (runs on CPU)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_03246_b200 import parallel


def _worker(rank, world, port, L):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = parallel.layers_of_rank(L, rank, world)
        local = {l: 1.0 + 0.25 * l for l in mine}
        full = parallel.gather_importances(local, L)
        assert torch.allclose(full, 1.0 + 0.25 * torch.arange(L, dtype=torch.float64))
        assert parallel.max_over_ranks(float(rank + 1)) == float(world)
        assert parallel.sum_over_ranks(float(len(mine))) == float(L)
    finally:
        dist.destroy_process_group()


def test_layer_sharding_is_a_partition():
    for L in (1, 7, 24, 32):
        for world in (1, 2, 3, 8):
            owned = [parallel.layers_of_rank(L, r, world) for r in range(world)]
            flat = sorted(x for o in owned for x in o)
            assert flat == list(range(L))
            assert max(len(o) for o in owned) - min(len(o) for o in owned) <= 1


def test_importance_gather_world2():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_worker, args=(2, port, 7), nprocs=2, join=True)
