"""Host logic of the data-parallel path with two gloo ranks on CPU: the batch is sharded without gaps or
overlap, and the gradient blob ends up as the sum (or mean) of the ranks' blobs with its padding untouched."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_1909_09577_b200 import data_parallel as dp
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    vals = torch.arange(1024, dtype=torch.float32) * (rank + 1)
    for op in ("sum", "mean"):
        blob = vals.clone().view(torch.uint8)
        dp.all_reduce_gradients(blob, op=op)
        out[(rank, op)] = blob.view(torch.float32).numpy().copy()
    out[(rank, "shard")] = list(dp.shard(33, rank, world))
    dist.barrier()
    dist.destroy_process_group()


def test_gradient_exchange_and_sharding():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29741, out), nprocs=world, join=True)
        res = dict(out)
    base = np.arange(1024, dtype=np.float32)
    for r in range(world):
        np.testing.assert_array_equal(res[(r, "sum")], base * 3)
        np.testing.assert_array_equal(res[(r, "mean")], base * 1.5)
    assert res[(0, "shard")] + res[(1, "shard")] == list(range(33))


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    from paper_1909_09577_b200 import data_parallel as dp
    blob = torch.arange(16, dtype=torch.float32).view(torch.uint8).clone()
    assert dp.all_reduce_gradients(blob) is None
    assert list(dp.shard(10, 0, 1)) == list(range(10))
