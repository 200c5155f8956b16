"""Multi-rank plumbing on CPU (gloo, world size 2): the batch-sharded layout of the paper's
Section 3.3 gives every rank whole sequences, so the only cross-rank traffic of the benchmark
is the max-over-ranks of the step time.  Checked here: the batch slices tile the batch, each
rank's oracle output on its slice equals the matching rows of the full-batch oracle output
(no data crosses ranks inside the attention), and the time reduction is a MAX."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from mqa_workloads import make_custom, shard_batch
from oracle import ref


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, H, D, L = 5, 4, 64, 70
        q, k, v, lengths = make_custom(B, H, D, L, seed=31, lengths=[70, 1, 33, 0, 64])
        b0, b1 = shard_batch(B, world, rank)
        mine = ref.mqa_decode_ref(q[b0:b1].contiguous(), k[b0:b1].contiguous(), v[b0:b1].contiguous(),
                                  lengths[b0:b1].contiguous(), 0.125, num_threads=1)
        full = ref.mqa_decode_ref(q, k, v, lengths, 0.125, num_threads=1)
        same = bool(np.array_equal(mine, full[b0:b1]))
        # the benchmark's only collective: max over ranks of the elapsed time
        t = torch.tensor([10.0 + rank, 1.0 - rank], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        sizes = torch.tensor([b1 - b0], dtype=torch.int64)
        dist.all_reduce(sizes, op=dist.ReduceOp.SUM)
        dist.barrier()
        ret[rank] = (same, t.tolist(), int(sizes[0]), (b0, b1))
    finally:
        dist.destroy_process_group()


def test_batch_sharding_over_two_gloo_ranks():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, port, ret), nprocs=world, join=True)
    assert len(ret) == world
    covered = []
    for r in range(world):
        same, t, total, (b0, b1) = ret[r]
        assert same, f"rank {r}: its slice differs from the full-batch result"
        assert t == [11.0, 1.0]
        assert total == 5
        covered.extend(range(b0, b1))
    assert covered == list(range(5))


def test_shard_batch_tiles_any_batch():
    for B in (1, 2, 7, 512, 513):
        for world in (1, 2, 3, 8):
            got = []
            for r in range(world):
                b0, b1 = shard_batch(B, world, r)
                assert 0 <= b0 <= b1 <= B
                got.extend(range(b0, b1))
            assert got == list(range(B))
            sizes = [shard_batch(B, world, r)[1] - shard_batch(B, world, r)[0] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
