"""Batch-sharded attention across ranks (Section 3.3, Figure 5), on CPU with gloo: the q and out exchanges
between the heads-sharded and the batch-sharded layout, with the fp64 oracle standing in for the local
attention kernel.  Every rank must end up with its head group of the full-batch oracle result."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from mqa_workloads import make_custom, shard_batch
from oracle import ref
from paper_2211_05102_b200 import sharded


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _oracle_attention(q, k, v, lengths, scale):
    if q.shape[0] == 0:
        return torch.empty(q.shape, dtype=torch.float32)
    return torch.from_numpy(ref.mqa_decode_ref(q.contiguous(), k.contiguous(), v.contiguous(),
                                               lengths.contiguous(), scale, num_threads=1)).float()


def _worker(rank, world, port, B, H, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        D, L = 64, 90
        lens = [(17 * i + 3) % (L + 1) for i in range(B)]
        q, k, v, lengths = make_custom(B, H, D, L, seed=77, lengths=lens)
        full = ref.mqa_decode_ref(q, k, v, lengths, 0.125, num_threads=1)          # [B, H, D] fp64
        hpd = H // world
        b0, b1 = sharded.batch_slice(B, world, rank)
        att = sharded.BatchShardedAttention(B, H, D, L, local_attention=_oracle_attention)
        q_heads = q[:, rank * hpd:(rank + 1) * hpd, :].contiguous()                 # this rank's head group
        out_heads = att.step(q_heads, k[b0:b1].contiguous(), v[b0:b1].contiguous(), lengths[b0:b1].contiguous(), 0.125)
        expect = full[:, rank * hpd:(rank + 1) * hpd, :].astype(np.float32)
        # the exchange itself, round trip: heads -> batch -> heads is the identity
        rt = sharded.batch_to_heads(sharded.heads_to_batch(q_heads), B)
        qb = sharded.heads_to_batch(q_heads)
        ret[rank] = (tuple(out_heads.shape), bool(np.array_equal(out_heads.numpy(), expect)),
                     bool(torch.equal(rt, q_heads)), bool(torch.equal(qb, q[b0:b1])), (b0, b1))
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,B,H", [(2, 5, 4), (2, 4, 6), (3, 7, 6)])
def test_batch_sharded_step_matches_the_full_batch(world, B, H):
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, port, B, H, ret), nprocs=world, join=True)
    assert len(ret) == world
    covered = []
    for r in range(world):
        shape, same, roundtrip, q_batch_ok, (b0, b1) = ret[r]
        assert shape == (B, H // world, 64)
        assert same, f"rank {r}: its head group differs from the full-batch oracle"
        assert roundtrip and q_batch_ok
        assert (b0, b1) == shard_batch(B, world, r)
        covered.extend(range(b0, b1))
    assert covered == list(range(B))


def test_exchanged_bytes():
    # PaLM-540B-shaped step on 8 ranks: q leaves as bf16 head groups, out comes back as fp32 batch slices
    e = sharded.exchanged_bytes_per_step(512, 48, 256, 8)
    assert e["q_bytes_sent"] == 512 * 6 * 256 * 2 * 7 // 8
    assert e["out_bytes_sent"] == 64 * 48 * 256 * 4 * 7 // 8
    kv_per_rank = 2 * 64 * 2048 * 256 * 2
    assert (e["q_bytes_sent"] + e["out_bytes_sent"]) < kv_per_rank // 20     # the exchange is small next to the cache
