"""mqa_decode_scatter on one GPU: the destination buffers of the fused output exchange are separate local
allocations here (the kernel stores through plain pointers and cannot tell them from peer memory).  Every
destination must hold its head group of the oracle result in the rows of this rank's batch slice, and nothing
else may be written."""
import math

import numpy as np
import pytest
import torch

from mqa_workloads import make_custom, poison_padding
from oracle import ref
from paper_2211_05102_b200 import binding

from gpu_util import TOL

pytestmark = pytest.mark.gpu
CANARY = -float(2 ** 100)      # exactly representable in fp32


def _run(B, H, D, Lmax, lengths, n_dst, b_offset, B_total, seed):
    q, k, v, ln = make_custom(B, H, D, Lmax, seed=seed, lengths=lengths)
    k, v = poison_padding(k, v, ln, 0x7FC0)
    expect = ref.mqa_decode_ref(q, k, v, ln, 1.0 / math.sqrt(D))
    dev = torch.device("cuda:0")
    hpd = H // n_dst
    dst = [torch.full((B_total, hpd, D), CANARY, dtype=torch.float32, device=dev) for _ in range(n_dst)]
    ws = binding.alloc_workspace(B, H, D, Lmax)
    binding.mqa_decode_scatter(q.to(dev), k.to(dev), v.to(dev), ln.to(dev), dst, b_offset, 1.0 / math.sqrt(D), ws)
    assert binding.mqa_check_status(ws) == binding.MQA_OK
    torch.cuda.synchronize()
    worst = 0.0
    for r in range(n_dst):
        got = dst[r].cpu().double().numpy()
        mine = got[b_offset:b_offset + B]
        ref_r = expect[:, r * hpd:(r + 1) * hpd, :]
        ratio = np.abs(mine - ref_r) / (TOL * (1.0 + np.abs(ref_r)))
        worst = max(worst, float(ratio.max()))
        assert (got[:b_offset] == CANARY).all() and (got[b_offset + B:] == CANARY).all(), "rows of other ranks were touched"
    assert worst <= 1.0, f"max err/tol = {worst:.3f}"
    return worst


@pytest.mark.parametrize("n_dst", [1, 2, 3, 8])
def test_scatter_whole_and_cut_sequences(n_dst):
    # long sequences are cut across blocks (merged in the kernel), short ones are written by one block,
    # empty ones are zeroed: all three store paths scatter
    H = 48
    lengths = [3000, 0, 1, 129, 2500, 64, 700, 0, 1800, 333, 2047, 5]
    _run(len(lengths), H, 256, 3000, lengths, n_dst, b_offset=5, B_total=24, seed=900 + n_dst)


@pytest.mark.parametrize("H,D,n_dst", [(16, 128, 4), (64, 256, 16), (8, 256, 8), (32, 128, 2)])
def test_scatter_shapes(H, D, n_dst):
    lengths = [257 + 31 * i for i in range(20)]
    _run(len(lengths), H, D, 900, lengths, n_dst, b_offset=0, B_total=len(lengths), seed=1234 + H)


def test_scatter_uniform_batch_adaptive():
    # equal tile counts: the adaptive plan shares the tiles among fewer blocks; the scattered stores follow
    _run(64, 48, 256, 1024, [1024] * 64, 8, b_offset=64, B_total=192, seed=5)


def test_scatter_rejects_bad_arguments():
    dev = torch.device("cuda:0")
    B, H, D, Lmax = 2, 48, 256, 64
    q, k, v, ln = make_custom(B, H, D, Lmax, seed=1, lengths=[64, 3])
    ws = binding.alloc_workspace(B, H, D, Lmax)
    args = (q.to(dev), k.to(dev), v.to(dev), ln.to(dev))
    five = [torch.empty((B, 9, D), dtype=torch.float32, device=dev) for _ in range(5)]   # 48 % 5 != 0
    with pytest.raises((binding.MqaError, AssertionError)):
        binding.mqa_decode_scatter(*args, five, 0, 1 / 16, ws)
    two = [torch.empty((B, 24, D), dtype=torch.float32, device=dev) for _ in range(2)]
    with pytest.raises(binding.MqaError):
        binding.mqa_decode_scatter(*args, two, 1, 1 / 16, ws)       # b_offset + B > B_total
    q64, k64, v64, ln64 = make_custom(B, 4, 64, Lmax, seed=1, lengths=[64, 3])
    with pytest.raises(binding.MqaError):                           # D = 64 has no tensor-core path
        binding.mqa_decode_scatter(q64.to(dev), k64.to(dev), v64.to(dev), ln64.to(dev),
                                   [torch.empty((B, 2, 64), dtype=torch.float32, device=dev) for _ in range(2)],
                                   0, 0.125, binding.alloc_workspace(B, 4, 64, Lmax))


@pytest.mark.parametrize("fused", [False, True])
def test_batch_sharded_attention_single_rank(fused):
    """The whole step object on a one-rank NCCL group (this run has one GPU): exchanges degenerate to copies,
    the fused path scatters into its own symmetric buffer."""
    import os
    import torch.distributed as dist
    from paper_2211_05102_b200 import sharded

    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29533")
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda:0"))
    try:
        B, H, D, Lmax = 9, 48, 256, 600
        q, k, v, ln = make_custom(B, H, D, Lmax, seed=31, lengths=[600, 1, 0, 300, 129, 64, 599, 17, 256])
        expect = ref.mqa_decode_ref(q, k, v, ln, 1 / 16)
        dev = torch.device("cuda:0")
        try:
            att = sharded.BatchShardedAttention(B, H, D, Lmax, device=dev, fused_out=fused)
        except (RuntimeError, ImportError, AttributeError) as e:   # symmetric memory unavailable in this build of torch
            if fused:
                pytest.skip(f"symmetric memory not available: {e}")
            raise
        out = att.step(q.to(dev), k.to(dev), v.to(dev), ln.to(dev), 1 / 16)
        torch.cuda.synchronize()
        got = out.cpu().double().numpy()
        ratio = np.abs(got - expect) / (TOL * (1.0 + np.abs(expect)))
        assert float(ratio.max()) <= 1.0
    finally:
        if created:
            dist.destroy_process_group()
