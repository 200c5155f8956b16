"""Batch-sharded multiquery decode attention over the GPUs of one node.

Section 3.3 of the paper: with one shared key/value head, sharding attention over heads would replicate the
whole K/V cache on every chip, so the attention is sharded over the *batch* instead; the projections around
it stay sharded over heads, and an all-to-all moves the one-token tensors between the two layouts
(Figure 4 and Figure 5 show the layouts and the cache that each chip then loads: 1/n of it).

Layouts, for a group of N ranks, B_total sequences, H heads (H divisible by N):
  heads-sharded:  rank r holds [B_total, H/N, D]  - head group r of every sequence
  batch-sharded:  rank r holds [B_r, H, D]        - all heads of its contiguous slice of the batch
                                                    (`batch_slice`), and that slice of the K/V cache.

One decode step on every rank (`BatchShardedAttention.step`):
  1. q: heads-sharded -> batch-sharded (all-to-all of bf16 [B_total, H/N, D]; the smaller of the two exchanges);
  2. local attention over the rank's own cache slice (`mqa_decode`): no collective inside;
  3. out: batch-sharded -> heads-sharded, either
       - as a second all-to-all (NCCL on GPUs, gloo on CPU), or
       - fused into the attention kernel (`fused_out=True`): `mqa_decode_scatter` stores every output row
         straight into the destination rank's buffer through peer pointers (symmetric memory over NVLink),
         and the ranks meet at a barrier instead of running a collective.

Not run on more than one GPU in this build (one GPU per run): the exchange logic is covered by world-size-2
gloo tests on CPU with a CPU attention injected for step 2, and the scattering kernel by single-GPU tests in
which the destination buffers are separate local allocations (the kernel cannot tell them from peer memory).
"""
from __future__ import annotations

from typing import Callable, Sequence

import torch
import torch.distributed as dist


def batch_slice(B_total: int, world_size: int, rank: int) -> tuple[int, int]:
    """Contiguous slice [b0, b1) of the batch that ``rank`` owns (sizes differ by at most one)."""
    base, rem = divmod(B_total, world_size)
    b0 = rank * base + min(rank, rem)
    return b0, b0 + base + (1 if rank < rem else 0)


def heads_to_batch(x_heads: torch.Tensor, group=None) -> torch.Tensor:
    """[B_total, H/N, D] on every rank (head group = rank) -> [B_rank, H, D] (all heads of the rank's slice)."""
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    B_total, hpd, D = x_heads.shape
    sizes = [batch_slice(B_total, world, j)[1] - batch_slice(B_total, world, j)[0] for j in range(world)]
    B_r = sizes[rank]
    # rank j gets the rows of its slice; from rank i arrives head group i of this rank's rows
    recv = torch.empty((world * B_r, hpd, D), dtype=x_heads.dtype, device=x_heads.device)
    dist.all_to_all_single(recv, x_heads.contiguous(), output_split_sizes=[B_r] * world, input_split_sizes=sizes,
                           group=group)
    # [source rank = head group, row, head in group, D] -> [row, head, D]
    return recv.view(world, B_r, hpd, D).permute(1, 0, 2, 3).reshape(B_r, world * hpd, D).contiguous()


def batch_to_heads(x_batch: torch.Tensor, B_total: int, group=None) -> torch.Tensor:
    """[B_rank, H, D] (all heads of the rank's slice) -> [B_total, H/N, D] (the rank's head group of every sequence)."""
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    B_r, H, D = x_batch.shape
    assert H % world == 0
    hpd = H // world
    sizes = [batch_slice(B_total, world, j)[1] - batch_slice(B_total, world, j)[0] for j in range(world)]
    assert sizes[rank] == B_r
    # head group j of this rank's rows goes to rank j; from rank i arrive its rows of this rank's head group
    send = x_batch.view(B_r, world, hpd, D).permute(1, 0, 2, 3).reshape(world * B_r, hpd, D).contiguous()
    recv = torch.empty((B_total, hpd, D), dtype=x_batch.dtype, device=x_batch.device)
    dist.all_to_all_single(recv, send, output_split_sizes=sizes, input_split_sizes=[B_r] * world, group=group)
    return recv                            # batch slices in rank order = batch order


def symmetric_out_buffers(B_total: int, heads_per_rank: int, D: int, device, group=None):
    """One fp32 [B_total, H/N, D] buffer per rank, each mapped into every rank's address space.

    Returns (this rank's buffer as a tensor, list of (device pointer, B_total) per rank) for
    `mqa_decode_scatter`.  Uses PyTorch's symmetric memory (plain peer mappings; no multicast object is
    created or used by the kernel)."""
    import torch.distributed._symmetric_memory as symm_mem

    name = group.group_name if group is not None else dist.group.WORLD.group_name
    mine = symm_mem.empty((B_total, heads_per_rank, D), dtype=torch.float32, device=device)
    handle = symm_mem.rendezvous(mine, name)
    return mine, [(int(ptr), B_total) for ptr in handle.buffer_ptrs]


class BatchShardedAttention:
    """One rank's side of batch-sharded decode attention (see the module docstring).

    ``local_attention(q, k, v, lengths, scale) -> out`` replaces the CUDA kernel in CPU tests; by default the
    library's `mqa_decode` runs, and there is no fallback: without the CUDA extension the call fails."""

    def __init__(self, B_total: int, H: int, D: int, Lmax: int, group=None, device=None,
                 local_attention: Callable | None = None, fused_out: bool = False):
        self.group = group
        self.world, self.rank = dist.get_world_size(group), dist.get_rank(group)
        if H % self.world != 0:
            raise ValueError("the heads must divide evenly among the ranks")
        self.B_total, self.H, self.D, self.Lmax = B_total, H, D, Lmax
        self.b0, self.b1 = batch_slice(B_total, self.world, self.rank)
        self.device = device
        self.local_attention = local_attention
        self.fused_out = fused_out
        self._ws = None
        self._out_local = None
        self._out_heads = None
        self._dst = None
        if local_attention is None:
            from . import binding
            self._binding = binding
            self._ws = binding.alloc_workspace(max(1, self.b1 - self.b0), H, D, Lmax, device=device)
            if fused_out:
                self._out_heads, self._dst = symmetric_out_buffers(B_total, H // self.world, D, device, group)
            else:
                self._out_local = torch.empty((self.b1 - self.b0, H, D), dtype=torch.float32, device=device)
        elif fused_out:
            raise ValueError("the fused output path needs the CUDA kernel")

    def step(self, q_heads: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, lengths: torch.Tensor,
             scale: float) -> torch.Tensor:
        """q_heads: [B_total, H/N, D] bf16 (this rank's head group); k_cache/v_cache: [B_rank, Lmax, D];
        lengths: [B_rank].  Returns this rank's head group of the output, [B_total, H/N, D] fp32."""
        q_batch = heads_to_batch(q_heads, self.group)
        if self.local_attention is not None:
            out_batch = self.local_attention(q_batch, k_cache, v_cache, lengths, scale)
            return batch_to_heads(out_batch, self.B_total, self.group)
        if self.b1 > self.b0:
            if self.fused_out:
                self._binding.mqa_decode_scatter(q_batch, k_cache, v_cache, lengths, self._dst, self.b0, scale, self._ws)
            else:
                self._binding.mqa_decode(q_batch, k_cache, v_cache, lengths, self._out_local, scale, self._ws)
        if self.fused_out:
            # every rank's stores into this rank's buffer are complete once all ranks' kernels have finished
            torch.cuda.current_stream().synchronize()
            dist.barrier(group=self.group)
            return self._out_heads
        return batch_to_heads(self._out_local, self.B_total, self.group)


def exchanged_bytes_per_step(B_total: int, H: int, D: int, world: int) -> dict:
    """Bytes each rank sends per decode step: q (bf16) one way, out (fp32) the other; the share that stays on
    the rank itself (1/N) does not cross NVLink.  Compare with the K/V bytes a rank reads: 2*B_r*L*D*2."""
    per_rank_q = B_total * (H // world) * D * 2
    per_rank_out = (B_total // world) * H * D * 4
    off_rank = (world - 1) / world
    return {"q_bytes_sent": int(per_rank_q * off_rank), "out_bytes_sent": int(per_rank_out * off_rank)}
