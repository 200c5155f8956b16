"""Seeded synthetic inputs and workload shapes for multiquery decode attention.

This module holds no arithmetic of the method: it only draws numbers and names
shapes.  It is the single piece shared by the CUDA path's tests/benchmark and
the CPU oracle's tests, so both sides see bit-identical inputs.

Recipe: q, K, V drawn i.i.d. N(0,1) in fp32 from a seeded CPU
``torch.Generator`` (stable across machines), rounded to bf16
(round-to-nearest-even).  With scale = 1/sqrt(D) the logits are then about
N(0,1): a flat softmax, the bandwidth-relevant regime.  The shapes follow the
paper's evaluation: context 2048 (Section 4, Figure 1), batch up to 512
(Section 2), contexts of 8192-32768 tokens (Section 4.2), and PaLM 540B's 48
heads of width 256 (Table D.1).  They stand in for the PaLM checkpoints the
paper measured on, which are not public.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    D: int
    Lmax: int
    seed: int
    ragged: bool = False          # lengths uniform in [1, Lmax] instead of all Lmax
    k_outlier_frac: float = 0.0   # fraction of K rows that get additive N(0, var) noise
    k_outlier_var: float = 0.0

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.D)


# The five configurations the benchmark metric is defined on.
WORKLOADS = {
    "tiny": Workload("tiny", B=2, H=4, D=64, Lmax=128, seed=221105101),
    "palm8b": Workload("palm8b", B=8, H=16, D=256, Lmax=2048, seed=221105102),
    "palm62b": Workload("palm62b", B=64, H=32, D=256, Lmax=2048, seed=221105103),
    "palm540b": Workload("palm540b", B=512, H=48, D=256, Lmax=2048, seed=221105104),
    # one eighth of palm540b (same H, D, L): small enough for multi-pass profiler captures
    "palm540b_b64": Workload("palm540b_b64", B=64, H=48, D=256, Lmax=2048, seed=221105106),
    "ragged32k": Workload("ragged32k", B=16, H=48, D=256, Lmax=32768, seed=221105105,
                          ragged=True, k_outlier_frac=0.01, k_outlier_var=2.0),
}


def _randn_bf16(shape, gen: torch.Generator, chunk_rows: int = 64) -> torch.Tensor:
    """N(0,1) fp32 -> bf16, generated in slabs so fp32 temporaries stay small."""
    out = torch.empty(shape, dtype=torch.bfloat16)
    flat = out.view(shape[0], -1)
    for r0 in range(0, shape[0], chunk_rows):
        r1 = min(shape[0], r0 + chunk_rows)
        tmp = torch.randn((r1 - r0, flat.shape[1]), generator=gen, dtype=torch.float32)
        flat[r0:r1] = tmp.to(torch.bfloat16)
    return out


def make_lengths(w: Workload, gen: torch.Generator) -> torch.Tensor:
    if w.ragged:
        return torch.randint(1, w.Lmax + 1, (w.B,), generator=gen, dtype=torch.int64).to(torch.int32)
    return torch.full((w.B,), w.Lmax, dtype=torch.int32)


def make_inputs(w: Workload, seed: int | None = None):
    """Return (q, k_cache, v_cache, lengths) as CPU tensors (bf16, bf16, bf16, int32).

    Outlier rows (``k_outlier_frac`` > 0): each cache row (b,l) is chosen
    independently with that probability, and each of its D elements receives an
    independent N(0, k_outlier_var) addend in fp32 before the bf16 rounding.
    """
    gen = torch.Generator(device="cpu")
    gen.manual_seed(w.seed if seed is None else seed)
    lengths = make_lengths(w, gen)
    q = _randn_bf16((w.B, w.H, w.D), gen)
    if w.k_outlier_frac > 0.0:
        k = torch.empty((w.B, w.Lmax, w.D), dtype=torch.bfloat16)
        std = math.sqrt(w.k_outlier_var)
        for b in range(w.B):
            base = torch.randn((w.Lmax, w.D), generator=gen, dtype=torch.float32)
            pick = torch.rand((w.Lmax,), generator=gen) < w.k_outlier_frac
            noise = torch.randn((w.Lmax, w.D), generator=gen, dtype=torch.float32) * std
            base += noise * pick[:, None].to(torch.float32)
            k[b] = base.to(torch.bfloat16)
    else:
        k = _randn_bf16((w.B, w.Lmax, w.D), gen)
    v = _randn_bf16((w.B, w.Lmax, w.D), gen)
    return q, k, v, lengths


def make_custom(B: int, H: int, D: int, Lmax: int, seed: int, lengths=None):
    """Small ad-hoc case: same recipe, explicit lengths (list/tensor) or all Lmax."""
    w = Workload(f"custom_B{B}_H{H}_D{D}_L{Lmax}", B, H, D, Lmax, seed)
    q, k, v, ln = make_inputs(w)
    if lengths is not None:
        ln = torch.as_tensor(lengths, dtype=torch.int32).reshape(B).clone()
    return q, k, v, ln


def poison_padding(k: torch.Tensor, v: torch.Tensor, lengths: torch.Tensor, pattern: int = 0x7FC0):
    """Overwrite cache rows at and beyond each length with a bf16 bit pattern
    (default: quiet NaN).  Returns new tensors."""
    k2, v2 = k.clone(), v.clone()
    pat = torch.tensor([pattern if pattern < 0x8000 else pattern - 0x10000], dtype=torch.int16)
    for b in range(k.shape[0]):
        n = int(max(0, min(int(lengths[b]), k.shape[1])))
        k2[b, n:].view(torch.int16)[:] = pat
        v2[b, n:].view(torch.int16)[:] = pat
    return k2, v2


def shard_batch(B: int, world_size: int, rank: int) -> tuple[int, int]:
    """Contiguous batch slice [b0, b1) owned by ``rank``: the paper's
    batch-sharded attention layout (Section 3.3) gives every chip B/n_chips
    whole sequences, so no data crosses chips inside the attention."""
    base, rem = divmod(B, world_size)
    b0 = rank * base + min(rank, rem)
    return b0, b0 + base + (1 if rank < rem else 0)
