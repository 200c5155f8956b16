"""Multihead versus multiquery decode attention at equal attention-parameter count, on one GPU.

The paper's Section 4.2 ablation: PaLM 540B with multiquery attention (one K/V head of width 256)
against a multihead variant (48 K/V heads of width 128), where the multihead KV cache is
n_heads/2 = 24 times larger and its load time dominates long-context decoding (Section 3.3, Figure 8,
Table 1).  This script times both through the C ABI on synthetic N(0,1) caches and prints one JSON line
per context length.

    python -m paper_2211_05102_b200.ablation [--batch 32] [--heads 48] [--lengths 512,2048,8192]
"""
from __future__ import annotations

import argparse
import json
import math

import torch

from . import binding


def _time_us(fn, iters=20, warm=5):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(iters):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e3 / iters


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--heads", type=int, default=48)
    ap.add_argument("--lengths", default="512,2048,8192")
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    B, H = args.batch, args.heads
    g = torch.Generator(device="cpu").manual_seed(221105)
    for L in [int(x) for x in args.lengths.split(",")]:
        lengths = torch.full((B,), L, dtype=torch.int32, device=dev)
        # multiquery: one K/V head of width 256
        q = torch.randn((B, H, 256), generator=g).to(torch.bfloat16).to(dev)
        k = torch.randn((B, L, 256), generator=g).to(torch.bfloat16).to(dev)
        v = torch.randn((B, L, 256), generator=g).to(torch.bfloat16).to(dev)
        out = torch.empty((B, H, 256), dtype=torch.float32, device=dev)
        ws = binding.alloc_workspace(B, H, 256, L)
        t_mqa = _time_us(lambda: binding.mqa_decode(q, k, v, lengths, out, 1 / 16, ws))
        mqa_bytes = 2 * B * L * 256 * 2
        del k, v
        # multihead: H K/V heads of width 128
        q2 = torch.randn((B, H, 128), generator=g).to(torch.bfloat16).to(dev)
        k2 = torch.randn((B, H, L, 128), generator=g).to(torch.bfloat16).to(dev)
        v2 = torch.randn((B, H, L, 128), generator=g).to(torch.bfloat16).to(dev)
        out2 = torch.empty((B, H, 128), dtype=torch.float32, device=dev)
        _, ws2 = binding.mqa_decode_grouped(q2, k2, v2, lengths, out2, 1 / math.sqrt(128))
        t_mha = _time_us(lambda: binding.mqa_decode_grouped(q2, k2, v2, lengths, out2, 1 / math.sqrt(128), ws2))
        mha_bytes = 2 * B * H * L * 128 * 2
        print(json.dumps({
            "batch": B, "heads": H, "context": L,
            "multiquery": {"d_head": 256, "kv_bytes": mqa_bytes, "us": round(t_mqa, 1), "GBps": round(mqa_bytes / t_mqa / 1e3)},
            "multihead": {"d_head": 128, "kv_bytes": mha_bytes, "us": round(t_mha, 1), "GBps": round(mha_bytes / t_mha / 1e3)},
            "cache_ratio": mha_bytes / mqa_bytes, "time_ratio": round(t_mha / t_mqa, 1)}), flush=True)
        del k2, v2


if __name__ == "__main__":
    main()
