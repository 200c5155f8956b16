"""Byte and flop accounting for multiquery decode attention (host arithmetic only).

The paper's memory-time model (Section 2, "Memory costs"): the KV cache is read
from HBM once per decode step, so the floor on the step's time is
cache bytes / HBM bandwidth.  The same model gives Table 1's maximum context
lengths and Section 2.1's 3 TB multihead cache, which the tests use as pins.
"""
from __future__ import annotations

BF16_BYTES = 2


def kv_bytes_per_token(n_layers: int, kv_heads: int, d_head: int, elem_bytes: int = BF16_BYTES) -> int:
    """Bytes of K plus V that one cached token occupies across all layers."""
    return 2 * n_layers * kv_heads * d_head * elem_bytes


def max_context_length(total_hbm_bytes: float, kv_fraction: float, batch: int,
                       n_layers: int, kv_heads: int, d_head: int, replication: int = 1,
                       elem_bytes: int = BF16_BYTES) -> float:
    """Longest context whose cache fits the reserved share of memory (Table 1).
    ``replication`` is how many chips hold a copy of each cache entry (the
    heads-sharded multiquery layout replicates the single K/V head on every chip)."""
    per_tok = kv_bytes_per_token(n_layers, kv_heads, d_head, elem_bytes) * replication
    return total_hbm_bytes * kv_fraction / (per_tok * batch)


def ideal_kv_bytes(total_valid_rows: int, D: int, elem_bytes: int = BF16_BYTES) -> int:
    """Algorithmic HBM bytes of one decode-attention step of one layer: every valid
    K row and V row is read once and shared by all query heads (Section 3.3)."""
    return 2 * int(total_valid_rows) * D * elem_bytes


def step_flops(total_valid_rows: int, H: int, D: int) -> int:
    """2*H*D for the logits plus 2*H*D for the weighted value sum, per cached row."""
    return 4 * H * D * int(total_valid_rows)


def memory_time_us(nbytes: float, gb_per_s: float) -> float:
    return nbytes / (gb_per_s * 1e9) * 1e6
