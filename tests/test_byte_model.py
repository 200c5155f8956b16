"""The byte model behind the roofline, pinned to the figures the paper prints
(Table 1 and Section 2.1); fixture: tests/golden/table1_max_context.txt."""
import os

import pytest

from paper_2211_05102_b200 import roofline

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_max_context.txt")


def _rows():
    rows, extra = [], {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = line.split()
        if len(f) == 2:
            extra[f[0]] = float(f[1])
        else:
            rows.append((f[0], int(f[1]), int(f[2]), int(f[3]), int(f[4]), int(f[5])))
    return rows, extra


def test_table1_max_context_lengths():
    rows, _ = _rows()
    total = 64 * 32 * 2**30          # 64 chips x 32 GiB (Section 4)
    assert len(rows) == 3
    for name, d_head, kv_heads, repl, ctx128, ctx512 in rows:
        for batch, printed in ((128, ctx128), (512, ctx512)):
            got = roofline.max_context_length(total, 0.30, batch, 118, kv_heads, d_head, repl)
            # the paper rounds to 2-3 significant figures
            assert got == pytest.approx(printed, rel=0.015), (name, batch, got, printed)


def test_three_terabyte_multihead_cache():
    _, extra = _rows()
    got = roofline.kv_bytes_per_token(118, 48, 128) * 512 * 2048
    assert got == pytest.approx(extra["kv_total_multihead_bytes"], rel=0.02)


def test_ideal_bytes_of_the_named_configs():
    assert roofline.ideal_kv_bytes(2 * 128, 64) == 64 * 1024
    assert roofline.ideal_kv_bytes(8 * 2048, 256) == 16 * 2**20
    assert roofline.ideal_kv_bytes(64 * 2048, 256) == 128 * 2**20
    assert roofline.ideal_kv_bytes(512 * 2048, 256) == 2**30
    assert roofline.step_flops(512 * 2048, 48, 256) == pytest.approx(51.5e9, rel=0.01)
