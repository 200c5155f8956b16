"""Append-and-attend (one whole generate step of the attention layer; paper Sections 2.2 and 3.3).

CPU part: the oracle's append step pinned against the split/merge identity (attending over n+1 rows
equals merging the attention over the old n rows with the one-row attention over the new row) and
against a cache built independently.  GPU part: the library's mqa_append_decode against the oracle,
including the in-place cache and length updates."""
import math

import numpy as np
import pytest
import torch

from mqa_workloads import make_custom
from oracle import ref


def _new_rows(B, D, seed):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn((B, D), generator=g).to(torch.bfloat16), torch.randn((B, D), generator=g).to(torch.bfloat16))


def test_oracle_append_equals_merge_of_old_cache_and_new_row():
    B, H, D, L = 3, 4, 16, 12
    q, k, v, lengths = make_custom(B, H, D, L, seed=41, lengths=[11, 0, 5])
    k_new, v_new = _new_rows(B, D, 42)
    sc = 0.3
    out, k2, v2, l2 = ref.mqa_append_decode_ref(q, k_new, v_new, k, v, lengths, sc)
    assert l2.tolist() == [12, 1, 6]
    for b in range(B):
        n = int(lengths[b])
        # the new row, alone, as a one-row cache
        m1, z1, a1 = ref.mqa_ref_partial(q, k2, v2, l2, b, n, n + 1, sc)
        m0, z0, a0 = ref.mqa_ref_partial(q, k, v, lengths, b, 0, n, sc)
        for h in range(H):
            merged = ref.mqa_ref_merge(np.array([m0[h], m1[h]]), np.array([z0[h], z1[h]]), np.stack([a0[h], a1[h]]))
            np.testing.assert_allclose(out[b, h], merged, rtol=1e-12, atol=1e-14)
    # rows other than the appended one are untouched; the appended rows hold the new bits
    kb, vb = ref.as_bits(k), ref.as_bits(v)
    for b in range(B):
        n = int(lengths[b])
        assert np.array_equal(k2[b, :n], kb[b, :n]) and np.array_equal(k2[b, n + 1:], kb[b, n + 1:])
        assert np.array_equal(k2[b, n], ref.as_bits(k_new)[b]) and np.array_equal(v2[b, n], ref.as_bits(v_new)[b])


def test_oracle_append_on_a_full_cache_changes_nothing():
    B, H, D, L = 2, 2, 8, 4
    q, k, v, lengths = make_custom(B, H, D, L, seed=43, lengths=[4, 2])
    k_new, v_new = _new_rows(B, D, 44)
    out, k2, v2, l2 = ref.mqa_append_decode_ref(q, k_new, v_new, k, v, lengths, 0.5)
    assert l2.tolist() == [4, 3]
    assert np.array_equal(k2[0], ref.as_bits(k)[0]) and np.array_equal(v2[0], ref.as_bits(v)[0])
    assert np.array_equal(out[0], ref.mqa_decode_ref(q, k, v, lengths, 0.5)[0])


@pytest.mark.gpu
@pytest.mark.parametrize("B,H,D,Lmax,lengths", [
    (4, 48, 256, 700, [699, 0, 127, 128]),
    (3, 16, 128, 300, [10, 255, 299]),
    (2, 4, 64, 128, [5, 64]),
])
def test_append_decode_matches_the_oracle(B, H, D, Lmax, lengths):
    from paper_2211_05102_b200 import binding
    from gpu_util import assert_close
    q, k, v, ln = make_custom(B, H, D, Lmax, seed=45 + H, lengths=lengths)
    k_new, v_new = _new_rows(B, D, 46)
    scale = 1.0 / math.sqrt(D)
    expect, k2, v2, l2 = ref.mqa_append_decode_ref(q, k_new, v_new, k, v, ln, scale)
    dev = torch.device("cuda:0")
    kd, vd, ld = k.to(dev), v.to(dev), ln.to(dev)
    out = torch.empty((B, H, D), dtype=torch.float32, device=dev)
    ws = binding.alloc_workspace(B, H, D, Lmax)
    binding.mqa_append_decode(q.to(dev), k_new.to(dev), v_new.to(dev), kd, vd, ld, out, scale, ws)
    assert binding.mqa_check_status(ws) == binding.MQA_OK
    assert_close(out.cpu(), expect, "append+decode")
    assert ld.cpu().tolist() == l2.tolist()
    assert np.array_equal(ref.as_bits(kd.cpu()), k2) and np.array_equal(ref.as_bits(vd.cpu()), v2)
    assert binding.mqa_last_launch_count() >= 2
    # a second step on the updated cache
    k_new2, v_new2 = _new_rows(B, D, 47)
    expect2, k3, v3, l3 = ref.mqa_append_decode_ref(q, k_new2, v_new2, k2, v2, l2, scale)
    binding.mqa_append_decode(q.to(dev), k_new2.to(dev), v_new2.to(dev), kd, vd, ld, out, scale, ws)
    full = any(int(x) >= Lmax for x in l2)       # a sequence that the first step filled up
    assert binding.mqa_check_status(ws) == (binding.MQA_ERR_CACHE_FULL if full else binding.MQA_OK)
    assert_close(out.cpu(), expect2, "second step")
    assert ld.cpu().tolist() == l3.tolist()


@pytest.mark.gpu
def test_append_to_a_full_cache_is_reported_and_harmless():
    from paper_2211_05102_b200 import binding
    from gpu_util import assert_close
    B, H, D, Lmax = 2, 16, 128, 256
    q, k, v, ln = make_custom(B, H, D, Lmax, seed=48, lengths=[256, 100])
    k_new, v_new = _new_rows(B, D, 49)
    expect, k2, v2, l2 = ref.mqa_append_decode_ref(q, k_new, v_new, k, v, ln, 0.1)
    dev = torch.device("cuda:0")
    kd, vd, ld = k.to(dev), v.to(dev), ln.to(dev)
    out = torch.empty((B, H, D), dtype=torch.float32, device=dev)
    ws = binding.alloc_workspace(B, H, D, Lmax)
    binding.mqa_append_decode(q.to(dev), k_new.to(dev), v_new.to(dev), kd, vd, ld, out, 0.1, ws)
    assert binding.mqa_check_status(ws) == binding.MQA_ERR_CACHE_FULL
    assert binding.mqa_check_status(ws) == binding.MQA_OK          # the status word was reset
    assert_close(out.cpu(), expect, "full cache")
    assert ld.cpu().tolist() == [256, 101]
    assert np.array_equal(ref.as_bits(kd.cpu()), k2)
