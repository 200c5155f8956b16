"""Pins for the fp64 oracle against things the mathematics and the paper fix.

None of these re-type the oracle's own formula: they use closed forms,
invariances, brute-force multihead attention written a different way, and a
library float64 attention routine.  (Paper: Section 3.3 defines multiquery
attention as n_heads query heads sharing one key/value head.)
"""
import math

import numpy as np
import pytest
import torch

from mqa_workloads import WORKLOADS, make_custom, make_inputs, poison_padding
from oracle import ref


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float64).numpy()


def bits(x: float) -> int:
    return int(torch.tensor([x], dtype=torch.bfloat16).view(torch.int16).item()) & 0xFFFF


SMALL = [(1, 1, 1, 1), (2, 3, 4, 5), (3, 5, 8, 9), (2, 4, 64, 33), (1, 48, 256, 70)]


@pytest.mark.parametrize("B,H,D,L", SMALL)
def test_weights_are_a_distribution(B, H, D, L):
    q, k, v, _ = make_custom(B, H, D, L, seed=11)
    lengths = torch.tensor([(L if b % 2 == 0 else max(1, L // 2)) for b in range(B)], dtype=torch.int32)
    w = ref.mqa_ref_weights(q, k, lengths, 1.0 / math.sqrt(D))
    assert (w >= 0).all()
    for b in range(B):
        n = int(lengths[b])
        np.testing.assert_allclose(w[b, :, :n].sum(-1), 1.0, rtol=0, atol=1e-12)
        assert (w[b, :, n:] == 0).all()


def test_weights_times_v_is_the_output():
    q, k, v, lengths = make_custom(2, 5, 16, 21, seed=5, lengths=[21, 13])
    sc = 0.3
    w = ref.mqa_ref_weights(q, k, lengths, sc)
    out = ref.mqa_decode_ref(q, k, v, lengths, sc)
    expect = np.einsum("bhl,bld->bhd", w, bf16_to_f64(v))
    np.testing.assert_allclose(out, expect, rtol=1e-12, atol=1e-13)


def test_length_one_returns_v0_bit_exactly():
    q, k, v, _ = make_custom(3, 4, 32, 8, seed=3)
    lengths = torch.ones(3, dtype=torch.int32)
    out = ref.mqa_decode_ref(q, k, v, lengths, 0.7)
    v0 = bf16_to_f64(v[:, 0, :])
    for h in range(4):
        assert np.array_equal(out[:, h, :], v0)


def test_constant_v_returns_the_constant():
    q, k, v, lengths = make_custom(2, 6, 16, 40, seed=4, lengths=[40, 17])
    c = torch.tensor(1.375, dtype=torch.bfloat16)
    v[:] = c
    out = ref.mqa_decode_ref(q, k, v, lengths, 0.25)
    np.testing.assert_allclose(out, float(c), rtol=1e-12)


def test_length_two_is_a_sigmoid_blend():
    q, k, v, _ = make_custom(2, 3, 8, 4, seed=6)
    lengths = torch.full((2,), 2, dtype=torch.int32)
    sc = 0.35
    out = ref.mqa_decode_ref(q, k, v, lengths, sc)
    qf, kf, vf = bf16_to_f64(q), bf16_to_f64(k), bf16_to_f64(v)
    for b in range(2):
        for h in range(3):
            s0 = float(np.float32(sc)) * float(qf[b, h] @ kf[b, 0])
            s1 = float(np.float32(sc)) * float(qf[b, h] @ kf[b, 1])
            g = 1.0 / (1.0 + math.exp(-(s0 - s1)))
            expect = g * vf[b, 0] + (1.0 - g) * vf[b, 1]
            np.testing.assert_allclose(out[b, h], expect, rtol=1e-12, atol=1e-14)


def test_zero_query_or_zero_scale_gives_the_mean_of_valid_rows():
    q, k, v, lengths = make_custom(2, 3, 16, 12, seed=7, lengths=[12, 5])
    vf = bf16_to_f64(v)
    out = ref.mqa_decode_ref(q, k, v, lengths, 0.0)
    for b in range(2):
        n = int(lengths[b])
        np.testing.assert_allclose(out[b], np.broadcast_to(vf[b, :n].mean(0), out[b].shape), rtol=1e-12, atol=1e-14)
    q0 = torch.zeros_like(q)
    out = ref.mqa_decode_ref(q0, k, v, lengths, 0.5)
    for b in range(2):
        n = int(lengths[b])
        np.testing.assert_allclose(out[b], np.broadcast_to(vf[b, :n].mean(0), out[b].shape), rtol=1e-12, atol=1e-14)


def test_one_dominant_logit_selects_its_value_row():
    B, H, D, L = 1, 2, 16, 10
    q, k, v, lengths = make_custom(B, H, D, L, seed=8)
    j = 6
    qf = q[0, 0].to(torch.float32)
    # make k_j strongly aligned with head 0's query and the other rows orthogonal-ish small
    k[0] = (k[0].to(torch.float32) * 0.01).to(torch.bfloat16)
    k[0, j] = (qf * (60.0 / float(qf @ qf))).to(torch.bfloat16)
    out = ref.mqa_decode_ref(q, k, v, lengths, 1.0)
    np.testing.assert_allclose(out[0, 0], bf16_to_f64(v[0, j]), rtol=0, atol=1e-12)


def test_joint_row_permutation_leaves_the_output_unchanged():
    q, k, v, lengths = make_custom(2, 4, 16, 19, seed=9)
    out = ref.mqa_decode_ref(q, k, v, lengths, 0.25)
    perm = torch.randperm(19, generator=torch.Generator().manual_seed(1))
    out2 = ref.mqa_decode_ref(q, k[:, perm].contiguous(), v[:, perm].contiguous(), lengths, 0.25)
    np.testing.assert_allclose(out2, out, rtol=1e-12, atol=1e-14)


def test_common_key_shift_leaves_the_output_unchanged():
    # adding u to every key row shifts all logits of head h by scale*q_h.u
    B, H, D, L = 1, 3, 8, 11
    gen = torch.Generator().manual_seed(10)
    # small integers are exact in bf16 before and after the shift
    q = torch.randint(-3, 4, (B, H, D), generator=gen).to(torch.bfloat16)
    k = torch.randint(-3, 4, (B, L, D), generator=gen).to(torch.bfloat16)
    v = torch.randn((B, L, D), generator=gen).to(torch.bfloat16)
    u = torch.randint(-3, 4, (D,), generator=gen).to(torch.bfloat16)
    lengths = torch.tensor([L], dtype=torch.int32)
    out = ref.mqa_decode_ref(q, k, v, lengths, 0.125)
    out2 = ref.mqa_decode_ref(q, (k + u).contiguous(), v, lengths, 0.125)
    np.testing.assert_allclose(out2, out, rtol=1e-12, atol=1e-14)


def test_duplicating_every_row_leaves_the_output_unchanged():
    q, k, v, lengths = make_custom(2, 3, 8, 7, seed=12)
    out = ref.mqa_decode_ref(q, k, v, lengths, 0.4)
    k2 = torch.cat([k, k], dim=1).contiguous()
    v2 = torch.cat([v, v], dim=1).contiguous()
    out2 = ref.mqa_decode_ref(q, k2, v2, lengths * 2, 0.4)
    np.testing.assert_allclose(out2, out, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("B,H,D,L", [(1, 1, 1, 1), (2, 3, 4, 5), (3, 5, 8, 9)])
def test_brute_force_multihead_with_replicated_kv(B, H, D, L):
    """Multihead attention, one K/V copy per head, written with explicit Python loops."""
    q, k, v, _ = make_custom(B, H, D, L, seed=13)
    lengths = torch.tensor([max(1, L - b) for b in range(B)], dtype=torch.int32)
    sc = 1.0 / math.sqrt(D)
    out = ref.mqa_decode_ref(q, k, v, lengths, sc)
    qf, kf, vf = bf16_to_f64(q), bf16_to_f64(k), bf16_to_f64(v)
    k_mh = np.repeat(kf[:, None], H, axis=1)   # [B,H,L,D]: every head gets its own copy
    v_mh = np.repeat(vf[:, None], H, axis=1)
    sc64 = float(np.float32(sc))
    for b in range(B):
        n = int(lengths[b])
        for h in range(H):
            logits = [sc64 * sum(qf[b, h, d] * k_mh[b, h, l, d] for d in range(D)) for l in range(n)]
            big = max(logits)
            e = [math.exp(x - big) for x in logits]
            tot = math.fsum(e)
            for d in range(D):
                expect = math.fsum(e[l] * v_mh[b, h, l, d] for l in range(n)) / tot
                assert abs(out[b, h, d] - expect) <= 1e-12 * (1 + abs(expect))


@pytest.mark.parametrize("B,H,D,L", [(2, 4, 64, 128), (3, 16, 128, 257), (2, 48, 256, 300)])
def test_library_float64_attention(B, H, D, L):
    """torch's scaled_dot_product_attention on CPU in float64, K/V expanded over heads."""
    q, k, v, _ = make_custom(B, H, D, L, seed=14)
    gen = torch.Generator().manual_seed(15)
    lengths = torch.randint(1, L + 1, (B,), generator=gen, dtype=torch.int64).to(torch.int32)
    lengths[0] = L
    sc = 1.0 / math.sqrt(D)
    out = ref.mqa_decode_ref(q, k, v, lengths, sc)
    q64 = q.to(torch.float64)[:, :, None, :]                      # [B,H,1,D]
    k64 = k.to(torch.float64)[:, None].expand(B, H, L, D)
    v64 = v.to(torch.float64)[:, None].expand(B, H, L, D)
    mask = (torch.arange(L)[None, :] < lengths[:, None].to(torch.int64))[:, None, None, :]
    lib = torch.nn.functional.scaled_dot_product_attention(
        q64, k64, v64, attn_mask=mask, scale=float(np.float32(sc)))
    np.testing.assert_allclose(out, lib[:, :, 0, :].numpy(), rtol=1e-11, atol=1e-12)


def test_tiny_config_matches_library_attention():
    w = WORKLOADS["tiny"]
    q, k, v, lengths = make_inputs(w)
    out = ref.mqa_decode_ref(q, k, v, lengths, w.scale)
    q64 = q.to(torch.float64)[:, :, None, :]
    k64 = k.to(torch.float64)[:, None].expand(w.B, w.H, w.Lmax, w.D)
    v64 = v.to(torch.float64)[:, None].expand(w.B, w.H, w.Lmax, w.D)
    lib = torch.nn.functional.scaled_dot_product_attention(q64, k64, v64, scale=w.scale)
    np.testing.assert_allclose(out, lib[:, :, 0, :].numpy(), rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("cuts", [[0, 1, 23], [0, 7, 8, 23], [0, 23], [0, 5, 5, 23], [0, 3, 11, 17, 23, 40]])
def test_split_then_merge_equals_the_definition(cuts):
    """Attention over [0,n) equals the log-sum-exp merge of partials over any cut of the
    sequence axis (pins the merge formula of the combine step against the definition)."""
    B, H, D, L = 2, 4, 16, 40
    q, k, v, lengths = make_custom(B, H, D, L, seed=16, lengths=[23, 40])
    sc = 0.3
    out = ref.mqa_decode_ref(q, k, v, lengths, sc)
    b = 0
    parts = [ref.mqa_ref_partial(q, k, v, lengths, b, a, e, sc) for a, e in zip(cuts[:-1], cuts[1:])]
    for h in range(H):
        m = np.array([p[0][h] for p in parts])
        z = np.array([p[1][h] for p in parts])
        acc = np.stack([p[2][h] for p in parts])
        merged = ref.mqa_ref_merge(m, z, acc)
        np.testing.assert_allclose(merged, out[b, h], rtol=1e-12, atol=1e-14)


def test_partial_of_an_empty_range_is_neutral():
    q, k, v, lengths = make_custom(1, 2, 8, 10, seed=17, lengths=[4])
    m, z, acc = ref.mqa_ref_partial(q, k, v, lengths, 0, 6, 10, 0.5)   # beyond the length
    assert np.isneginf(m).all() and (z == 0).all() and (acc == 0).all()
    out = ref.mqa_ref_merge(np.array([-np.inf, -np.inf]), np.zeros(2), np.zeros((2, 8)))
    assert (out == 0).all()


def test_padding_rows_are_never_read():
    q, k, v, lengths = make_custom(3, 4, 16, 20, seed=18, lengths=[20, 7, 1])
    out = ref.mqa_decode_ref(q, k, v, lengths, 0.25)
    for pat in (0x7FC0, 0x7F80, 0xFF80):
        k2, v2 = poison_padding(k, v, lengths, pat)
        out2 = ref.mqa_decode_ref(q, k2, v2, lengths, 0.25)
        assert np.array_equal(out, out2)
        assert np.isfinite(out2).all()


def test_zero_length_and_clamping():
    q, k, v, _ = make_custom(3, 2, 8, 6, seed=19)
    out = ref.mqa_decode_ref(q, k, v, torch.tensor([0, -5, 99], dtype=torch.int32), 0.5)
    assert (out[0] == 0).all() and (out[1] == 0).all()
    full = ref.mqa_decode_ref(q, k, v, torch.tensor([6, 6, 6], dtype=torch.int32), 0.5)
    assert np.array_equal(out[2], full[2])


def test_result_does_not_depend_on_thread_count():
    q, k, v, lengths = make_custom(4, 6, 32, 50, seed=20, lengths=[50, 1, 33, 17])
    a = ref.mqa_decode_ref(q, k, v, lengths, 0.2, num_threads=1)
    b = ref.mqa_decode_ref(q, k, v, lengths, 0.2, num_threads=4)
    assert np.array_equal(a, b)


def test_sequences_and_heads_do_not_mix():
    """A transposed batch/head index or a wrong stride would couple rows: change one
    sequence's cache and one head's query and check that only they move."""
    q, k, v, lengths = make_custom(3, 4, 16, 12, seed=21)
    out = ref.mqa_decode_ref(q, k, v, lengths, 0.25)
    k2 = k.clone(); k2[1] = (k2[1].to(torch.float32) * -1.5).to(torch.bfloat16)
    q2 = q.clone(); q2[2, 3] = (q2[2, 3].to(torch.float32) + 1).to(torch.bfloat16)
    out2 = ref.mqa_decode_ref(q2, k2, v, lengths, 0.25)
    assert np.array_equal(out[0], out2[0])
    assert not np.array_equal(out[1], out2[1])
    assert np.array_equal(out[2, :3], out2[2, :3])
    assert not np.array_equal(out[2, 3], out2[2, 3])
