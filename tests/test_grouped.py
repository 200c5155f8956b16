"""Key/value heads > 1 (grouped-query and multihead decode; the paper's Section 4.2 ablation compares
multihead with multiquery attention).  CPU: the grouped oracle pinned against the multiquery oracle
(KVH = 1), a library float64 multihead attention (KVH = H) and a per-group decomposition.  GPU: the
library's mqa_decode_grouped against the oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import ref


def _inputs(B, H, KVH, D, L, seed, lengths=None):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn((B, H, D), generator=g).to(torch.bfloat16)
    k = torch.randn((B, KVH, L, D), generator=g).to(torch.bfloat16)
    v = torch.randn((B, KVH, L, D), generator=g).to(torch.bfloat16)
    ln = torch.tensor(lengths if lengths is not None else [L] * B, dtype=torch.int32)
    return q, k, v, ln


def test_one_kv_head_is_multiquery():
    q, k, v, ln = _inputs(3, 6, 1, 16, 21, 51, [21, 1, 9])
    a = ref.gqa_decode_ref(q, k, v, ln, 0.25)
    b = ref.mqa_decode_ref(q, k[:, 0].contiguous(), v[:, 0].contiguous(), ln, 0.25)
    np.testing.assert_allclose(a, b, rtol=1e-13, atol=1e-15)


def test_h_kv_heads_is_library_multihead_attention():
    B, H, D, L = 2, 5, 32, 40
    q, k, v, ln = _inputs(B, H, H, D, L, 52, [40, 17])
    out = ref.gqa_decode_ref(q, k, v, ln, 1 / math.sqrt(D))
    mask = (torch.arange(L)[None, :] < ln[:, None].long())[:, None, None, :]
    lib = torch.nn.functional.scaled_dot_product_attention(
        q.double()[:, :, None, :], k.double(), v.double(), attn_mask=mask, scale=float(np.float32(1 / math.sqrt(D))))
    np.testing.assert_allclose(out, lib[:, :, 0].numpy(), rtol=1e-11, atol=1e-12)


def test_each_group_is_its_own_multiquery_problem():
    B, H, KVH, D, L = 2, 8, 4, 16, 30
    q, k, v, ln = _inputs(B, H, KVH, D, L, 53, [30, 11])
    out = ref.gqa_decode_ref(q, k, v, ln, 0.2)
    per = H // KVH
    for g in range(KVH):
        sub = ref.mqa_decode_ref(q[:, g * per:(g + 1) * per].contiguous(), k[:, g].contiguous(), v[:, g].contiguous(), ln, 0.2)
        np.testing.assert_allclose(out[:, g * per:(g + 1) * per], sub, rtol=1e-13, atol=1e-15)
    # changing one key/value head moves only its own query heads
    k2 = k.clone(); k2[:, 1] = (k2[:, 1].float() * -1).to(torch.bfloat16)
    out2 = ref.gqa_decode_ref(q, k2, v, ln, 0.2)
    assert np.array_equal(out[:, :per], out2[:, :per]) and np.array_equal(out[:, 2 * per:], out2[:, 2 * per:])
    assert not np.array_equal(out[:, per:2 * per], out2[:, per:2 * per])


@pytest.mark.gpu
@pytest.mark.parametrize("B,H,KVH,D,L,lengths", [
    (3, 48, 3, 256, 700, [700, 1, 129]),      # 16 query heads per K/V head: tensor-core path
    (2, 64, 8, 128, 500, [500, 333]),         # 8 per group
    (2, 16, 16, 128, 300, [300, 64]),         # multihead: one query head per K/V head (FMA path)
    (2, 8, 2, 64, 200, [0, 200]),             # D = 64 (FMA path), an empty sequence
])
def test_grouped_decode_matches_the_oracle(B, H, KVH, D, L, lengths):
    from paper_2211_05102_b200 import binding
    from gpu_util import assert_close
    q, k, v, ln = _inputs(B, H, KVH, D, L, 54 + H, lengths)
    expect = ref.gqa_decode_ref(q, k, v, ln, 1 / math.sqrt(D))
    dev = torch.device("cuda:0")
    out = torch.full((B, H, D), float("nan"), dtype=torch.float32, device=dev)
    _, ws = binding.mqa_decode_grouped(q.to(dev), k.to(dev), v.to(dev), ln.to(dev), out, 1 / math.sqrt(D))
    assert binding.mqa_check_status(ws) == binding.MQA_OK
    assert_close(out.cpu(), expect, f"KVH={KVH}")


def test_grouped_argument_errors():
    from paper_2211_05102_b200 import binding, build
    build.build()
    L = binding.lib()
    args = (0x1000, 0x2000, 0x3000, 0x4000, 0x5000)
    assert L.mqa_decode_grouped(*args, 2, 48, 5, 256, 128, 0.1, 0x10000, 1 << 28, None) == binding.MQA_ERR_UNSUPPORTED_SHAPE
    assert L.mqa_decode_grouped(*args, 2, 48, 0, 256, 128, 0.1, 0x10000, 1 << 28, None) == binding.MQA_ERR_INVALID_ARG
    assert L.mqa_decode_grouped_workspace_bytes(2, 48, 5, 256, 128) == 0
    assert L.mqa_decode_grouped_workspace_bytes(2, 48, 3, 256, 128) == binding.mqa_decode_workspace_bytes(6, 16, 256, 128)
