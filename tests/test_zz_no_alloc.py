"""The allocation-free entry point, mqa_decode_static.

Some users of this library cannot allocate device memory (their host application
owns the whole GPU, or their serving loop may not call the allocator), so they
cannot hand mqa_decode a workspace.  mqa_decode_static keeps its scratch in a
fixed array inside the library instead.  This test calls it through the C ABI
twice in a row, on different inputs, and checks each result against the regular
entry point; the second call also shows that whatever the first call left in the
shared array does no harm.  The file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

from mqa_workloads import make_custom
from paper_2211_05102_b200 import binding

pytestmark = pytest.mark.gpu

TOL = 2e-3   # same bound as the parity tests: |a - b| <= TOL * (1 + |b|)


def _regular(qd, kd, vd, ld, scale):
    B, H, D = qd.shape
    out = torch.empty((B, H, D), dtype=torch.float32, device=qd.device)
    ws = binding.alloc_workspace(B, H, D, kd.shape[1], device=qd.device)
    binding.mqa_decode(qd, kd, vd, ld, out, scale, ws)
    assert binding.mqa_check_status(ws) == binding.MQA_OK
    return out


def test_static_workspace_matches_the_regular_entry_point_twice():
    dev = torch.device("cuda:0")
    cases = [
        # a long ragged batch that is cut across many blocks, then a different, smaller one
        (5, 48, 256, 6000, [6000, 1, 2500, 0, 4097], 91),
        (3, 16, 128, 900, [900, 17, 640], 92),
    ]
    for (B, H, D, Lmax, lengths, seed) in cases:
        q, k, v, ln = make_custom(B, H, D, Lmax, seed=seed, lengths=lengths)
        qd, kd, vd, ld = q.to(dev), k.to(dev), v.to(dev), ln.to(dev)
        scale = 1.0 / float(np.sqrt(D))
        expect = _regular(qd, kd, vd, ld, scale)
        out = torch.full((B, H, D), float("nan"), dtype=torch.float32, device=dev)
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated(dev)
        binding.mqa_decode_static(qd, kd, vd, ld, out, scale)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated(dev) == before
        a, b = out.double().cpu().numpy(), expect.double().cpu().numpy()
        assert np.isfinite(a).all()
        assert (np.abs(a - b) <= TOL * (1 + np.abs(b))).all()


def test_static_workspace_rejects_what_does_not_fit():
    """A batch whose per-sequence records alone exceed the fixed array is refused on the host,
    before anything is launched (the pointers below are never dereferenced)."""
    rc = binding.lib().mqa_decode_static(0x1000, 0x2000, 0x3000, 0x4000, 0x5000,
                                         3_000_000, 1, 64, 1, 1.0, None)
    assert rc == binding.MQA_ERR_WORKSPACE_TOO_SMALL
    assert 256 + 12 * 3_000_000 > binding.MQA_STATIC_WORKSPACE_BYTES
