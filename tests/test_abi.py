"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2211_05102_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "mqa_decode.h")


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mqa_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(L):
    names = declared_functions()
    assert "mqa_decode" in names and "mqa_decode_plan" in names and len(names) >= 10
    for n in names:
        assert hasattr(L, n), f"{n} declared in the header but not exported"
    assert sorted(binding.EXPORTS) == [n for n in names]


def test_status_strings(L):
    seen = {binding.status_string(i) for i in range(9)}
    assert len(seen) == 9
    assert binding.status_string(1234) == "unknown status"


def test_workspace_bytes(L):
    assert binding.mqa_decode_workspace_bytes(0, 4, 64, 128) == 0
    assert binding.mqa_decode_workspace_bytes(2, 4, 96, 128) == 0      # D unsupported
    assert binding.mqa_decode_workspace_bytes(2, 65, 64, 128) == 0     # H > 64
    n = binding.mqa_decode_workspace_bytes(2, 4, 64, 128)
    slot = (2 * 4 + 4 * 64) * 4
    assert n == 256 + 256 + 256 + 2 * binding.MQA_MAX_CTAS * slot
    big = binding.mqa_decode_workspace_bytes(512, 48, 256, 2048)
    assert big == 256 + 4096 + 2048 + 2 * binding.MQA_MAX_CTAS * (2 * 48 + 48 * 256) * 4
    assert binding.mqa_decode_host_scratch_bytes(2, 4, 64, 128) > n


def test_plan_heuristic(L):
    p = binding.mqa_decode_plan(2, 4, 64, 128)
    assert p.path == binding.MQA_PATH_FMA and p.tile_rows == 64 and 1 <= p.num_ctas <= 4
    p = binding.mqa_decode_plan(512, 48, 256, 2048)
    assert p.path in (binding.MQA_PATH_FMA, binding.MQA_PATH_TC)
    assert p.tile_rows == (128 if p.path == binding.MQA_PATH_TC else 64)
    assert 1 <= p.num_ctas <= binding.MQA_MAX_CTAS
    with pytest.raises(binding.MqaError) as e:
        binding.mqa_decode_plan(2, 4, 96, 128)
    assert e.value.status == binding.MQA_ERR_UNSUPPORTED_SHAPE
    with pytest.raises(binding.MqaError) as e:
        binding.mqa_decode_plan(2, 4, 64, 0)
    assert e.value.status == binding.MQA_ERR_INVALID_ARG
    with pytest.raises(binding.MqaError) as e:
        binding.mqa_decode_plan(2, 4, 64, 128, path=binding.MQA_PATH_TC)   # D=64 has no tensor-core path
    assert e.value.status == binding.MQA_ERR_UNSUPPORTED_SHAPE


def _call(L, q=0x1000, k=0x2000, v=0x3000, ln=0x4000, out=0x5000, B=2, H=4, D=64, Lmax=128,
          ws=0x10000, ws_bytes=None, plan=None):
    if ws_bytes is None:
        ws_bytes = binding.mqa_decode_workspace_bytes(B, H, D, Lmax) or 1 << 20
    if plan is None:
        plan = binding.Plan(binding.MQA_PATH_FMA, 4, 64)
    return L.mqa_decode_with_plan(q, k, v, ln, out, B, H, D, Lmax, 0.125, ctypes.byref(plan), ws, ws_bytes, None)


def test_argument_errors_launch_nothing(L):
    """Fake (never dereferenced) pointers: every check below fails on the host."""
    assert _call(L, q=None) == binding.MQA_ERR_INVALID_ARG
    assert _call(L, out=None) == binding.MQA_ERR_INVALID_ARG
    assert _call(L, ws=None) == binding.MQA_ERR_INVALID_ARG
    assert _call(L, B=0) == binding.MQA_ERR_INVALID_ARG
    assert _call(L, Lmax=-1) == binding.MQA_ERR_INVALID_ARG
    assert _call(L, D=96) == binding.MQA_ERR_UNSUPPORTED_SHAPE
    assert _call(L, H=65) == binding.MQA_ERR_UNSUPPORTED_SHAPE
    assert _call(L, k=0x2008) == binding.MQA_ERR_MISALIGNED
    assert _call(L, out=0x5004) == binding.MQA_ERR_MISALIGNED
    assert _call(L, ws=0x10010) == binding.MQA_ERR_MISALIGNED
    assert _call(L, ws_bytes=1024) == binding.MQA_ERR_WORKSPACE_TOO_SMALL
    assert _call(L, plan=binding.Plan(binding.MQA_PATH_FMA, 0, 64)) == binding.MQA_ERR_INVALID_ARG
    assert _call(L, plan=binding.Plan(binding.MQA_PATH_FMA, binding.MQA_MAX_CTAS + 1, 64)) == binding.MQA_ERR_INVALID_ARG
    assert _call(L, plan=binding.Plan(binding.MQA_PATH_FMA, 4, 128)) == binding.MQA_ERR_INVALID_ARG
    assert _call(L, plan=binding.Plan(7, 4, 64)) == binding.MQA_ERR_INVALID_ARG
    assert _call(L, plan=binding.Plan(binding.MQA_PATH_TC, 4, 128)) == binding.MQA_ERR_UNSUPPORTED_SHAPE  # D=64
    assert L.mqa_append_decode(0x1000, None, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000, 2, 4, 64, 128, 0.1, 0x10000, 1 << 26, None) \
        == binding.MQA_ERR_INVALID_ARG
    assert L.mqa_append_decode(0x1000, 0x2008, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000, 2, 4, 64, 128, 0.1, 0x10000, 1 << 26, None) \
        == binding.MQA_ERR_MISALIGNED
    assert L.mqa_append_decode(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000, 2, 4, 64, 128, 0.1, 0x10000, 512, None) \
        == binding.MQA_ERR_WORKSPACE_TOO_SMALL
    assert L.mqa_check_status(None, None) == binding.MQA_ERR_INVALID_ARG
    assert L.mqa_workspace_init(None, 1 << 20, None) == binding.MQA_ERR_INVALID_ARG
    assert L.mqa_workspace_init(0x10000, 8, None) == binding.MQA_ERR_WORKSPACE_TOO_SMALL


def test_without_a_device_the_call_reports_cuda_error(L):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    assert _call(L) == binding.MQA_ERR_CUDA
