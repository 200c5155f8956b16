"""ctypes binding of the C ABI in ``include/mqa_decode.h`` (argument marshalling only).

Every arithmetic step runs inside the CUDA library; this module converts torch
tensors to raw pointers and checks return codes.  It fails loudly if the
library is missing: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmqa_decode.so")

MQA_OK = 0
MQA_ERR_INVALID_ARG = 1
MQA_ERR_UNSUPPORTED_SHAPE = 2
MQA_ERR_MISALIGNED = 3
MQA_ERR_WORKSPACE_TOO_SMALL = 4
MQA_ERR_ARCH = 5
MQA_ERR_CUDA = 6
MQA_ERR_TIMEOUT = 7
MQA_ERR_CACHE_FULL = 8

MQA_PATH_AUTO = 0
MQA_PATH_FMA = 1
MQA_PATH_TC = 2
MQA_MAX_CTAS = 592

EXPORTS = [
    "mqa_status_string", "mqa_decode_workspace_bytes", "mqa_workspace_init", "mqa_decode_plan",
    "mqa_decode", "mqa_decode_with_plan", "mqa_decode_profiled", "mqa_check_status", "mqa_decode_host_scratch_bytes",
    "mqa_decode_host", "mqa_last_launch_count", "mqa_debug_schedule", "mqa_decode_static", "mqa_append_decode", "mqa_decode_grouped", "mqa_decode_grouped_workspace_bytes",
    "mqa_uniform_ctas", "mqa_decode_scatter",
]


class Plan(ctypes.Structure):
    _fields_ = [("path", ctypes.c_int), ("num_ctas", ctypes.c_int), ("tile_rows", ctypes.c_int),
                ("adaptive", ctypes.c_int)]

    def __repr__(self):
        return (f"Plan(path={self.path}, num_ctas={self.num_ctas}, tile_rows={self.tile_rows}, "
                f"adaptive={self.adaptive})")


class MqaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2211_05102_b200.build` "
                "(there is no CPU fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        vp, ci, cf, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        L.mqa_status_string.argtypes = [ci]; L.mqa_status_string.restype = ctypes.c_char_p
        L.mqa_decode_workspace_bytes.argtypes = [ci, ci, ci, ci]; L.mqa_decode_workspace_bytes.restype = sz
        L.mqa_workspace_init.argtypes = [vp, sz, vp]; L.mqa_workspace_init.restype = ci
        L.mqa_decode_plan.argtypes = [ci, ci, ci, ci, ci, ctypes.POINTER(Plan)]; L.mqa_decode_plan.restype = ci
        L.mqa_decode.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, cf, vp, sz, vp]; L.mqa_decode.restype = ci
        L.mqa_decode_with_plan.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, cf, ctypes.POINTER(Plan), vp, sz, vp]
        L.mqa_decode_with_plan.restype = ci
        L.mqa_decode_profiled.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, cf, ctypes.POINTER(Plan), vp, sz, vp, vp]
        L.mqa_decode_profiled.restype = ci
        L.mqa_check_status.argtypes = [vp, vp]; L.mqa_check_status.restype = ci
        L.mqa_decode_host_scratch_bytes.argtypes = [ci, ci, ci, ci]; L.mqa_decode_host_scratch_bytes.restype = sz
        L.mqa_decode_host.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, cf, vp, sz, vp]; L.mqa_decode_host.restype = ci
        L.mqa_last_launch_count.argtypes = []; L.mqa_last_launch_count.restype = ci
        L.mqa_decode_static.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, cf, vp]; L.mqa_decode_static.restype = ci
        L.mqa_append_decode.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, cf, vp, sz, vp]
        L.mqa_append_decode.restype = ci
        L.mqa_decode_grouped.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, vp, sz, vp]
        L.mqa_decode_grouped.restype = ci
        L.mqa_decode_grouped_workspace_bytes.argtypes = [ci, ci, ci, ci, ci]
        L.mqa_decode_grouped_workspace_bytes.restype = sz
        L.mqa_debug_schedule.argtypes = [vp, ci, ci, ci, ci, ci, vp, ci]; L.mqa_debug_schedule.restype = ci
        L.mqa_uniform_ctas.argtypes = [ci, ci, ci]; L.mqa_uniform_ctas.restype = ci
        L.mqa_decode_scatter.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, cf, vp, sz, vp]
        L.mqa_decode_scatter.restype = ci
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().mqa_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != MQA_OK:
        raise MqaError(status, where)


def mqa_decode_workspace_bytes(B: int, H: int, D: int, Lmax: int) -> int:
    return int(lib().mqa_decode_workspace_bytes(B, H, D, Lmax))


def mqa_decode_host_scratch_bytes(B: int, H: int, D: int, Lmax: int) -> int:
    return int(lib().mqa_decode_host_scratch_bytes(B, H, D, Lmax))


def mqa_decode_plan(B: int, H: int, D: int, Lmax: int, path: int = MQA_PATH_AUTO) -> Plan:
    plan = Plan()
    _check(lib().mqa_decode_plan(B, H, D, Lmax, path, ctypes.byref(plan)), "mqa_decode_plan")
    return plan


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def alloc_workspace(B: int, H: int, D: int, Lmax: int, device="cuda", stream=None) -> torch.Tensor:
    """A torch-owned device buffer of the required size with its header initialised."""
    n = mqa_decode_workspace_bytes(B, H, D, Lmax)
    if n == 0:
        raise MqaError(MQA_ERR_UNSUPPORTED_SHAPE, "mqa_decode_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    mqa_workspace_init(ws, stream)
    return ws


def mqa_workspace_init(workspace: torch.Tensor, stream=None):
    _check(lib().mqa_workspace_init(workspace.data_ptr(), workspace.numel(), _stream_ptr(stream)),
           "mqa_workspace_init")


def _shapes(q, k_cache, v_cache, lengths, out):
    B, H, D = q.shape
    Lmax = k_cache.shape[1]
    assert q.dtype == torch.bfloat16 and k_cache.dtype == torch.bfloat16 and v_cache.dtype == torch.bfloat16
    assert lengths.dtype == torch.int32 and out.dtype == torch.float32
    assert k_cache.shape == (B, Lmax, D) and v_cache.shape == (B, Lmax, D)
    assert lengths.shape == (B,) and out.shape == (B, H, D)
    for t in (q, k_cache, v_cache, lengths, out):
        assert t.is_contiguous()
    return B, H, D, Lmax


def mqa_decode(q, k_cache, v_cache, lengths, out, scale: float, workspace, stream=None, plan: Plan | None = None):
    """Enqueue one decode-attention step on ``stream`` (device tensors). Returns ``out``."""
    B, H, D, Lmax = _shapes(q, k_cache, v_cache, lengths, out)
    for t in (q, k_cache, v_cache, lengths, out, workspace):
        assert t.is_cuda
    L = lib()
    if plan is None:
        rc = L.mqa_decode(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), lengths.data_ptr(),
                          out.data_ptr(), B, H, D, Lmax, float(scale),
                          workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    else:
        rc = L.mqa_decode_with_plan(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), lengths.data_ptr(),
                                    out.data_ptr(), B, H, D, Lmax, float(scale), ctypes.byref(plan),
                                    workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _check(rc, "mqa_decode")
    return out


def mqa_decode_profiled(q, k_cache, v_cache, lengths, out, scale: float, workspace, event_after_split,
                        stream=None, plan: Plan | None = None):
    """Like mqa_decode, and records ``event_after_split`` (a torch.cuda.Event that has been
    recorded at least once, so its handle exists) between the split and the combine kernel."""
    B, H, D, Lmax = _shapes(q, k_cache, v_cache, lengths, out)
    handle = int(event_after_split.cuda_event)
    if handle == 0:
        raise ValueError("event has no handle yet: record it once before passing it")
    rc = lib().mqa_decode_profiled(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), lengths.data_ptr(),
                                   out.data_ptr(), B, H, D, Lmax, float(scale),
                                   ctypes.byref(plan) if plan is not None else None,
                                   workspace.data_ptr(), workspace.numel(), _stream_ptr(stream), handle)
    _check(rc, "mqa_decode_profiled")
    return out


MQA_STATIC_WORKSPACE_BYTES = 20 << 20


def mqa_decode_static(q, k_cache, v_cache, lengths, out, scale: float, stream=None):
    """mqa_decode for callers that cannot allocate device memory: no workspace argument,
    the scratch is a fixed array inside the library (shapes beyond it are rejected)."""
    B, H, D, Lmax = _shapes(q, k_cache, v_cache, lengths, out)
    for t in (q, k_cache, v_cache, lengths, out):
        assert t.is_cuda
    rc = lib().mqa_decode_static(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), lengths.data_ptr(),
                                 out.data_ptr(), B, H, D, Lmax, float(scale), _stream_ptr(stream))
    _check(rc, "mqa_decode_static")
    return out


def mqa_append_decode(q, k_new, v_new, k_cache, v_cache, lengths, out, scale: float, workspace, stream=None):
    """Append this step's K/V rows to the caches (in place, lengths incremented), then attend."""
    B, H, D, Lmax = _shapes(q, k_cache, v_cache, lengths, out)
    assert k_new.shape == (B, D) and v_new.shape == (B, D)
    assert k_new.dtype == torch.bfloat16 and v_new.dtype == torch.bfloat16
    for t in (q, k_new, v_new, k_cache, v_cache, lengths, out, workspace):
        assert t.is_cuda and t.is_contiguous()
    rc = lib().mqa_append_decode(q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), k_cache.data_ptr(),
                                 v_cache.data_ptr(), lengths.data_ptr(), out.data_ptr(), B, H, D, Lmax,
                                 float(scale), workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _check(rc, "mqa_append_decode")
    return out


def mqa_decode_grouped(q, k_cache, v_cache, lengths, out, scale: float, workspace=None, stream=None):
    """Grouped-query / multihead decode: k_cache, v_cache are [B, KVH, Lmax, D]; q, out are [B, H, D]."""
    B, H, D = q.shape
    KVH, Lmax = k_cache.shape[1], k_cache.shape[2]
    assert k_cache.shape == (B, KVH, Lmax, D) and v_cache.shape == k_cache.shape
    assert lengths.shape == (B,) and out.shape == (B, H, D)
    for t in (q, k_cache, v_cache, lengths, out):
        assert t.is_cuda and t.is_contiguous()
    if workspace is None:
        n = int(lib().mqa_decode_grouped_workspace_bytes(B, H, KVH, D, Lmax))
        if n == 0:
            raise MqaError(MQA_ERR_UNSUPPORTED_SHAPE, "mqa_decode_grouped_workspace_bytes")
        workspace = torch.empty(n, dtype=torch.uint8, device=q.device)
        mqa_workspace_init(workspace, stream)
    rc = lib().mqa_decode_grouped(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), lengths.data_ptr(),
                                  out.data_ptr(), B, H, KVH, D, Lmax, float(scale),
                                  workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _check(rc, "mqa_decode_grouped")
    return out, workspace


def mqa_check_status(workspace, stream=None) -> int:
    return int(lib().mqa_check_status(workspace.data_ptr(), _stream_ptr(stream)))


def mqa_decode_host(q, k_cache, v_cache, lengths, out, scale: float, scratch, stream=None):
    """Host tensors in, host tensor out; ``scratch`` is a device byte buffer."""
    B, H, D, Lmax = _shapes(q, k_cache, v_cache, lengths, out)
    for t in (q, k_cache, v_cache, lengths, out):
        assert not t.is_cuda
    assert scratch.is_cuda
    rc = lib().mqa_decode_host(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), lengths.data_ptr(),
                               out.data_ptr(), B, H, D, Lmax, float(scale),
                               scratch.data_ptr(), scratch.numel(), _stream_ptr(stream))
    _check(rc, "mqa_decode_host")
    return out


def mqa_last_launch_count() -> int:
    return int(lib().mqa_last_launch_count())


def mqa_decode_scatter(q, k_cache, v_cache, lengths, out_dst, b_offset: int, scale: float, workspace, stream=None):
    """One rank's batch-sharded decode attention with the output scattered by head group.

    ``out_dst``: list of n_dst fp32 CUDA tensors [B_total, H/n_dst, D] (this GPU's or peers' memory), or a list of
    (device pointer, B_total) pairs for memory that is not wrapped in a tensor.  Returns None."""
    assert q.is_cuda and q.dtype == torch.bfloat16 and q.dim() == 3
    B, H, D = q.shape
    Lmax = k_cache.shape[1]
    n_dst = len(out_dst)
    ptrs, totals = [], []
    for t in out_dst:
        if isinstance(t, torch.Tensor):
            assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and t.shape[1:] == (H // n_dst, D)
            ptrs.append(t.data_ptr()); totals.append(t.shape[0])
        else:
            ptrs.append(int(t[0])); totals.append(int(t[1]))
    assert len(set(totals)) == 1, "all destinations hold the same number of rows"
    arr = (ctypes.c_void_p * n_dst)(*ptrs)
    rc = lib().mqa_decode_scatter(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), lengths.data_ptr(),
                                  arr, n_dst, int(b_offset), totals[0], B, H, D, Lmax, float(scale),
                                  workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _check(rc, "mqa_decode_scatter")


def mqa_uniform_ctas(B: int, tiles_per_sequence: int, num_ctas: int) -> int:
    """Block count an adaptive plan uses for a batch of B sequences of equal tile count (host-only)."""
    n = lib().mqa_uniform_ctas(B, tiles_per_sequence, num_ctas)
    if n < 0:
        raise MqaError(-n, "mqa_uniform_ctas")
    return n


def mqa_debug_schedule(lengths, Lmax: int, tile_rows: int, num_ctas: int, cta: int, max_segments: int = 4096):
    """Host replay of the tile schedule of one block: list of
    (b, t0, t1, whole, slot, owns_first, last_cta) tuples. ``lengths`` is a CPU int32 tensor."""
    assert not lengths.is_cuda and lengths.dtype == torch.int32 and lengths.is_contiguous()
    rec = torch.zeros((max_segments, 7), dtype=torch.int32)
    n = lib().mqa_debug_schedule(lengths.data_ptr(), lengths.numel(), Lmax, tile_rows, num_ctas, cta,
                                 rec.data_ptr(), max_segments)
    if n < 0:
        raise MqaError(-n, "mqa_debug_schedule")
    assert n <= max_segments
    return [tuple(int(x) for x in rec[i]) for i in range(n)]
