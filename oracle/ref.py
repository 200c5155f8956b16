"""ctypes loader for the fp64 C oracle (``oracle/mqa_ref.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark, never by the product package.  It shares no
code with the CUDA path.  The operation is the multiquery attention of the
paper's Section 3.3 (one shared key/value head for all query heads), for the
single-token generate phase, written as the plain softmax-attention definition
in double precision.

Arrays: ``q`` [B,H,D], ``k``/``v`` [B,Lmax,D] as bf16 bit patterns
(numpy uint16, or torch.bfloat16 CPU tensors), ``lengths`` [B] int32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mqa_ref.c")
_LIB = os.path.join(_HERE, "libmqa_ref.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C11 + OpenMP). Returns the .so path."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-Wall",
           _SRC, "-o", _LIB, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        i32p = ctypes.POINTER(ctypes.c_int32)
        f64p = ctypes.POINTER(ctypes.c_double)
        ci = ctypes.c_int
        lib.mqa_decode_ref_f64.argtypes = [u16p, u16p, u16p, i32p, f64p, ci, ci, ci, ci,
                                           ctypes.c_float, ci]
        lib.mqa_decode_ref_f64.restype = ci
        lib.mqa_ref_weights_f64.argtypes = [u16p, u16p, i32p, f64p, ci, ci, ci, ci,
                                            ctypes.c_float]
        lib.mqa_ref_weights_f64.restype = ci
        lib.mqa_ref_partial_f64.argtypes = [u16p, u16p, u16p, i32p, ci, ci, ci,
                                            f64p, f64p, f64p, ci, ci, ci, ci, ctypes.c_float]
        lib.mqa_ref_partial_f64.restype = ci
        lib.mqa_ref_merge_f64.argtypes = [f64p, f64p, f64p, ci, ci, f64p]
        lib.mqa_ref_merge_f64.restype = ci
        lib.gqa_decode_ref_f64.argtypes = [u16p, u16p, u16p, i32p, f64p, ci, ci, ci, ci, ci, ctypes.c_float]
        lib.gqa_decode_ref_f64.restype = ci
        lib.mqa_ref_max_threads.argtypes = []
        lib.mqa_ref_max_threads.restype = ci
        _lib = lib
    return _lib


def as_bits(x) -> np.ndarray:
    """bf16 bit patterns as a C-contiguous numpy uint16 array (no rounding here)."""
    if isinstance(x, np.ndarray):
        if x.dtype != np.uint16:
            raise TypeError("numpy inputs must already be uint16 bf16 bit patterns")
        return np.ascontiguousarray(x)
    import torch
    if not isinstance(x, torch.Tensor) or x.dtype != torch.bfloat16:
        raise TypeError("expected a torch.bfloat16 tensor or a numpy uint16 array")
    return np.ascontiguousarray(x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16))


def _lens(lengths) -> np.ndarray:
    if not isinstance(lengths, np.ndarray):
        lengths = lengths.detach().cpu().numpy()
    return np.ascontiguousarray(lengths.astype(np.int32, copy=False))


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def max_threads() -> int:
    return int(_load().mqa_ref_max_threads())


def mqa_decode_ref(q, k, v, lengths, scale: float, num_threads: int | None = None) -> np.ndarray:
    """Reference output [B,H,D] in float64."""
    lib = _load()
    qb, kb, vb, ln = as_bits(q), as_bits(k), as_bits(v), _lens(lengths)
    B, H, D = qb.shape
    Lmax = kb.shape[1]
    assert kb.shape == (B, Lmax, D) and vb.shape == (B, Lmax, D) and ln.shape == (B,)
    out = np.empty((B, H, D), dtype=np.float64)
    nt = num_threads if num_threads is not None else (os.cpu_count() or 1)
    rc = lib.mqa_decode_ref_f64(_p(qb, ctypes.c_uint16), _p(kb, ctypes.c_uint16),
                                _p(vb, ctypes.c_uint16), _p(ln, ctypes.c_int32),
                                _p(out, ctypes.c_double), B, H, D, Lmax,
                                ctypes.c_float(scale), int(nt))
    if rc != 0:
        raise RuntimeError("mqa_decode_ref_f64 failed")
    return out


def mqa_ref_weights(q, k, lengths, scale: float) -> np.ndarray:
    """Softmax weights [B,H,Lmax] in float64 (zero at and beyond each length)."""
    lib = _load()
    qb, kb, ln = as_bits(q), as_bits(k), _lens(lengths)
    B, H, D = qb.shape
    Lmax = kb.shape[1]
    w = np.empty((B, H, Lmax), dtype=np.float64)
    rc = lib.mqa_ref_weights_f64(_p(qb, ctypes.c_uint16), _p(kb, ctypes.c_uint16),
                                 _p(ln, ctypes.c_int32), _p(w, ctypes.c_double),
                                 B, H, D, Lmax, ctypes.c_float(scale))
    if rc != 0:
        raise RuntimeError("mqa_ref_weights_f64 failed")
    return w


def mqa_ref_partial(q, k, v, lengths, b: int, l0: int, l1: int, scale: float):
    """(m[H], z[H], acc[H,D]) of rows [l0,l1) of sequence b (natural-log domain)."""
    lib = _load()
    qb, kb, vb, ln = as_bits(q), as_bits(k), as_bits(v), _lens(lengths)
    B, H, D = qb.shape
    Lmax = kb.shape[1]
    m = np.empty(H, dtype=np.float64)
    z = np.empty(H, dtype=np.float64)
    acc = np.empty((H, D), dtype=np.float64)
    rc = lib.mqa_ref_partial_f64(_p(qb, ctypes.c_uint16), _p(kb, ctypes.c_uint16),
                                 _p(vb, ctypes.c_uint16), _p(ln, ctypes.c_int32),
                                 int(b), int(l0), int(l1),
                                 _p(m, ctypes.c_double), _p(z, ctypes.c_double),
                                 _p(acc, ctypes.c_double), B, H, D, Lmax,
                                 ctypes.c_float(scale))
    if rc != 0:
        raise RuntimeError("mqa_ref_partial_f64 failed")
    return m, z, acc


def mqa_ref_merge(m: np.ndarray, z: np.ndarray, acc: np.ndarray) -> np.ndarray:
    """Merge S partials of one (sequence, head): m,z [S], acc [S,D] -> out [D]."""
    lib = _load()
    m = np.ascontiguousarray(m, dtype=np.float64)
    z = np.ascontiguousarray(z, dtype=np.float64)
    acc = np.ascontiguousarray(acc, dtype=np.float64)
    S, D = acc.shape
    out = np.empty(D, dtype=np.float64)
    rc = lib.mqa_ref_merge_f64(_p(m, ctypes.c_double), _p(z, ctypes.c_double),
                               _p(acc, ctypes.c_double), S, D, _p(out, ctypes.c_double))
    if rc != 0:
        raise RuntimeError("mqa_ref_merge_f64 failed")
    return out


def mqa_append_decode_ref(q, k_new, v_new, k, v, lengths, scale: float, num_threads: int | None = None):
    """One generate step of the attention layer: the step's new key/value row of every sequence joins
    its cache (paper Section 2.2: each decode step produces one token per sequence; Section 3.3: that
    step has one token of Q, K and V per sequence against a cache of many), then the query attends over
    the lengthened cache by the plain definition.

    Returns (out[B,H,D] float64, k_bits, v_bits, new_lengths) with the caches as uint16 bf16 bit arrays.
    A sequence whose length is outside [0, Lmax) gets nothing appended and keeps its length.
    """
    qb, kb, vb, ln = as_bits(q), as_bits(k).copy(), as_bits(v).copy(), _lens(lengths).copy()
    knb, vnb = as_bits(k_new), as_bits(v_new)
    B, Lmax, D = kb.shape
    assert knb.shape == (B, D) and vnb.shape == (B, D)
    for b in range(B):
        n = int(ln[b])
        if 0 <= n < Lmax:
            kb[b, n, :] = knb[b]
            vb[b, n, :] = vnb[b]
            ln[b] = n + 1
    out = mqa_decode_ref(qb, kb, vb, ln, scale, num_threads)
    return out, kb, vb, ln


def gqa_decode_ref(q, k, v, lengths, scale: float) -> np.ndarray:
    """Reference for KVH key/value heads per sequence (Section 4.2's multihead / multiquery comparison):
    q [B,H,D], k/v [B,KVH,Lmax,D]; query head h reads key/value head h // (H // KVH). Returns [B,H,D] float64."""
    lib = _load()
    qb, kb, vb, ln = as_bits(q), as_bits(k), as_bits(v), _lens(lengths)
    B, H, D = qb.shape
    KVH, Lmax = kb.shape[1], kb.shape[2]
    assert kb.shape == (B, KVH, Lmax, D) and vb.shape == kb.shape and ln.shape == (B,)
    out = np.empty((B, H, D), dtype=np.float64)
    rc = lib.gqa_decode_ref_f64(_p(qb, ctypes.c_uint16), _p(kb, ctypes.c_uint16), _p(vb, ctypes.c_uint16),
                                _p(ln, ctypes.c_int32), _p(out, ctypes.c_double), B, H, KVH, D, Lmax,
                                ctypes.c_float(scale))
    if rc != 0:
        raise RuntimeError("gqa_decode_ref_f64 failed")
    return out
