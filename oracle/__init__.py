"""CPU oracle for the lightning-indexer hot path -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU legs may import this
package; the CUDA library and its Python binding never do. The arithmetic
lives in ``indexer_oracle.cpp`` (FP64, OpenMP over rows) and ``schedule.py``
(the Full/Shared loop); this file compiles the C++ once with g++ and wraps it
with ctypes over NumPy arrays.

Array conventions (all NumPy, C-contiguous):
  bf16 data   -> ``uint16`` arrays holding the raw bit patterns
  e4m3 data   -> ``uint8``  arrays holding the raw codes, plus fp32 per-token scales
  w, scales   -> ``float32``
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "indexer_oracle.cpp"
_LIB = _HERE / "liboracle.so"

BF16 = 0
FP8_E4M3 = 1


def build(force: bool = False) -> Path:
    """Compile the oracle shared library next to its source (g++ -O2 -fopenmp)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.run(
            ["g++", "-O2", "-fopenmp", "-std=c++17", "-shared", "-fPIC", "-o", str(tmp), str(_SRC)],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        lib.orc_threads.restype = ctypes.c_int
        lib.orc_bf16_to_f64.restype = ctypes.c_double
        lib.orc_bf16_to_f64.argtypes = [ctypes.c_uint16]
        lib.orc_e4m3_to_f64.restype = ctypes.c_double
        lib.orc_e4m3_to_f64.argtypes = [ctypes.c_uint8]
        lib.orc_f32_to_bf16.restype = ctypes.c_uint16
        lib.orc_f32_to_bf16.argtypes = [ctypes.c_float]
        lib.orc_f32_to_e4m3.restype = ctypes.c_uint8
        lib.orc_f32_to_e4m3.argtypes = [ctypes.c_float]
        vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        lib.orc_topk.restype = ctypes.c_int
        lib.orc_topk.argtypes = [vp, i64, i32, vp]
        lib.orc_prefill.restype = ctypes.c_int
        lib.orc_prefill.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i32, i32, i32, i32, vp, i64, vp, i64, vp]
        lib.orc_quantize_e4m3.restype = ctypes.c_int
        lib.orc_quantize_e4m3.argtypes = [vp, i64, i64, vp, vp]
        lib.orc_decode.restype = ctypes.c_int
        lib.orc_decode.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, i64, vp]
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().orc_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(a, dtype, name):
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if a.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {a.dtype}")
    return a


def _data_dtype(dtype):
    return np.uint16 if dtype == BF16 else np.uint8


def bf16_to_f64(bits) -> float:
    return float(_load().orc_bf16_to_f64(int(bits)))


def e4m3_to_f64(code) -> float:
    return float(_load().orc_e4m3_to_f64(int(code)))


def f32_to_bf16(x) -> int:
    return int(_load().orc_f32_to_bf16(float(x)))


def f32_to_e4m3(x) -> int:
    return int(_load().orc_f32_to_e4m3(float(x)))


def topk(scores, k_top: int) -> np.ndarray:
    """Top-k of one score row (Sec. 3 'Notation'): ascending indices, -1 padded."""
    s = _check(scores, np.float64, "scores")
    out = np.empty(k_top, dtype=np.int32)
    rc = _load().orc_topk(_ptr(s), s.shape[0], k_top, _ptr(out))
    if rc:
        raise ValueError("orc_topk: bad arguments")
    return out


def indexer_prefill(q, k, w, k_top, dtype=BF16, q_scale=None, k_scale=None, q_begin=0, rows=None,
                    want_scores=True, want_topk=True):
    """Indexer scores + causal top-k for prefill rows.

    q [q_len,H,d], k [L_k,d] raw codes; w [q_len,H] fp32. ``rows``: local row
    indices into q to evaluate (default all). Returns (scores [n,L_k] float64
    with -inf where s > t, topk [n,k_top] int32), either possibly None.
    """
    dd = _data_dtype(dtype)
    q = _check(q, dd, "q")
    k = _check(k, dd, "k")
    w = _check(w, np.float32, "w")
    q_scale = _check(q_scale, np.float32, "q_scale")
    k_scale = _check(k_scale, np.float32, "k_scale")
    q_len, H, d = q.shape
    L_k = k.shape[0]
    assert k.shape[1] == d and w.shape == (q_len, H)
    rows_a = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n = q_len if rows_a is None else rows_a.shape[0]
    scores = np.empty((n, L_k), dtype=np.float64) if want_scores else None
    tk = np.empty((n, k_top), dtype=np.int32) if want_topk else None
    rc = _load().orc_prefill(_ptr(q), _ptr(k), _ptr(w), _ptr(q_scale), _ptr(k_scale), q_begin, q_len, L_k,
                             H, d, k_top, dtype, _ptr(rows_a), n, _ptr(scores), L_k, _ptr(tk))
    if rc:
        raise ValueError("orc_prefill: bad arguments")
    return scores, tk


def indexer_decode(q_step, k_cache, w, k_offsets, lens, k_top, dtype=BF16, q_scale=None, k_scale=None,
                   want_scores=True, want_topk=True):
    """One decode step (Sec. 4.2 'Decode'). q_step [B,H,d], k_cache [rows,d] raw
    codes, w [B,H]; sequence b owns cache rows k_offsets[b] .. +lens[b]-1.
    Returns (scores [B,max(lens)] float64 with -inf padding, topk [B,k_top])."""
    dd = _data_dtype(dtype)
    q_step = _check(q_step, dd, "q_step")
    k_cache = _check(k_cache, dd, "k_cache")
    w = _check(w, np.float32, "w")
    q_scale = _check(q_scale, np.float32, "q_scale")
    k_scale = _check(k_scale, np.float32, "k_scale")
    k_offsets = np.ascontiguousarray(k_offsets, dtype=np.int64)
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    B, H, d = q_step.shape
    assert k_cache.shape[1] == d and w.shape == (B, H)
    assert int((k_offsets + lens).max(initial=0)) <= k_cache.shape[0]
    ld = int(lens.max(initial=0))
    scores = np.empty((B, ld), dtype=np.float64) if want_scores else None
    tk = np.empty((B, k_top), dtype=np.int32) if want_topk else None
    rc = _load().orc_decode(_ptr(q_step), _ptr(k_cache), _ptr(w), _ptr(q_scale), _ptr(k_scale),
                            _ptr(k_offsets), _ptr(lens), B, H, d, k_top, dtype, _ptr(scores), ld, _ptr(tk))
    if rc:
        raise ValueError("orc_decode: bad arguments")
    return scores, tk


def quantize_e4m3(x_bf16):
    """Per-token e4m3 quantiser (Sec. 2.1, 'FP8 arithmetic'): x [n_tokens, ...] bf16 codes (uint16).
    Returns (codes uint8 of the same shape, scale [n_tokens] fp32): scale = max(amax, 1e-12) / 448,
    code = e4m3(x / scale), round to nearest even, saturating; all in binary32."""
    x = _check(x_bf16, np.uint16, "x")
    n = x.shape[0]
    row = int(np.prod(x.shape[1:])) if x.ndim > 1 else 1
    codes = np.empty(x.shape, dtype=np.uint8)
    scale = np.empty((n,), dtype=np.float32)
    rc = _load().orc_quantize_e4m3(_ptr(x), n, row, _ptr(codes), _ptr(scale))
    if rc:
        raise ValueError("orc_quantize_e4m3: bad arguments")
    return codes, scale
