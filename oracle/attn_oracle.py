"""ctypes loader for the double-precision CPU attention oracle (``attn_oracle.c``).

TEST INFRASTRUCTURE, not part of the product: only tests, the smoke check and the
benchmark's CPU-baseline leg may import this.  It shares nothing with the CUDA
library.  Inputs are BF16 bit patterns as ``numpy.uint16`` arrays in the layouts
Q ``[B, Sq, Hq, D]``, K/V ``[B, Sk, Hkv, D]``; outputs are float64.

The arithmetic is the definition in the paper's Section 2.2 ("Attention
computation"), written out in ``attn_oracle.c``; this file only marshals arguments.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_oracle.c")
_LIB = os.path.join(_HERE, "libattn_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile ``attn_oracle.c`` with gcc into ``libattn_oracle.so`` beside it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            u16p = ctypes.POINTER(ctypes.c_uint16)
            i32p = ctypes.POINTER(ctypes.c_int32)
            f64p = ctypes.POINTER(ctypes.c_double)
            i64 = ctypes.c_int64
            shape = [i64] * 6
            lib.attn_oracle_rows.argtypes = [u16p, u16p, u16p, *shape, ctypes.c_int, ctypes.c_float,
                                             i32p, i64, f64p, f64p, ctypes.c_int]
            lib.attn_oracle_rows.restype = ctypes.c_int
            lib.attn_oracle_full.argtypes = [u16p, u16p, u16p, *shape, ctypes.c_int, ctypes.c_float,
                                             f64p, f64p, ctypes.c_int]
            lib.attn_oracle_full.restype = ctypes.c_int
            lib.attn_oracle_weights.argtypes = [u16p, u16p, u16p, *shape, ctypes.c_int, ctypes.c_float,
                                                i64, i64, i64, f64p]
            lib.attn_oracle_weights.restype = ctypes.c_int
            f32p = ctypes.POINTER(ctypes.c_float)
            lib.attn_oracle_merge.argtypes = [u16p, f32p, u16p, f32p, i64, i64, f64p, f64p]
            lib.attn_oracle_merge.restype = ctypes.c_int
            lib.attn_oracle_merge_n.argtypes = [u16p, f32p, i64, i64, i64, f64p, f64p]
            lib.attn_oracle_merge_n.restype = ctypes.c_int
            _lib = lib
    return _lib


def default_threads() -> int:
    return len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)


def _prep(q, k, v):
    q = np.ascontiguousarray(q, dtype=np.uint16)
    k = np.ascontiguousarray(k, dtype=np.uint16)
    v = np.ascontiguousarray(v, dtype=np.uint16)
    if q.ndim != 4 or k.ndim != 4 or v.ndim != 4:
        raise ValueError("q, k, v must be 4-D [B, S, H, D] uint16 (BF16 bits)")
    B, Sq, Hq, D = q.shape
    Bk, Sk, Hkv, Dk = k.shape
    if v.shape != k.shape or Bk != B or Dk != D:
        raise ValueError("inconsistent q/k/v shapes")
    return q, k, v, (B, Hq, Hkv, Sq, Sk, D)


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def attention_full(q, k, v, causal: bool, scale: float, threads: int | None = None):
    """All rows.  Returns (O float64 [B,Sq,Hq,D], LSE float64 [B,Hq,Sq])."""
    q, k, v, (B, Hq, Hkv, Sq, Sk, D) = _prep(q, k, v)
    o = np.empty((B, Sq, Hq, D), dtype=np.float64)
    lse = np.empty((B, Hq, Sq), dtype=np.float64)
    rc = _load().attn_oracle_full(_p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16), _p(v, ctypes.c_uint16),
                                  B, Hq, Hkv, Sq, Sk, D, int(bool(causal)), float(scale),
                                  _p(o, ctypes.c_double), _p(lse, ctypes.c_double),
                                  threads or default_threads())
    if rc != 0:
        raise ValueError(f"attn_oracle_full failed with code {rc}")
    return o, lse


def attention_rows(q, k, v, causal: bool, scale: float, rows, threads: int | None = None):
    """Selected rows.  ``rows``: int array [n, 3] of (b, hq, i).
    Returns (O float64 [n, D], LSE float64 [n])."""
    q, k, v, (B, Hq, Hkv, Sq, Sk, D) = _prep(q, k, v)
    rows = np.ascontiguousarray(rows, dtype=np.int32).reshape(-1, 3)
    n = rows.shape[0]
    o = np.empty((n, D), dtype=np.float64)
    lse = np.empty((n,), dtype=np.float64)
    rc = _load().attn_oracle_rows(_p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16), _p(v, ctypes.c_uint16),
                                  B, Hq, Hkv, Sq, Sk, D, int(bool(causal)), float(scale),
                                  _p(rows, ctypes.c_int32), n,
                                  _p(o, ctypes.c_double), _p(lse, ctypes.c_double),
                                  threads or default_threads())
    if rc != 0:
        raise ValueError(f"attn_oracle_rows failed with code {rc}")
    return o, lse


def softmax_weights(q, k, v, causal: bool, scale: float, b: int, hq: int, i: int):
    """Normalised weights p_j (float64 [Sk], zero where masked) of one query row."""
    q, k, v, (B, Hq, Hkv, Sq, Sk, D) = _prep(q, k, v)
    p = np.empty((Sk,), dtype=np.float64)
    rc = _load().attn_oracle_weights(_p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16), _p(v, ctypes.c_uint16),
                                     B, Hq, Hkv, Sq, Sk, D, int(bool(causal)), float(scale),
                                     b, hq, i, _p(p, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"attn_oracle_weights failed with code {rc}")
    return p


def merge(o1, lse1, o2, lse2):
    """LSE-weighted merge of two partial results over disjoint key sets.
    o1, o2: uint16 BF16 bits [..., D]; lse1, lse2: float32 [...] with one entry per row of o
    (same row order).  Returns (O float64 [..., D], LSE float64 [...])."""
    o1 = np.ascontiguousarray(o1, dtype=np.uint16)
    o2 = np.ascontiguousarray(o2, dtype=np.uint16)
    lse1 = np.ascontiguousarray(lse1, dtype=np.float32)
    lse2 = np.ascontiguousarray(lse2, dtype=np.float32)
    D = o1.shape[-1]
    rows = o1.size // D
    if o2.shape != o1.shape or lse1.size != rows or lse2.size != rows:
        raise ValueError("inconsistent shapes")
    o = np.empty(o1.shape, dtype=np.float64)
    lse = np.empty(lse1.shape, dtype=np.float64)
    rc = _load().attn_oracle_merge(_p(o1, ctypes.c_uint16), _p(lse1, ctypes.c_float), _p(o2, ctypes.c_uint16),
                                   _p(lse2, ctypes.c_float), rows, D, _p(o, ctypes.c_double),
                                   _p(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"attn_oracle_merge failed with code {rc}")
    return o, lse


def merge_n(o_parts, lse_parts):
    """LSE-weighted merge of n partial results over pairwise disjoint key sets.
    o_parts: uint16 BF16 bits [n, ..., D]; lse_parts: float32 [n, ...] with one entry per row of a
    part (same row order).  Returns (O float64 [..., D], LSE float64 [...])."""
    o_parts = np.ascontiguousarray(o_parts, dtype=np.uint16)
    lse_parts = np.ascontiguousarray(lse_parts, dtype=np.float32)
    n, D = o_parts.shape[0], o_parts.shape[-1]
    rows = o_parts[0].size // D
    if lse_parts.shape[0] != n or lse_parts[0].size != rows:
        raise ValueError("inconsistent shapes")
    o = np.empty(o_parts.shape[1:], dtype=np.float64)
    lse = np.empty(lse_parts.shape[1:], dtype=np.float64)
    rc = _load().attn_oracle_merge_n(_p(o_parts, ctypes.c_uint16), _p(lse_parts, ctypes.c_float), n, rows, D,
                                     _p(o, ctypes.c_double), _p(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"attn_oracle_merge_n failed with code {rc}")
    return o, lse
