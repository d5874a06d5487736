"""ctypes front end of ``oracle.c`` (test infrastructure; see that file's header).

Arrays cross as numpy: bf16 inputs are uint16 bit patterns, every result is float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

_u16p = ctypes.POINTER(ctypes.c_uint16)
_f64p = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile oracle.c with gcc (strict IEEE: no -ffast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
               "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.oracle_gqa_attention.restype = ctypes.c_int
        lib.oracle_gqa_attention.argtypes = [_u16p, _u16p, _u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_int, ctypes.c_int, ctypes.c_double, _f64p, _f64p]
        lib.oracle_softmax_weights.restype = ctypes.c_int
        lib.oracle_softmax_weights.argtypes = [_u16p, _u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                               ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_int,
                                               ctypes.c_int, _f64p]
        lib.oracle_merge_lse.restype = ctypes.c_int
        lib.oracle_merge_lse.argtypes = [ctypes.c_int, ctypes.c_int, _f64p, _f64p, _f64p, _f64p]
        lib.oracle_xtensor_locate.restype = ctypes.c_int
        lib.oracle_xtensor_locate.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64,
                                              ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64)]
        lib.oracle_gqa_attention_batch.restype = ctypes.c_int
        lib.oracle_gqa_attention_batch.argtypes = [
            ctypes.c_int, ctypes.POINTER(_u16p), ctypes.POINTER(_u16p), ctypes.POINTER(_u16p),
            ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32), ctypes.c_int, ctypes.c_int,
            ctypes.c_int, ctypes.c_double, ctypes.POINTER(_f64p), ctypes.POINTER(_f64p), ctypes.c_int]
        _lib = lib
    return _lib


def _u16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("bf16 inputs must be uint16 bit patterns")
    return a


def _check_shapes(q, k, v):
    if q.ndim != 3 or k.ndim != 3 or v.shape != k.shape or q.shape[2] != k.shape[2]:
        raise ValueError("expected q [q_len,H_q,D], k/v [kv_len,H_kv,D]")
    return q.shape[0], k.shape[0], q.shape[1], k.shape[1], q.shape[2]


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float) -> Tuple[np.ndarray, np.ndarray]:
    """One request -> (O [q_len,H_q,D] float64, LSE [q_len,H_q] float64, natural log)."""
    q, k, v = _u16(q), _u16(k), _u16(v)
    q_len, kv_len, hq, hkv, d = _check_shapes(q, k, v)
    out = np.empty((q_len, hq, d), np.float64)
    lse = np.empty((q_len, hq), np.float64)
    st = _load().oracle_gqa_attention(q.ctypes.data_as(_u16p), k.ctypes.data_as(_u16p), v.ctypes.data_as(_u16p),
                                      q_len, kv_len, hq, hkv, d, float(scale), out.ctypes.data_as(_f64p),
                                      lse.ctypes.data_as(_f64p))
    if st != 0:
        raise ValueError(f"oracle_gqa_attention rejected the sizes (status {st})")
    return out, lse


def attention_batch(qs: Sequence[np.ndarray], ks: Sequence[np.ndarray], vs: Sequence[np.ndarray], scale: float,
                    n_threads: Optional[int] = None) -> Tuple[List[np.ndarray], List[np.ndarray]]:
    """Many requests over host threads (one request per task, the per-request routine unchanged)."""
    n = len(qs)
    qs = [_u16(a) for a in qs]
    ks = [_u16(a) for a in ks]
    vs = [_u16(a) for a in vs]
    dims = [_check_shapes(q, k, v) for q, k, v in zip(qs, ks, vs)]
    hq, hkv, d = dims[0][2:]
    if any(x[2:] != (hq, hkv, d) for x in dims):
        raise ValueError("all requests must share the head geometry")
    outs = [np.empty((x[0], hq, d), np.float64) for x in dims]
    lses = [np.empty((x[0], hq), np.float64) for x in dims]
    arr_u16 = _u16p * n
    arr_f64 = _f64p * n
    qp = arr_u16(*[a.ctypes.data_as(_u16p) for a in qs])
    kp = arr_u16(*[a.ctypes.data_as(_u16p) for a in ks])
    vp = arr_u16(*[a.ctypes.data_as(_u16p) for a in vs])
    op = arr_f64(*[a.ctypes.data_as(_f64p) for a in outs])
    lp = arr_f64(*[a.ctypes.data_as(_f64p) for a in lses])
    ql = (ctypes.c_int32 * n)(*[x[0] for x in dims])
    kl = (ctypes.c_int32 * n)(*[x[1] for x in dims])
    if n_threads is None:
        n_threads = os.cpu_count() or 1
    st = _load().oracle_gqa_attention_batch(n, qp, kp, vp, ql, kl, hq, hkv, d, float(scale), op, lp, int(n_threads))
    if st != 0:
        raise ValueError(f"oracle_gqa_attention_batch failed (status {st})")
    return outs, lses


def softmax_weights(q: np.ndarray, k: np.ndarray, scale: float, i: int, h: int) -> np.ndarray:
    """Normalised weights of query row i, head h over its visible keys."""
    q, k = _u16(q), _u16(k)
    q_len, kv_len, hq, hkv, d = _check_shapes(q, k, k)
    p = np.empty(kv_len, np.float64)
    n = _load().oracle_softmax_weights(q.ctypes.data_as(_u16p), k.ctypes.data_as(_u16p), q_len, kv_len, hq, hkv, d,
                                       float(scale), int(i), int(h), p.ctypes.data_as(_f64p))
    if n < 0:
        raise ValueError("oracle_softmax_weights rejected the arguments")
    return p[:n].copy()


def merge_lse(o_parts: np.ndarray, lse_parts: np.ndarray) -> Tuple[np.ndarray, float]:
    """Merge partial results of one query row: o_parts [S,D], lse_parts [S] -> (O [D], LSE)."""
    o_parts = np.ascontiguousarray(o_parts, np.float64)
    lse_parts = np.ascontiguousarray(lse_parts, np.float64)
    s, d = o_parts.shape
    o = np.empty(d, np.float64)
    lse = ctypes.c_double(0.0)
    st = _load().oracle_merge_lse(s, d, o_parts.ctypes.data_as(_f64p), lse_parts.ctypes.data_as(_f64p),
                                  o.ctypes.data_as(_f64p), ctypes.byref(lse))
    if st != 0:
        raise ValueError("oracle_merge_lse: no part has a visible key")
    return o, lse.value


def xtensor_locate(virt_addr: int, virt_start: int, page_size: int) -> Tuple[int, int]:
    """Eq. 2 of the xTensor section: (physical page index, offset inside the page)."""
    idx, off = ctypes.c_uint64(0), ctypes.c_uint64(0)
    st = _load().oracle_xtensor_locate(virt_addr, virt_start, page_size, ctypes.byref(idx), ctypes.byref(off))
    if st != 0:
        raise ValueError("address below the range start or zero page size")
    return idx.value, off.value
