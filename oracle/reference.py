"""TEST INFRASTRUCTURE — ctypes front end of the fp64 C oracle (wpp_oracle.c).

Inputs are CPU tensors/arrays holding bf16 bit patterns (torch.bfloat16 or
numpy uint16).  Outputs are numpy float64.  Nothing here touches CUDA.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wpp_oracle.c")
_LIB = os.path.join(_HERE, "libwpp_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile wpp_oracle.c with gcc (no fast-math, so summation order is as written)."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-shared", "-fPIC",
                                   "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        p = ctypes.c_void_p
        i32 = ctypes.c_int32
        lib.wpp_oracle_threads.restype = ctypes.c_int
        lib.wpp_oracle_append.restype = ctypes.c_int
        lib.wpp_oracle_append.argtypes = [p, p, p, p, p, p, p, i32, i32, i32, i32, i32, i32]
        lib.wpp_oracle_attention.restype = ctypes.c_int
        lib.wpp_oracle_attention.argtypes = [p, p, p, p, p, p, i32, i32, i32, i32, i32, i32,
                                             ctypes.c_double, p, p]
        lib.wpp_oracle_attention_units.restype = ctypes.c_int
        lib.wpp_oracle_attention_units.argtypes = [p, p, p, p, p, p, i32, i32, i32, i32, i32, i32,
                                                   ctypes.c_double, p, ctypes.c_int64, p, p, p]
        _lib = lib
    return _lib


def oracle_threads() -> int:
    return int(_load().wpp_oracle_threads())


def _bits(x) -> np.ndarray:
    """bf16 tensor or uint16 array -> C-contiguous numpy uint16 (shares memory when it can)."""
    if isinstance(x, np.ndarray):
        assert x.dtype == np.uint16
        return np.ascontiguousarray(x)
    import torch
    assert x.dtype == torch.bfloat16 and x.device.type == "cpu"
    return x.contiguous().view(torch.int16).numpy().view(np.uint16)


def _i32(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def oracle_append(k_new, v_new, k_pool, v_pool, block_tables, prefix_lens, chunk_lens):
    """Return copies (numpy uint16) of the pools with the chunk's K/V written into their pages.

    pools [num_pages, Hkv, B, d]; k_new/v_new [T, Hkv, d]; bit patterns are copied untouched.
    """
    kp = _bits(k_pool).copy()
    vp = _bits(v_pool).copy()
    kn, vn = _bits(k_new), _bits(v_new)
    bt, P, C = _i32(block_tables), _i32(prefix_lens), _i32(chunk_lens)
    num_pages, Hkv, B, d = kp.shape
    assert kn.shape == (int(C.sum()), Hkv, d) and vn.shape == kn.shape and vp.shape == kp.shape
    rc = _load().wpp_oracle_append(_ptr(kn), _ptr(vn), _ptr(kp), _ptr(vp), _ptr(bt), _ptr(P), _ptr(C),
                                   P.shape[0], Hkv, d, B, bt.shape[1], num_pages)
    if rc != 0:
        raise ValueError("oracle_append: block table entry out of range")
    return kp, vp


def _scale(d, sm_scale):
    return 1.0 / math.sqrt(float(d)) if not sm_scale else float(sm_scale)


def oracle_attention(q, k_pool, v_pool, block_tables, prefix_lens, chunk_lens, sm_scale=None):
    """All rows: returns (out float64 [T, Hq, d], lse float64 [T, Hq]).  Pools are the post-append pools."""
    qb, kp, vp = _bits(q), _bits(k_pool), _bits(v_pool)
    bt, P, C = _i32(block_tables), _i32(prefix_lens), _i32(chunk_lens)
    T, Hq, d = qb.shape
    _, Hkv, B, _ = kp.shape
    assert T == int(C.sum())
    out = np.empty((T, Hq, d), dtype=np.float64)
    lse = np.empty((T, Hq), dtype=np.float64)
    rc = _load().wpp_oracle_attention(_ptr(qb), _ptr(kp), _ptr(vp), _ptr(bt), _ptr(P), _ptr(C), P.shape[0],
                                      Hq, Hkv, d, B, bt.shape[1], _scale(d, sm_scale), _ptr(out), _ptr(lse))
    if rc != 0:
        raise ValueError(f"oracle_attention failed ({rc})")
    return out, lse


def oracle_attention_units(q, k_pool, v_pool, block_tables, prefix_lens, chunk_lens, units, sm_scale=None,
                           return_top2=False):
    """Selected (request, chunk row, query head) triples: returns (out [n, d], lse [n]) and, if asked, the
    largest and second largest score of each row [n, 2] (how well conditioned the row's softmax is)."""
    qb, kp, vp = _bits(q), _bits(k_pool), _bits(v_pool)
    bt, P, C = _i32(block_tables), _i32(prefix_lens), _i32(chunk_lens)
    units = _i32(units).reshape(-1, 3)
    T, Hq, d = qb.shape
    _, Hkv, B, _ = kp.shape
    n = units.shape[0]
    out = np.empty((n, d), dtype=np.float64)
    lse = np.empty((n,), dtype=np.float64)
    top2 = np.empty((n, 2), dtype=np.float64) if return_top2 else None
    rc = _load().wpp_oracle_attention_units(_ptr(qb), _ptr(kp), _ptr(vp), _ptr(bt), _ptr(P), _ptr(C),
                                            P.shape[0], Hq, Hkv, d, B, bt.shape[1], _scale(d, sm_scale),
                                            _ptr(units), n, _ptr(out), _ptr(lse),
                                            _ptr(top2) if return_top2 else None)
    if rc != 0:
        raise ValueError(f"oracle_attention_units failed ({rc})")
    return (out, lse, top2) if return_top2 else (out, lse)


def merge_partials(outs, lses):
    """Merge attention results computed over disjoint key sets (the split-KV combine, in fp64).

    lse = log sum_s exp(lse_s);  O = sum_s exp(lse_s - lse) O_s.   outs [S, ..., d], lses [S, ...].
    """
    outs = np.asarray(outs, dtype=np.float64)
    lses = np.asarray(lses, dtype=np.float64)
    m = lses.max(axis=0)
    w = np.exp(lses - m)
    lse = m + np.log(w.sum(axis=0))
    o = (w[..., None] * outs).sum(axis=0) / w.sum(axis=0)[..., None]
    return o, lse
