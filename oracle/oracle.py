"""ctypes front door of the fp64 CPU oracle (``vosti_oracle.c``).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's
cpu_baseline / reference arm may import this; the product path must not.
It shares nothing with the CUDA library and never imports it.

bf16 tensors cross this boundary as ``numpy.uint16`` bit patterns; results
come back as ``float64``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vosti_oracle.c")
_LIB = os.path.join(_HERE, "libvosti_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, IEEE semantics, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"],
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
            lib.vosti_oracle_num_threads.restype = ctypes.c_int
            lib.vosti_oracle_attention_dense.restype = ctypes.c_int
            lib.vosti_oracle_attention_dense.argtypes = [
                u16p, u16p, u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_int64, f64p, f64p]
            lib.vosti_oracle_paged_attention.restype = ctypes.c_int
            lib.vosti_oracle_paged_attention.argtypes = [
                u16p, u16p, i32p, i32p, i32p, i32p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64, ctypes.c_double,
                ctypes.c_int64, i32p, ctypes.c_int64, f64p, f64p]
            lib.vosti_oracle_kv_append.restype = ctypes.c_int
            lib.vosti_oracle_kv_append.argtypes = [
                u16p, u16p, u16p, i32p, i32p, i32p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                ctypes.c_int, ctypes.c_int, ctypes.c_int64]
            _lib = lib
    return _lib


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _ptr(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def num_threads() -> int:
    return int(_load().vosti_oracle_num_threads())


def attention_dense(q, k, v, start: int, scale: float, window: int = 0, return_lse: bool = False):
    """q [s,Hq,d], k/v [n,Hkv,d] (uint16 bf16 bits) -> float64 [s,Hq,d].

    Row i is at logical position ``start + i`` and sees keys ``0..start+i``, or
    only the last ``window`` of them when ``window > 0``.  With ``return_lse``
    also returns the natural-log log-sum-exp of the scaled scores, [s,Hq].
    """
    q, k, v = _u16(q), _u16(k), _u16(v)
    s, Hq, d = q.shape
    n, Hkv, d2 = k.shape
    assert d == d2 and v.shape == k.shape
    out = np.empty((s, Hq, d), dtype=np.float64)
    lse = np.empty((s, Hq), dtype=np.float64) if return_lse else None
    rc = _load().vosti_oracle_attention_dense(
        _ptr(q, ctypes.c_uint16), _ptr(k, ctypes.c_uint16), _ptr(v, ctypes.c_uint16),
        s, n, int(start), Hq, Hkv, d, float(scale), int(window), _ptr(out, ctypes.c_double),
        _ptr(lse, ctypes.c_double) if return_lse else None)
    if rc:
        raise ValueError(f"oracle attention_dense failed: {rc}")
    return (out, lse) if return_lse else out


def paged_attention(q, pool, q_lens, start_pos, seq_lens, block_tables, *, n_kv_heads: int,
                    page_size: int, scale: float, sel=None, window: int = 0, return_lse: bool = False):
    """Paged front-end.  q [T,Hq,d] uint16; pool uint16 of shape
    [num_pages,Hkv,2,P,d]; block_tables int32 [B,stride].

    ``sel`` = optional int32 [n,3] rows of (request, token, head): only those
    outputs are computed and the result is [n,d]; otherwise [T,Hq,d].
    """
    q, pool = _u16(q), _u16(pool)
    T, Hq, d = q.shape
    num_pages = pool.shape[0]
    assert pool.shape[1:] == (n_kv_heads, 2, page_size, d), pool.shape
    q_lens, start_pos, seq_lens = _i32(q_lens), _i32(start_pos), _i32(seq_lens)
    bt = _i32(block_tables)
    B = q_lens.shape[0]
    assert bt.ndim == 2 and bt.shape[0] == B
    assert int(q_lens.sum()) == T
    if sel is None:
        out = np.empty((T, Hq, d), dtype=np.float64)
        lse = np.empty((T, Hq), dtype=np.float64) if return_lse else None
        selp, nsel = None, 0
    else:
        sel = _i32(sel).reshape(-1, 3)
        out = np.empty((sel.shape[0], d), dtype=np.float64)
        lse = np.empty((sel.shape[0],), dtype=np.float64) if return_lse else None
        selp, nsel = _ptr(sel, ctypes.c_int32), sel.shape[0]
    rc = _load().vosti_oracle_paged_attention(
        _ptr(q, ctypes.c_uint16), _ptr(pool, ctypes.c_uint16), _ptr(q_lens, ctypes.c_int32),
        _ptr(start_pos, ctypes.c_int32), _ptr(seq_lens, ctypes.c_int32),
        _ptr(bt, ctypes.c_int32), bt.shape[1], B, Hq, n_kv_heads, d, page_size, num_pages,
        float(scale), int(window), selp, nsel, _ptr(out, ctypes.c_double),
        _ptr(lse, ctypes.c_double) if return_lse else None)
    if rc:
        raise ValueError(f"oracle paged_attention failed: {rc}")
    return (out, lse) if return_lse else out


def kv_append(pool, k_new, v_new, q_lens, start_pos, block_tables) -> None:
    """Write k_new/v_new [T,Hkv,d] uint16 into ``pool`` (in place)."""
    assert pool.dtype == np.uint16 and pool.flags.c_contiguous and pool.flags.writeable
    k_new, v_new = _u16(k_new), _u16(v_new)
    num_pages, Hkv, two, P, d = pool.shape
    assert two == 2 and k_new.shape[1:] == (Hkv, d) and v_new.shape == k_new.shape
    q_lens, start_pos = _i32(q_lens), _i32(start_pos)
    bt = _i32(block_tables)
    assert int(q_lens.sum()) == k_new.shape[0]
    rc = _load().vosti_oracle_kv_append(
        _ptr(pool, ctypes.c_uint16), _ptr(k_new, ctypes.c_uint16), _ptr(v_new, ctypes.c_uint16),
        _ptr(q_lens, ctypes.c_int32), _ptr(start_pos, ctypes.c_int32), _ptr(bt, ctypes.c_int32),
        bt.shape[1], q_lens.shape[0], Hkv, d, P, num_pages)
    if rc:
        raise ValueError(f"oracle kv_append failed: {rc}")
