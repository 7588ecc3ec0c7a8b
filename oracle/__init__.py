"""CPU oracle of the mixed paged-attention step. TEST INFRASTRUCTURE ONLY.

The arithmetic lives in ``ts_oracle.c`` (plain C, fp32, one (token, head) at a time); this
module compiles it with gcc on first use and marshals numpy arrays into it. Only the tests,
the smoke check and the benchmark's CPU-baseline leg may import this package. It imports
nothing from the CUDA package and the CUDA package imports nothing from here.

bf16 tensors are carried as ``numpy.uint16`` bit patterns everywhere.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ts_oracle.c")
_BUILD_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_BUILD_DIR, "libts_oracle.so")
_lock = threading.Lock()
_lib = None
_lib_override = None  # set by use_library(): lets the tests run the pins against a mutated build


def build(force: bool = False) -> str:
    """Compile ts_oracle.c into a shared object next to it (gcc -O2 -fopenmp)."""
    os.makedirs(_BUILD_DIR, exist_ok=True)
    stale = (not os.path.exists(_LIB_PATH)) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB_PATH + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def use_library(path):
    """Point the module at another build of the oracle (``None`` restores the default).

    Exists for the tests that plant a mistake in a copy of ts_oracle.c and check that the pins
    notice it."""
    global _lib, _lib_override
    with _lock:
        _lib = None
        _lib_override = path


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(_lib_override or build())
            i32p = ctypes.POINTER(ctypes.c_int32)
            u16p = ctypes.POINTER(ctypes.c_uint16)
            f32p = ctypes.POINTER(ctypes.c_float)
            lib.oracle_kv_append.restype = None
            lib.oracle_kv_append.argtypes = [u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_int, i32p, ctypes.c_int, i32p, i32p, u16p, u16p]
            lib.oracle_attention.restype = ctypes.c_int
            lib.oracle_attention.argtypes = [u16p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_int, ctypes.c_float, ctypes.c_int, i32p,
                                             ctypes.c_int, i32p, i32p, u16p, ctypes.c_int, i32p,
                                             f32p, f32p, ctypes.c_int]
            lib.oracle_default_threads.restype = ctypes.c_int
            lib.oracle_default_threads.argtypes = []
            _lib = lib
    return _lib


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _u16(a) -> np.ndarray:
    a = np.asarray(a)
    if a.dtype != np.uint16:
        raise TypeError("bf16 data must be passed as uint16 bit patterns")
    return np.ascontiguousarray(a)


def default_threads() -> int:
    """Threads the oracle uses when ``threads=0``: the OpenMP default, capped by the affinity mask."""
    n = _load().oracle_default_threads()
    try:
        n = min(n, len(os.sched_getaffinity(0)))
    except AttributeError:
        pass
    return max(1, n)


def pool_elems(n_pages: int, Hkv: int, P: int, D: int) -> int:
    return n_pages * 2 * Hkv * P * D


def kv_append(pool: np.ndarray, Hkv: int, D: int, P: int, tables: np.ndarray, ctx_len, q_len,
              k_new: np.ndarray, v_new: np.ndarray) -> None:
    """In-place append of the step's new K/V into ``pool`` (flat uint16). Sec. 2.1.

    ``tables`` is an int32 array [n_rows, width] of page ids (row r = block table of row r).
    """
    lib = _load()
    if pool.dtype != np.uint16 or not pool.flags.c_contiguous or not pool.flags.writeable:
        raise TypeError("pool must be a writable contiguous uint16 array")
    tables = _i32(tables)
    ctx_len, q_len = _i32(ctx_len), _i32(q_len)
    k_new, v_new = _u16(k_new), _u16(v_new)
    n_rows = len(q_len)
    N = int(q_len.sum())
    assert tables.ndim == 2 and tables.shape[0] == n_rows
    assert k_new.size == N * Hkv * D and v_new.size == N * Hkv * D
    need = (ctx_len + q_len + P - 1) // P
    assert (need <= tables.shape[1]).all(), "block table too narrow"
    lib.oracle_kv_append(_ptr(pool, ctypes.c_uint16), Hkv, D, P, n_rows, _ptr(tables, ctypes.c_int32),
                         tables.shape[1], _ptr(ctx_len, ctypes.c_int32), _ptr(q_len, ctypes.c_int32),
                         _ptr(k_new, ctypes.c_uint16), _ptr(v_new, ctypes.c_uint16))


def attention(pool: np.ndarray, Hq: int, Hkv: int, D: int, P: int, scale: float, tables, ctx_len,
              q_len, q: np.ndarray, sel=None, threads: int = 0, return_weight_sum: bool = False):
    """Causal GQA attention of every (or the selected) new token against the paged pool.

    The pool must already hold the step's appended K/V. Returns fp32 [n_out, Hq, D]
    (and the softmax weight sums [n_out, Hq] when asked).
    """
    lib = _load()
    pool = _u16(pool)
    tables = _i32(tables)
    ctx_len, q_len = _i32(ctx_len), _i32(q_len)
    q = _u16(q)
    n_rows = len(q_len)
    N = int(q_len.sum())
    assert tables.ndim == 2 and tables.shape[0] == n_rows
    assert q.size == N * Hq * D
    if sel is not None:
        sel = _i32(sel)
        n_out = len(sel)
    else:
        n_out = N
    out = np.zeros((n_out, Hq, D), dtype=np.float32)
    ws = np.zeros((n_out, Hq), dtype=np.float32) if return_weight_sum else None
    if n_out:
        rc = lib.oracle_attention(
            _ptr(pool, ctypes.c_uint16), Hq, Hkv, D, P, float(scale), n_rows,
            _ptr(tables, ctypes.c_int32), tables.shape[1], _ptr(ctx_len, ctypes.c_int32),
            _ptr(q_len, ctypes.c_int32), _ptr(q, ctypes.c_uint16), n_out if sel is not None else 0,
            _ptr(sel, ctypes.c_int32) if sel is not None else None, _ptr(out, ctypes.c_float),
            _ptr(ws, ctypes.c_float) if ws is not None else None,
            threads if threads > 0 else default_threads())
        if rc != 0:
            raise RuntimeError("oracle_attention failed")
    return (out, ws) if return_weight_sum else out


def mixed_step(pool: np.ndarray, Hq: int, Hkv: int, D: int, P: int, scale: float, tables, ctx_len,
               q_len, q, k_new, v_new, sel=None, threads: int = 0):
    """One decoder iteration: append the new K/V into ``pool`` (in place), then attend."""
    kv_append(pool, Hkv, D, P, tables, ctx_len, q_len, k_new, v_new)
    return attention(pool, Hq, Hkv, D, P, scale, tables, ctx_len, q_len, q, sel=sel, threads=threads)
