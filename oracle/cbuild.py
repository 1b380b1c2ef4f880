"""Build and call the plain-C float64 oracle (test infrastructure only).

`build()` compiles csrc/attend_f64.c with gcc into oracle/_attend_f64.so;
`attend_paged()` marshals a PagedKVOracle batch to it.  Nothing here is
shared with, or imported by, the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csrc", "attend_f64.c")
_SO = os.path.join(_HERE, "_attend_f64.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.tide_oracle_threads.restype = ctypes.c_int
        lib.tide_oracle_attend_f64.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().tide_oracle_threads())


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def attend_paged(cache, rows, q_bits, scale: float, items=None, n_threads: int = 0):
    """cache: PagedKVOracle (with values); rows: list of (task, q_len, ctx_len);
    q_bits uint16 [sum q_len, Hq, D].  items: optional list of (row index, query
    index) to compute; default = every query of every row, in batch order.

    Returns O [n_items, Hq, D] float64 and LSE [n_items, Hq] float64."""
    lib = _load()
    cache.check_rows(rows)
    n_rows = len(rows)
    Hq, D = int(q_bits.shape[1]), int(q_bits.shape[2])
    qlen = np.asarray([r[1] for r in rows], dtype=np.int32)
    ctx = np.asarray([r[2] for r in rows], dtype=np.int32)
    qoff = np.zeros(n_rows, dtype=np.int64)
    if n_rows:
        qoff[1:] = np.cumsum(qlen[:-1])
    max_pages = max([(int(c) + cache.S - 1) // cache.S for c in ctx] + [1])
    tables = np.full((max(n_rows, 1), max_pages), -1, dtype=np.int32)
    for b, (task, _, L) in enumerate(rows):
        npg = (int(L) + cache.S - 1) // cache.S
        tables[b, :npg] = cache.pages[int(task)][:npg]
    if items is None:
        item_row = np.repeat(np.arange(n_rows, dtype=np.int32), qlen)
        item_q = np.concatenate([np.arange(n, dtype=np.int32) for n in qlen]) if n_rows else np.zeros(0, np.int32)
    else:
        item_row = np.asarray([it[0] for it in items], dtype=np.int32)
        item_q = np.asarray([it[1] for it in items], dtype=np.int32)
    n_items = int(item_row.shape[0])
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint16)
    out = np.empty((n_items, Hq, D), dtype=np.float64)
    lse = np.empty((n_items, Hq), dtype=np.float64)
    rc = lib.tide_oracle_attend_f64(
        _ptr(cache.pool_k), _ptr(cache.pool_v), ctypes.c_int64(cache.P),
        ctypes.c_int(cache.S), ctypes.c_int(cache.Hkv), ctypes.c_int(D), ctypes.c_int(Hq),
        _ptr(tables), ctypes.c_int(max_pages), ctypes.c_int(n_rows),
        _ptr(qlen), _ptr(ctx), _ptr(qoff), _ptr(q_bits), ctypes.c_double(scale),
        ctypes.c_int64(n_items), _ptr(item_row), _ptr(item_q), _ptr(out), _ptr(lse), ctypes.c_int(n_threads))
    if rc != 0:
        raise RuntimeError("tide_oracle_attend_f64 rejected its arguments")
    return out, lse
