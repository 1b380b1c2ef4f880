"""ctypes binding of libtide.so: the same names as include/tide.h, argument marshalling only.

Every step of the path runs inside the CUDA library; this module only turns torch tensors / numpy
arrays into pointers.  There is no fallback: if libtide.so is missing or cannot be loaded the import
of this module raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtide.so")

OK = 0
ERR_INVALID_ARG, ERR_UNKNOWN_TASK, ERR_TASK_EXISTS, ERR_DUPLICATE_TASK = -1, -2, -3, -4
ERR_NO_PAGES, ERR_TABLE_FULL, ERR_CTX_RANGE, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE_TIMEOUT = -5, -6, -7, -8, -9, -10
STATIC_MAX_ROWS = 64
# knobs of tide_tune (tide_tune_t)
(TUNE_ITEMS_PER_SM, TUNE_GROUPING, TUNE_MIN_SAVED_BYTES, TUNE_HOST_STEP_CHUNKS, TUNE_UMMA_MIN_ROWS, TUNE_WAIT_LIMIT_US,
 TUNE_DROP_FIRST_STAGE, TUNE_UMMA_TILE_KEYS, TUNE_UPLOAD_BY_KERNEL, TUNE_INLINE_DESCRIPTORS, TUNE_HOST_ZERO_COPY) = range(11)


class TideError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


class tide_row_t(ctypes.Structure):
    _fields_ = [("task", ctypes.c_int32), ("q_len", ctypes.c_int32), ("ctx_len", ctypes.c_int32)]


class tide_kv_config_t(ctypes.Structure):
    _fields_ = [
        ("num_layers", ctypes.c_int32), ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32), ("max_tasks", ctypes.c_int32),
        ("max_pages_per_task", ctypes.c_int32), ("max_batch_rows", ctypes.c_int32),
        ("num_pages", ctypes.c_int64), ("max_batch_tokens", ctypes.c_int64),
        ("pool", ctypes.c_void_p), ("pool_bytes", ctypes.c_size_t),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("free_order", ctypes.c_void_p),
    ]


EXPORTS = [
    "tide_strerror", "tide_kv_required_bytes", "tide_kv_create", "tide_kv_destroy", "tide_kv_reset",
    "tide_kv_alloc", "tide_kv_append", "tide_attend", "tide_step_host", "tide_kv_release", "tide_kv_truncate",
    "tide_kv_task_len", "tide_kv_page_table", "tide_kv_usage", "tide_kv_read", "tide_status", "tide_last_plan",
    "tide_set_profiling", "tide_phase_ms", "tide_attend_decode_static", "tide_kv_release_many", "tide_kv_prune", "tide_kv_fork", "tide_kv_page_refs",
    "tide_kv_extend", "tide_kv_write", "tide_step_begin", "tide_step_layer", "tide_step_fix_grids", "tide_last_sharing",
    "tide_tune",
]

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_10402_b200.build` "
                      "(there is no fallback path)")
lib = ctypes.CDLL(LIB_PATH)
lib.tide_strerror.restype = ctypes.c_char_p
lib.tide_strerror.argtypes = [ctypes.c_int]
for _name in EXPORTS[1:]:
    getattr(lib, _name).restype = ctypes.c_int


def strerror(code: int) -> str:
    return lib.tide_strerror(int(code)).decode()


def _check(code: int, what: str):
    if code != OK:
        raise TideError(code, what)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _ptr(x):
    """Device / host pointer of a torch tensor, numpy array, int or None."""
    if x is None:
        return ctypes.c_void_p(0)
    if isinstance(x, int):
        return ctypes.c_void_p(x)
    if isinstance(x, np.ndarray):
        return ctypes.c_void_p(x.ctypes.data)
    return ctypes.c_void_p(x.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return ctypes.c_void_p(stream)
    return ctypes.c_void_p(stream.cuda_stream)


def rows_array(rows):
    """[(task, q_len, ctx_len)] -> ctypes array of tide_row_t."""
    arr = (tide_row_t * len(rows))()
    for i, (t, n, c) in enumerate(rows):
        arr[i].task, arr[i].q_len, arr[i].ctx_len = int(t), int(n), int(c)
    return arr


def make_config(Hq, Hkv, D, S, num_pages, max_tasks, max_pages_per_task, max_batch_rows, max_batch_tokens, num_layers=1):
    cfg = tide_kv_config_t()
    cfg.num_layers = int(num_layers)
    cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.page_size = int(Hq), int(Hkv), int(D), int(S)
    cfg.max_tasks, cfg.max_pages_per_task, cfg.max_batch_rows = int(max_tasks), int(max_pages_per_task), int(max_batch_rows)
    cfg.num_pages, cfg.max_batch_tokens = int(num_pages), int(max_batch_tokens)
    return cfg


def tide_kv_required_bytes(cfg):
    pb, wb = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib.tide_kv_required_bytes(ctypes.byref(cfg), ctypes.byref(pb), ctypes.byref(wb)), "tide_kv_required_bytes")
    return pb.value, wb.value


class TideKV:
    """One paged cache on the current CUDA device.  Methods mirror the C entry points one to one."""

    def __init__(self, Hq, Hkv, D, S, num_pages, max_tasks, max_pages_per_task, max_batch_rows, max_batch_tokens,
                 free_order=None, device="cuda", num_layers=1):
        import torch
        self.cfg = make_config(Hq, Hkv, D, S, num_pages, max_tasks, max_pages_per_task, max_batch_rows, max_batch_tokens,
                               num_layers)
        self.num_layers = int(num_layers)
        pb, wb = tide_kv_required_bytes(self.cfg)
        # PyTorch only supplies device memory (and streams)
        self.pool = torch.empty(pb + 1024, dtype=torch.uint8, device=device)
        self.workspace = torch.empty(wb + 256, dtype=torch.uint8, device=device)
        pool_ptr = (self.pool.data_ptr() + 1023) // 1024 * 1024
        ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256
        self.cfg.pool, self.cfg.pool_bytes = pool_ptr, pb
        self.cfg.workspace, self.cfg.workspace_bytes = ws_ptr, wb
        self._free_order = None if free_order is None else _i32(free_order)
        self.cfg.free_order = None if free_order is None else self._free_order.ctypes.data
        self.Hq, self.Hkv, self.D, self.S = int(Hq), int(Hkv), int(D), int(S)
        self.handle = ctypes.c_void_p(0)
        _check(lib.tide_kv_create(ctypes.byref(self.cfg), ctypes.byref(self.handle)), "tide_kv_create")

    def close(self):
        if self.handle:
            lib.tide_kv_destroy(self.handle)
            self.handle = ctypes.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- lifecycle ----
    def reset(self, free_order=None):
        fo = None if free_order is None else _i32(free_order)
        _check(lib.tide_kv_reset(self.handle, _ptr(fo)), "tide_kv_reset")

    def alloc(self, task, reserve_tokens=0):
        _check(lib.tide_kv_alloc(self.handle, ctypes.c_int32(task), ctypes.c_int64(reserve_tokens)), "tide_kv_alloc")

    def release(self, task):
        _check(lib.tide_kv_release(self.handle, ctypes.c_int32(task)), "tide_kv_release")

    def fork(self, parent, child, stream=None):
        _check(lib.tide_kv_fork(self.handle, ctypes.c_int32(0), ctypes.c_int32(parent), ctypes.c_int32(child), _stream(stream)), "tide_kv_fork")

    def page_refs(self, task):
        n = ctypes.c_int32(0)
        _check(lib.tide_kv_page_refs(self.handle, ctypes.c_int32(task), None, ctypes.c_int32(0), ctypes.byref(n)), "tide_kv_page_refs")
        out = np.empty(n.value, dtype=np.int32)
        _check(lib.tide_kv_page_refs(self.handle, ctypes.c_int32(task), _ptr(out), ctypes.c_int32(n.value), ctypes.byref(n)), "tide_kv_page_refs")
        return out

    def release_many(self, task_ids):
        ids = _i32(task_ids)
        _check(lib.tide_kv_release_many(self.handle, ctypes.c_int32(ids.shape[0]), _ptr(ids)), "tide_kv_release_many")

    def prune(self, task, keep_prefix, tail_begin, stream=None):
        _check(lib.tide_kv_prune(self.handle, ctypes.c_int32(0), ctypes.c_int32(task), ctypes.c_int32(keep_prefix),
                                 ctypes.c_int32(tail_begin), _stream(stream)), "tide_kv_prune")

    def truncate(self, task, new_len):
        _check(lib.tide_kv_truncate(self.handle, ctypes.c_int32(task), ctypes.c_int32(new_len)), "tide_kv_truncate")

    def append(self, task_ids, indptr, new_k, new_v, stream=None):
        ids, ip = _i32(task_ids), _i32(indptr)
        assert ip.shape[0] == ids.shape[0] + 1
        _check(lib.tide_kv_append(self.handle, ctypes.c_int32(0), ctypes.c_int32(ids.shape[0]), _ptr(ids), _ptr(ip),
                                  _ptr(new_k), _ptr(new_v), _stream(stream)), "tide_kv_append")

    def extend(self, task_ids, indptr, stream=None):
        ids, ip = _i32(task_ids), _i32(indptr)
        assert ip.shape[0] == ids.shape[0] + 1
        _check(lib.tide_kv_extend(self.handle, ctypes.c_int32(ids.shape[0]), _ptr(ids), _ptr(ip), _stream(stream)), "tide_kv_extend")

    def write(self, layer, task_ids, indptr, new_k, new_v, stream=None):
        ids, ip = _i32(task_ids), _i32(indptr)
        assert ip.shape[0] == ids.shape[0] + 1
        _check(lib.tide_kv_write(self.handle, ctypes.c_int32(layer), ctypes.c_int32(ids.shape[0]), _ptr(ids), _ptr(ip),
                                 _ptr(new_k), _ptr(new_v), _stream(stream)), "tide_kv_write")

    def step_begin(self, rows, stream=None):
        arr = rows if not isinstance(rows, (list, tuple)) else rows_array(rows)
        _check(lib.tide_step_begin(self.handle, ctypes.c_int32(len(arr)), arr, _stream(stream)), "tide_step_begin")

    def step_fix_grids(self, max_decode_items=0, max_tile_items=0, max_umma_items=0, max_merge_rows=0, max_tokens=0):
        _check(lib.tide_step_fix_grids(self.handle, ctypes.c_int32(max_decode_items), ctypes.c_int32(max_tile_items),
                                       ctypes.c_int32(max_umma_items), ctypes.c_int32(max_merge_rows),
                                       ctypes.c_int32(max_tokens)), "tide_step_fix_grids")

    def step_layer(self, layer, new_k, new_v, q, scale, out, lse=None, stream=None):
        _check(lib.tide_step_layer(self.handle, ctypes.c_int32(layer), _ptr(new_k), _ptr(new_v), _ptr(q),
                                   ctypes.c_float(scale), _ptr(out), _ptr(lse), _stream(stream)), "tide_step_layer")

    def attend(self, rows, q, scale, out, lse=None, page_table=None, stream=None, layer=0):
        arr = rows if not isinstance(rows, (list, tuple)) else rows_array(rows)
        _check(lib.tide_attend(self.handle, ctypes.c_int32(layer), ctypes.c_int32(len(arr)), arr, _ptr(page_table), _ptr(q),
                               ctypes.c_float(scale), _ptr(out), _ptr(lse), _stream(stream)), "tide_attend")

    def attend_decode_static(self, rows, q, scale, out, lse=None, stream=None):
        """tide_attend_decode_static: decode-style rows only, scratch in the library's fixed device array."""
        arr = rows if not isinstance(rows, (list, tuple)) else rows_array(rows)
        _check(lib.tide_attend_decode_static(self.handle, ctypes.c_int32(len(arr)), arr, _ptr(q), ctypes.c_float(scale),
                                             _ptr(out), _ptr(lse), _stream(stream)), "tide_attend_decode_static")

    def step_host(self, rows, new_k, new_v, q, scale, out, lse=None, stream=None):
        arr = rows if not isinstance(rows, (list, tuple)) else rows_array(rows)
        _check(lib.tide_step_host(self.handle, ctypes.c_int32(0), ctypes.c_int32(len(arr)), arr, _ptr(new_k), _ptr(new_v),
                                  _ptr(q), ctypes.c_float(scale), _ptr(out), _ptr(lse), _stream(stream)), "tide_step_host")

    # ---- introspection ----
    def task_len(self, task):
        v = ctypes.c_int32(0)
        _check(lib.tide_kv_task_len(self.handle, ctypes.c_int32(task), ctypes.byref(v)), "tide_kv_task_len")
        return v.value

    def page_table(self, task):
        n = ctypes.c_int32(0)
        _check(lib.tide_kv_page_table(self.handle, ctypes.c_int32(task), None, ctypes.c_int32(0), ctypes.byref(n)), "tide_kv_page_table")
        out = np.empty(n.value, dtype=np.int32)
        _check(lib.tide_kv_page_table(self.handle, ctypes.c_int32(task), _ptr(out), ctypes.c_int32(n.value), ctypes.byref(n)), "tide_kv_page_table")
        return out

    def usage(self):
        u, f = ctypes.c_int64(0), ctypes.c_int64(0)
        _check(lib.tide_kv_usage(self.handle, ctypes.byref(u), ctypes.byref(f)), "tide_kv_usage")
        return u.value, f.value

    def read(self, task, stream=None, layer=0):
        """Logical K, V of a task as torch uint16-bit tensors (int16 view) [len, Hkv, D] on the device."""
        import torch
        L = self.task_len(task)
        k = torch.empty((L, self.Hkv, self.D), dtype=torch.int16, device=self.pool.device)
        v = torch.empty_like(k)
        _check(lib.tide_kv_read(self.handle, ctypes.c_int32(layer), ctypes.c_int32(task), _ptr(k), _ptr(v), _stream(stream)), "tide_kv_read")
        return k, v

    def status(self, stream=None):
        return lib.tide_status(self.handle, _stream(stream))

    def tune(self, knob, value):
        _check(lib.tide_tune(self.handle, ctypes.c_int(knob), ctypes.c_int64(int(value))), "tide_tune")

    def set_profiling(self, enable):
        _check(lib.tide_set_profiling(self.handle, ctypes.c_int(1 if enable else 0)), "tide_set_profiling")

    def phase_ms(self):
        v = [ctypes.c_float(0) for _ in range(4)]
        _check(lib.tide_phase_ms(self.handle, *[ctypes.byref(x) for x in v]), "tide_phase_ms")
        return {"append": v[0].value, "decode": v[1].value, "tile": v[2].value, "merge": v[3].value}

    def last_sharing(self):
        a, b = ctypes.c_int64(0), ctypes.c_int64(0)
        _check(lib.tide_last_sharing(self.handle, ctypes.byref(a), ctypes.byref(b)), "tide_last_sharing")
        return {"groups": a.value, "rows": b.value}

    def last_plan(self):
        a, b, c, d = (ctypes.c_int64(0) for _ in range(4))
        _check(lib.tide_last_plan(self.handle, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c), ctypes.byref(d)), "tide_last_plan")
        return {"decode_items": a.value, "prefill_items": b.value, "merge_rows": c.value, "kernel_launches": d.value}
