"""tide-kv: the GPU hot path behind Continuous Task Batching, for B200 (sm_100a).

A paged bf16 KV cache whose tasks keep their state across environment pauses,
a page-append scatter for resumed tasks' observation tokens, and GQA attention
of a mixed decode / resume batch over the preserved cache.  Everything runs in
hand-written CUDA behind a C ABI (include/tide.h); `tide` is the thin ctypes
binding with the same names.  `inputs` holds the seeded synthetic workloads.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "tide"]


def __getattr__(name):
    if name == "tide":
        import importlib
        return importlib.import_module(".tide", __name__)
    raise AttributeError(name)
