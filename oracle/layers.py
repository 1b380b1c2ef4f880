"""Oracle for a cache with several layers (test infrastructure only).

The paper schedules on tokens (Section 4.1: each rank is a token budget pool) and never mentions layers; a model
with L attention layers simply keeps L K/V histories per task, all of the same length.  The reading both
implementations follow: a cache with L layers behaves as L independent one-layer caches that receive the same
sequence of operations, each with its own layer's K/V rows.  Because the allocator rule never looks at values,
the L caches always hold identical page tables, lengths and free stacks - which is why an implementation may
keep one table for all layers.  This module is that definition written out: L `PagedKVOracle` objects stepped
side by side, with the identity of their bookkeeping asserted after every operation.
"""
from __future__ import annotations

import numpy as np

from .paged_kv import PagedKVOracle


class LayeredKVOracle:
    def __init__(self, num_layers: int, **geometry):
        assert num_layers >= 1
        self.L = int(num_layers)
        self.layers = [PagedKVOracle(**geometry) for _ in range(self.L)]

    def layer(self, l: int) -> PagedKVOracle:
        return self.layers[l]

    def _same_bookkeeping(self):
        h0 = self.layers[0].state_hash()
        for c in self.layers[1:]:
            assert c.state_hash() == h0, "layers disagree on page tables / lengths / free stack"

    def _all(self, name, *args):
        """Calls the same operation on every layer; a refusal must come from every layer alike (the first
        layer's exception is re-raised after the others were seen to refuse too)."""
        first_err = None
        for i, c in enumerate(self.layers):
            try:
                getattr(c, name)(*args)
                assert first_err is None, "a later layer accepted what layer 0 refused"
            except Exception as e:  # noqa: BLE001 - re-raised below
                assert i == 0 or first_err is not None, "a later layer refused what layer 0 accepted"
                if first_err is None:
                    first_err = e
        self._same_bookkeeping()
        if first_err is not None:
            raise first_err

    # ---- operations that carry no values ---------------------------------------------------------------
    def alloc(self, task, reserve_tokens=0):
        self._all("alloc", task, reserve_tokens)

    def release(self, task):
        self._all("release", task)

    def release_many(self, tasks):
        self._all("release_many", tasks)

    def truncate(self, task, new_len):
        self._all("truncate", task, new_len)

    def fork(self, parent, child):
        self._all("fork", parent, child)

    def prune(self, task, keep_prefix, tail_begin):
        self._all("prune", task, keep_prefix, tail_begin)

    def reset(self, free_order=None):
        self._all("reset", free_order)

    # ---- append: layer l receives new_k[l], new_v[l] ---------------------------------------------------
    def append(self, task_ids, indptr, new_k, new_v):
        """new_k / new_v: uint16 [L, T, Hkv, D]."""
        new_k, new_v = np.asarray(new_k), np.asarray(new_v)
        assert new_k.shape[0] == self.L and new_v.shape[0] == self.L
        first_err = None
        for i, c in enumerate(self.layers):
            try:
                c.append(task_ids, indptr, new_k[i], new_v[i])
                assert first_err is None
            except Exception as e:  # noqa: BLE001
                assert i == 0 or first_err is not None
                if first_err is None:
                    first_err = e
        self._same_bookkeeping()
        if first_err is not None:
            raise first_err

    # ---- introspection (any layer answers for all) ---------------------------------------------------
    def task_len(self, task):
        return self.layers[0].task_len(task)

    def page_table(self, task):
        return self.layers[0].page_table(task)

    def page_refs(self, task):
        return self.layers[0].page_refs(task)

    def free_pages(self):
        return self.layers[0].free_pages()

    def used_tokens(self):
        return self.layers[0].used_tokens()

    def read(self, l, task, length=None):
        return self.layers[l].read(task, length)
