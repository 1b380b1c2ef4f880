"""Oracle page allocator and logical KV cache (test infrastructure only).

The paper's Continuous Task Batching keeps a paused task's KV state resident
and resumes it with the observation tokens appended (Section 4, first
paragraph; Section 1, CTB bullet).  It treats each rollout rank as a token
budget pool whose usage is tracked per task (Section 4.1) and flushes all
state at each weight synchronisation (Section 5.2).  The paper does not give
an allocator; the rule below is the reading both implementations follow so
that page tables can be compared bit for bit:

  * free pages form a LIFO stack; successive pops of a fresh pool return
    free_order[0], free_order[1], ...
  * append processes tasks in array order and tokens in order; a page is
    popped exactly when a token lands on slot 0 of a new logical page, so a
    partial last page is filled before a new page is taken
  * append validates everything first and changes nothing on error
  * release pushes a task's pages back last-to-first, so re-appending the same
    length straight away receives the same pages in the same order
  * truncate(task, new_len) pushes back pages ceil(new_len/S).. last-to-first
  * pages are reference counted so that the trajectories of a GRPO group can
    share their common prefix (Section 2.1: G trajectories per prompt; end of
    Section 4: worker affinity keeps shared prefixes on one rank).
    fork(parent, child) gives the child the parent's FULL pages (count + 1
    each) and a fresh copy of the parent's partial last page, if any; a page
    goes back to the free stack only when its count drops to 0; an append that
    would write into a page whose count is above 1 (possible after a truncate
    into shared pages) first replaces it by a private copy, popped before the
    task's other pages

Cache contents are raw bf16 bit patterns (uint16); this module never does
floating-point arithmetic.  Physical storage here is token-major
[page][slot][kv_head][d]; that layout is the oracle's own business.
"""
from __future__ import annotations

import numpy as np

OK = 0
ERR_INVALID_ARG = -1
ERR_UNKNOWN_TASK = -2
ERR_TASK_EXISTS = -3
ERR_DUPLICATE_TASK = -4
ERR_NO_PAGES = -5
ERR_TABLE_FULL = -6
ERR_CTX_RANGE = -7


class OracleError(Exception):
    def __init__(self, code: int, msg: str = ""):
        super().__init__(f"oracle error {code}: {msg}")
        self.code = code


def _ceil_div(a: int, b: int) -> int:
    return -(-a // b)


class PagedKVOracle:
    """Plain-Python page allocator + paged bf16 store.

    store_values=False keeps only the integer bookkeeping (page tables,
    lengths, free stack), for workloads whose values are checked elsewhere.
    """

    def __init__(self, num_pages: int, page_size: int, num_kv_heads: int, head_dim: int,
                 max_tasks: int, max_pages_per_task: int, free_order=None, store_values: bool = True):
        if min(num_pages, page_size, num_kv_heads, head_dim, max_tasks, max_pages_per_task) <= 0:
            raise OracleError(ERR_INVALID_ARG, "non-positive geometry")
        self.P, self.S, self.Hkv, self.D = int(num_pages), int(page_size), int(num_kv_heads), int(head_dim)
        self.max_tasks, self.max_pages_per_task = int(max_tasks), int(max_pages_per_task)
        if free_order is None:
            free_order = np.arange(self.P, dtype=np.int64)
        free_order = np.asarray(free_order, dtype=np.int64)
        if free_order.shape != (self.P,) or not np.array_equal(np.sort(free_order), np.arange(self.P)):
            raise OracleError(ERR_INVALID_ARG, "free_order is not a permutation of [0, num_pages)")
        # python list used as a stack: pop() takes the END, so store reversed
        self.free = [int(p) for p in free_order[::-1]]
        self.live = {}          # task -> True
        self.len = {}           # task -> resident tokens
        self.pages = {}         # task -> list of physical pages
        self.ref = {}           # physical page -> number of tasks holding it (absent = free)
        self.store_values = store_values
        if store_values:
            self.pool_k = np.zeros((self.P, self.S, self.Hkv, self.D), dtype=np.uint16)
            self.pool_v = np.zeros((self.P, self.S, self.Hkv, self.D), dtype=np.uint16)

    # ---- introspection ---------------------------------------------------
    def free_pages(self) -> int:
        return len(self.free)

    def used_tokens(self) -> int:
        return sum(self.len.values())

    def task_len(self, task: int) -> int:
        self._check_live(task)
        return self.len[task]

    def page_table(self, task: int) -> np.ndarray:
        self._check_live(task)
        return np.asarray(self.pages[task], dtype=np.int32)

    def free_stack_top_first(self):
        return list(reversed(self.free))

    def state_hash(self):
        """A value that changes whenever any bookkeeping changes."""
        return (tuple(self.free), tuple(sorted((t, self.len[t], tuple(self.pages[t])) for t in self.live)),
                tuple(sorted(self.ref.items())))

    def _check_task_id(self, task: int):
        if not (0 <= task < self.max_tasks):
            raise OracleError(ERR_INVALID_ARG, f"task id {task} out of range")

    def _check_live(self, task: int):
        self._check_task_id(task)
        if task not in self.live:
            raise OracleError(ERR_UNKNOWN_TASK, f"task {task} is not live")

    # ---- lifecycle -------------------------------------------------------
    def alloc(self, task: int, reserve_tokens: int = 0):
        """Register a task with length 0.  Takes no pages.  reserve_tokens is
        the admission check of Section 4.1: admit only if the remaining
        headroom can hold the probed footprint."""
        self._check_task_id(task)
        if reserve_tokens < 0:
            raise OracleError(ERR_INVALID_ARG, "negative reserve")
        if task in self.live:
            raise OracleError(ERR_TASK_EXISTS, f"task {task} already live")
        if len(self.free) * self.S < reserve_tokens:
            raise OracleError(ERR_NO_PAGES, "headroom below the requested reserve")
        self.live[task] = True
        self.len[task] = 0
        self.pages[task] = []

    def append(self, task_ids, indptr, new_k=None, new_v=None):
        """Append indptr[j+1]-indptr[j] tokens to task_ids[j], for every j.

        new_k / new_v: uint16 [T, Hkv, D] (raw bf16 bits), T = indptr[-1]."""
        task_ids = [int(t) for t in task_ids]
        indptr = [int(x) for x in indptr]
        n = len(task_ids)
        if len(indptr) != n + 1 or indptr[0] != 0:
            raise OracleError(ERR_INVALID_ARG, "indptr must have n+1 entries starting at 0")
        for j in range(n):
            if indptr[j + 1] < indptr[j]:
                raise OracleError(ERR_INVALID_ARG, "indptr must be non-decreasing")
        for t in task_ids:
            self._check_live(t)
        if len(set(task_ids)) != n:
            raise OracleError(ERR_DUPLICATE_TASK, "a task appears twice in one append")
        T = indptr[-1]
        if self.store_values:
            for a in (new_k, new_v):
                if a is None or a.dtype != np.uint16 or a.shape != (T, self.Hkv, self.D):
                    raise OracleError(ERR_INVALID_ARG, "new_k/new_v must be uint16 [T,Hkv,D]")
        need_total = 0
        for j, t in enumerate(task_ids):
            c = indptr[j + 1] - indptr[j]
            after = _ceil_div(self.len[t] + c, self.S)
            need_total += after - _ceil_div(self.len[t], self.S)
            if c > 0 and self._last_page_is_shared(t):
                need_total += 1
            if after > self.max_pages_per_task:
                raise OracleError(ERR_TABLE_FULL, f"task {t} would need {after} pages")
        if need_total > len(self.free):
            raise OracleError(ERR_NO_PAGES, f"need {need_total} pages, {len(self.free)} free")
        # ---- mutation starts here ----
        for j, t in enumerate(task_ids):
            if indptr[j + 1] > indptr[j] and self._last_page_is_shared(t):
                self._make_last_page_private(t)
            for i in range(indptr[j + 1] - indptr[j]):
                pos = self.len[t] + i
                if pos % self.S == 0:
                    self.pages[t].append(self._pop())
                if self.store_values:
                    page, slot = self.pages[t][pos // self.S], pos % self.S
                    self.pool_k[page, slot] = new_k[indptr[j] + i]
                    self.pool_v[page, slot] = new_v[indptr[j] + i]
            self.len[t] += indptr[j + 1] - indptr[j]

    # ---- reference counting ---------------------------------------------
    def _pop(self) -> int:
        page = self.free.pop()
        self.ref[page] = 1
        return page

    def _unref(self, page: int):
        self.ref[page] -= 1
        if self.ref[page] == 0:
            del self.ref[page]
            self.free.append(page)

    def _last_page_is_shared(self, task: int) -> bool:
        return self.len[task] % self.S != 0 and self.ref[self.pages[task][-1]] > 1

    def _make_last_page_private(self, task: int):
        old = self.pages[task][-1]
        new = self._pop()
        if self.store_values:
            self.pool_k[new] = self.pool_k[old]
            self.pool_v[new] = self.pool_v[old]
        self.pages[task][-1] = new
        self._unref(old)

    def fork(self, parent: int, child: int):
        """child becomes a live task with the parent's current content; full pages are shared."""
        self._check_live(parent)
        self._check_task_id(child)
        if child in self.live:
            raise OracleError(ERR_TASK_EXISTS, f"task {child} already live")
        L = self.len[parent]
        n_full = L // self.S
        if L % self.S and not self.free:
            raise OracleError(ERR_NO_PAGES, "no page for the copy of the partial last page")
        self.live[child] = True
        self.len[child] = L
        self.pages[child] = list(self.pages[parent][:n_full])
        for page in self.pages[child]:
            self.ref[page] += 1
        if L % self.S:
            new = self._pop()
            if self.store_values:
                old = self.pages[parent][n_full]
                self.pool_k[new] = self.pool_k[old]
                self.pool_v[new] = self.pool_v[old]
            self.pages[child].append(new)

    def page_refs(self, task: int) -> np.ndarray:
        self._check_live(task)
        return np.asarray([self.ref[p] for p in self.pages[task]], dtype=np.int32)

    def release(self, task: int):
        self._check_live(task)
        for page in reversed(self.pages[task]):
            self._unref(page)
        del self.live[task], self.len[task], self.pages[task]

    def truncate(self, task: int, new_len: int):
        self._check_live(task)
        if not (0 <= new_len <= self.len[task]):
            raise OracleError(ERR_INVALID_ARG, "new_len outside [0, len]")
        keep = _ceil_div(new_len, self.S)
        while len(self.pages[task]) > keep:
            self._unref(self.pages[task].pop())
        self.len[task] = new_len

    def release_many(self, tasks):
        tasks = [int(t) for t in tasks]
        for t in tasks:
            self._check_live(t)
        if len(set(tasks)) != len(tasks):
            raise OracleError(ERR_DUPLICATE_TASK, "a task appears twice")
        for t in tasks:
            self.release(t)

    def prune(self, task: int, keep_prefix: int, tail_begin: int):
        """Sliding-window pruning (Appendix C.2): keep tokens [0, keep_prefix) and [tail_begin, len), written
        out as its definition: read the tail, truncate to keep_prefix, append the tail again."""
        self._check_live(task)
        if not (0 <= keep_prefix <= tail_begin <= self.len[task]):
            raise OracleError(ERR_INVALID_ARG, "need 0 <= keep_prefix <= tail_begin <= len")
        if keep_prefix == tail_begin:
            return
        if self.store_values:
            k, v = self.read(task)
            tail_k, tail_v = k[tail_begin:].copy(), v[tail_begin:].copy()
        n_tail = self.len[task] - tail_begin
        # like every call, prune changes nothing when it has to refuse: remember the bookkeeping, and put it
        # back if the append of the tail finds too few pages (possible only when the task shares pages, since
        # shared pages do not return to the free stack when the task lets go of them)
        before = (list(self.free), dict(self.len), {t: list(p) for t, p in self.pages.items()}, dict(self.ref))
        self.truncate(task, keep_prefix)
        try:
            if self.store_values:
                self.append([task], [0, n_tail], tail_k, tail_v)
            else:
                self.append([task], [0, n_tail])
        except OracleError:
            self.free, self.len, self.pages, self.ref = before
            raise

    def reset(self, free_order=None):
        """Flush every task (the cache flush at a weight synchronisation,
        Section 5.2) and restart the free stack from free_order."""
        if free_order is None:
            free_order = np.arange(self.P, dtype=np.int64)
        free_order = np.asarray(free_order, dtype=np.int64)
        if free_order.shape != (self.P,) or not np.array_equal(np.sort(free_order), np.arange(self.P)):
            raise OracleError(ERR_INVALID_ARG, "free_order is not a permutation")
        self.free = [int(p) for p in free_order[::-1]]
        self.live, self.len, self.pages, self.ref = {}, {}, {}, {}

    # ---- reads -----------------------------------------------------------
    def read(self, task: int, length=None):
        """Logical (contiguous) K and V bits [len, Hkv, D] gathered through the page table."""
        self._check_live(task)
        L = self.len[task] if length is None else int(length)
        if not (0 <= L <= self.len[task]):
            raise OracleError(ERR_CTX_RANGE, "length beyond resident tokens")
        k = np.empty((L, self.Hkv, self.D), dtype=np.uint16)
        v = np.empty((L, self.Hkv, self.D), dtype=np.uint16)
        for lp, page in enumerate(self.pages[task]):
            lo = lp * self.S
            if lo >= L:
                break
            c = min(self.S, L - lo)
            k[lo:lo + c] = self.pool_k[page, :c]
            v[lo:lo + c] = self.pool_v[page, :c]
        return k, v

    def check_rows(self, rows):
        """rows: iterable of (task, q_len, ctx_len).  The same task may appear in several rows."""
        for (task, q_len, ctx_len) in rows:
            self._check_live(int(task))
            if not (1 <= q_len <= ctx_len <= self.len[int(task)]):
                raise OracleError(ERR_CTX_RANGE, f"row ({task},{q_len},{ctx_len}) vs len {self.len[int(task)]}")
