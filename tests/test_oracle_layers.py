"""Pins for the multi-layer oracle and for prune's all-or-nothing rule.

The layered oracle is checked against a model with no pages at all: per layer and task a plain Python list of
token rows, on which fork is a list copy, truncate a slice and prune the concatenation of two slices.  Any bleed
between layers, any page bookkeeping slip or any reordering of the tail shows up as a different list.
The prune refusal is pinned on a pool small enough to trace by hand."""
import numpy as np
import pytest

from oracle.layers import LayeredKVOracle
from oracle.paged_kv import ERR_NO_PAGES, OracleError, PagedKVOracle


def _rows(rng, n, hkv, d):
    return rng.integers(0, 1 << 16, size=(n, hkv, d), dtype=np.uint16)


def test_layered_oracle_equals_per_layer_token_lists():
    rng = np.random.default_rng(11)
    L, S, HKV, D, P = 3, 4, 2, 8, 64
    orc = LayeredKVOracle(L, num_pages=P, page_size=S, num_kv_heads=HKV, head_dim=D, max_tasks=8, max_pages_per_task=16,
                          free_order=rng.permutation(P))
    shadow = [dict() for _ in range(L)]          # layer -> task -> list of (k_row, v_row)

    def append(tasks, counts):
        indptr = np.concatenate([[0], np.cumsum(counts)])
        T = int(indptr[-1])
        nk = np.stack([_rows(rng, T, HKV, D) for _ in range(L)])
        nv = np.stack([_rows(rng, T, HKV, D) for _ in range(L)])
        orc.append(tasks, indptr, nk, nv)
        for l in range(L):
            for j, t in enumerate(tasks):
                for i in range(indptr[j], indptr[j + 1]):
                    shadow[l][t].append((nk[l, i], nv[l, i]))

    def check():
        for l in range(L):
            for t, rows in shadow[l].items():
                k, v = orc.read(l, t)
                assert k.shape[0] == len(rows) == orc.task_len(t)
                for i, (rk, rv) in enumerate(rows):
                    assert np.array_equal(k[i], rk) and np.array_equal(v[i], rv), (l, t, i)

    for t in (0, 1, 2):
        orc.alloc(t)
        for l in range(L):
            shadow[l][t] = []
    append([0, 1, 2], [9, 4, 1])
    append([2, 0], [7, 3])
    check()
    orc.fork(0, 3)                                   # 12 tokens: three full pages shared, nothing copied
    orc.fork(1, 4)                                   # 4 tokens: one full page
    orc.fork(2, 5)                                   # 8 tokens
    for l in range(L):
        shadow[l][3], shadow[l][4], shadow[l][5] = list(shadow[l][0]), list(shadow[l][1]), list(shadow[l][2])
    append([3, 0, 4], [2, 5, 6])
    check()
    orc.truncate(3, 6)                               # into a shared page: the next append must copy it first
    for l in range(L):
        shadow[l][3] = shadow[l][3][:6]
    append([3], [5])
    check()
    orc.prune(0, 3, 10)                              # task 0 shares pages with task 3
    orc.prune(2, 4, 5)
    for l in range(L):
        shadow[l][0] = shadow[l][0][:3] + shadow[l][0][10:]
        shadow[l][2] = shadow[l][2][:4] + shadow[l][2][5:]
    check()
    orc.release(1)
    for l in range(L):
        del shadow[l][1]
    append([4, 5], [1, 9])
    check()
    # one table serves all layers
    for t in shadow[0]:
        for l in range(1, L):
            assert np.array_equal(orc.layer(l).page_table(t), orc.layer(0).page_table(t))


def test_prune_refuses_without_changing_anything_hand_traced():
    # 4 pages of 4 tokens, identity order.  Task 0 takes pages 0, 1 (8 tokens); task 1 is forked from it (shares
    # both, nothing copied) and grows by 8 tokens onto pages 2, 3.  The pool is now empty.
    c = PagedKVOracle(4, 4, 1, 2, max_tasks=2, max_pages_per_task=4, store_values=False)
    c.alloc(0)
    c.append([0], [0, 8])
    c.fork(0, 1)
    c.append([1], [0, 8])
    assert list(c.page_table(1)) == [0, 1, 2, 3] and c.free_pages() == 0
    # prune(task 1, keep 2, tail from 4): the shorter task has 14 tokens = 4 pages.  It keeps page 0, which it
    # shares, so it needs a private copy (1 page) plus 3 more; only pages 2 and 3 come back (page 1 is still
    # task 0's).  4 > 2: refused, and nothing may have changed.
    before = c.state_hash()
    with pytest.raises(OracleError) as e:
        c.prune(1, 2, 4)
    assert e.value.code == ERR_NO_PAGES
    assert c.state_hash() == before
    # once task 0 is gone every page is task 1's own: page 1 comes back too, no copy is needed, and the pages
    # return in the order 3, 2, 1 so they are taken again as 1, 2, 3.
    c.release(0)
    c.prune(1, 2, 4)
    assert list(c.page_table(1)) == [0, 1, 2, 3] and c.task_len(1) == 14 and c.free_pages() == 0


def test_reset_of_the_layered_oracle_flushes_every_layer_alike():
    """After a reset every layer hands pages out in the new order, holds no task, and keeps layers apart as before:
    checked against per-layer token lists that are simply emptied."""
    rng = np.random.default_rng(5)
    L, S, HKV, D, P = 3, 4, 1, 4, 8
    orc = LayeredKVOracle(L, num_pages=P, page_size=S, num_kv_heads=HKV, head_dim=D, max_tasks=4, max_pages_per_task=8,
                          free_order=[7, 6, 5, 4, 3, 2, 1, 0])
    orc.alloc(0)
    orc.alloc(1)
    orc.append([0, 1], [0, 6, 9], np.stack([_rows(rng, 9, HKV, D) for _ in range(L)]), np.stack([_rows(rng, 9, HKV, D) for _ in range(L)]))
    assert list(orc.page_table(0)) == [7, 6] and list(orc.page_table(1)) == [5]
    orc.fork(0, 2)
    orc.reset([1, 3, 5, 7, 0, 2, 4, 6])
    assert orc.free_pages() == P and orc.used_tokens() == 0
    for l in range(L):
        assert orc.layer(l).live == {} and orc.layer(l).ref == {}
        assert orc.layer(l).free_stack_top_first() == [1, 3, 5, 7, 0, 2, 4, 6]
    with pytest.raises(OracleError):
        orc.task_len(0)
    orc.alloc(2)
    nk = np.stack([_rows(rng, 5, HKV, D) for _ in range(L)])
    nv = np.stack([_rows(rng, 5, HKV, D) for _ in range(L)])
    orc.append([2], [0, 5], nk, nv)
    assert list(orc.page_table(2)) == [1, 3]
    for l in range(L):
        k, v = orc.read(l, 2)
        assert np.array_equal(k, nk[l]) and np.array_equal(v, nv[l])       # layer l holds layer l's rows, nothing older
    orc.reset(None)
    orc.alloc(0)
    orc.append([0], [0, 1], nk[:, :1], nv[:, :1])
    assert list(orc.page_table(0)) == [0]
    with pytest.raises(OracleError):
        orc.reset([0, 0, 1, 2, 3, 4, 5, 6])
    assert orc.task_len(0) == 1 and orc.free_pages() == P - 1
