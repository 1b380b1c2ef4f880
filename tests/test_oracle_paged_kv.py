"""Pins for the oracle's page allocator and paged store (CPU only)."""
import os

import numpy as np
import pytest

from oracle import paged_kv as pk
from oracle.paged_kv import OracleError, PagedKVOracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "allocator_trace.txt")
CODES = {"NO_PAGES": pk.ERR_NO_PAGES, "TABLE_FULL": pk.ERR_TABLE_FULL}


def _parse_state(text):
    tasks = {}
    text = text.strip()
    if text:
        for part in text.split(";"):
            t, ln, pages = part.strip().split(":")
            pages = pages.strip()[1:-1]
            tasks[int(t)] = (int(ln), [int(x) for x in pages.split(",")] if pages else [])
    return tasks


def _apply(c, op):
    kind, _, arg = op.partition(" ")
    if kind == "alloc":
        c.alloc(int(arg))
    elif kind == "release":
        c.release(int(arg))
    elif kind == "append":
        pairs = [p.split(":") for p in arg.split(",")]
        ids = [int(p[0]) for p in pairs]
        cnt = [int(p[1]) for p in pairs]
        indptr = np.concatenate([[0], np.cumsum(cnt)])
        T = int(indptr[-1])
        k = np.arange(T * c.Hkv * c.D, dtype=np.uint16).reshape(T, c.Hkv, c.D)
        c.append(ids, indptr, k, k + np.uint16(7))
    else:
        raise AssertionError(op)


def test_hand_traced_allocator_sequence():
    c = None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("pool"):
            _, P, S, order = line.split()
            c = PagedKVOracle(int(P), int(S), 1, 2, max_tasks=4, max_pages_per_task=6,
                              free_order=[int(x) for x in order.split(",")])
            continue
        op, tasks, free, used = [x.strip() for x in line.split("|")]
        if op.startswith("error"):
            _, code, rest = op.split(" ", 2)
            before = c.state_hash()
            with pytest.raises(OracleError) as e:
                _apply(c, rest)
            assert e.value.code == CODES[code]
            assert c.state_hash() == before
        else:
            _apply(c, op)
        want = _parse_state(tasks)
        assert set(c.live) == set(want)
        for t, (ln, pages) in want.items():
            assert c.task_len(t) == ln
            assert list(c.page_table(t)) == pages
        assert c.free_stack_top_first() == [int(x) for x in free.split(",")]
        assert c.used_tokens() == int(used)


def _random_ops(seed, steps=300):
    rng = np.random.default_rng(seed)
    P, S = 40, 4
    c = PagedKVOracle(P, S, 2, 4, max_tasks=8, max_pages_per_task=12, free_order=rng.permutation(P))
    shadow = {}  # task -> list of (k row, v row) appended so far: an independent record of logical content
    counter = 0
    for _ in range(steps):
        r = rng.random()
        live = sorted(c.live)
        try:
            if r < 0.2:
                t = int(rng.integers(0, 8))
                c.alloc(t)
                shadow[t] = []
            elif r < 0.75 and live:
                ids = list(rng.permutation(live)[: int(rng.integers(1, len(live) + 1))])
                cnt = rng.integers(0, 9, size=len(ids))
                indptr = np.concatenate([[0], np.cumsum(cnt)])
                T = int(indptr[-1])
                k = (np.arange(T * 8, dtype=np.uint32) + counter).astype(np.uint16).reshape(T, 2, 4)
                v = k ^ np.uint16(0x5555)
                counter += T * 8
                c.append(ids, indptr, k, v)
                for j, t in enumerate(ids):
                    for i in range(indptr[j], indptr[j + 1]):
                        shadow[int(t)].append((k[i].copy(), v[i].copy()))
            elif r < 0.85 and live:
                t = int(rng.choice(live))
                new_len = int(rng.integers(0, c.task_len(t) + 1))
                c.truncate(t, new_len)
                shadow[t] = shadow[t][:new_len]
            elif live:
                t = int(rng.choice(live))
                c.release(t)
                del shadow[t]
        except OracleError:
            pass
        yield c, shadow


def test_conservation_and_no_page_shared_under_random_ops():
    for c, _ in _random_ops(3):
        used = [p for t in c.live for p in c.pages[t]]
        assert len(used) == len(set(used)), "a page sits in two tables"
        assert not set(used) & set(c.free)
        assert len(used) + c.free_pages() == c.P
        for t in c.live:
            assert len(c.pages[t]) == -(-c.len[t] // c.S)


def test_logical_content_survives_any_op_sequence():
    last = None
    for c, shadow in _random_ops(11):
        last = (c, shadow)
    c, shadow = last
    assert c.live, "sequence ended with nothing resident; pick another seed"
    for t in c.live:
        k, v = c.read(t)
        assert k.shape[0] == len(shadow[t])
        for pos, (kr, vr) in enumerate(shadow[t]):
            assert np.array_equal(k[pos], kr) and np.array_equal(v[pos], vr)


def test_release_then_reappend_gets_same_pages():
    c = PagedKVOracle(16, 4, 1, 2, 4, 8, free_order=np.random.default_rng(0).permutation(16))
    c.alloc(0)
    z = np.zeros((13, 1, 2), np.uint16)
    c.append([0], [0, 13], z, z)
    pages = list(c.page_table(0))
    c.release(0)
    c.alloc(1)
    c.append([1], [0, 13], z, z)
    assert list(c.page_table(1)) == pages


def test_truncate_then_reappend_gets_same_pages():
    c = PagedKVOracle(16, 4, 1, 2, 4, 8, free_order=np.random.default_rng(1).permutation(16))
    c.alloc(0)
    z = np.zeros((13, 1, 2), np.uint16)
    c.append([0], [0, 13], z, z)
    pages = list(c.page_table(0))
    c.truncate(0, 6)           # keeps ceil(6/4) = 2 pages
    assert list(c.page_table(0)) == pages[:2] and c.task_len(0) == 6
    c.append([0], [0, 7], z[:7], z[:7])
    assert list(c.page_table(0)) == pages
    c.truncate(0, 0)
    assert list(c.page_table(0)) == [] and c.free_pages() == 16 and 0 in c.live


def test_incremental_appends_equal_bulk_append():
    rng = np.random.default_rng(5)
    k = rng.integers(0, 65536, size=(37, 2, 4)).astype(np.uint16)
    v = rng.integers(0, 65536, size=(37, 2, 4)).astype(np.uint16)
    a = PagedKVOracle(12, 4, 2, 4, 2, 12)
    a.alloc(0)
    a.append([0], [0, 37], k, v)
    b = PagedKVOracle(12, 4, 2, 4, 2, 12)
    b.alloc(0)
    off = 0
    for c in (1, 3, 4, 0, 9, 20):
        b.append([0], [0, c], k[off:off + c], v[off:off + c])
        off += c
    assert off == 37
    assert list(a.page_table(0)) == list(b.page_table(0))
    for x, y in zip(a.read(0), b.read(0)):
        assert np.array_equal(x, y)
    assert np.array_equal(a.read(0)[0], k) and np.array_equal(a.read(0)[1], v)


def test_every_error_leaves_state_unchanged():
    c = PagedKVOracle(3, 4, 1, 2, max_tasks=3, max_pages_per_task=2)
    z = np.zeros((16, 1, 2), np.uint16)
    c.alloc(0)
    c.alloc(1)
    c.append([0], [0, 3], z[:3], z[:3])

    def fails(code, fn):
        before = c.state_hash()
        with pytest.raises(OracleError) as e:
            fn()
        assert e.value.code == code
        assert c.state_hash() == before

    fails(pk.ERR_INVALID_ARG, lambda: c.alloc(3))
    fails(pk.ERR_INVALID_ARG, lambda: c.alloc(-1))
    fails(pk.ERR_TASK_EXISTS, lambda: c.alloc(0))
    fails(pk.ERR_NO_PAGES, lambda: c.alloc(2, reserve_tokens=9))    # 2 free pages * 4 = 8 < 9
    fails(pk.ERR_UNKNOWN_TASK, lambda: c.append([2], [0, 1], z[:1], z[:1]))
    fails(pk.ERR_DUPLICATE_TASK, lambda: c.append([0, 0], [0, 1, 2], z[:2], z[:2]))
    fails(pk.ERR_INVALID_ARG, lambda: c.append([0], [0, 2, 3], z[:3], z[:3]))
    fails(pk.ERR_INVALID_ARG, lambda: c.append([0, 1], [0, 2, 1], z[:1], z[:1]))
    fails(pk.ERR_TABLE_FULL, lambda: c.append([0], [0, 6], z[:6], z[:6]))          # 9 tokens -> 3 pages > 2
    fails(pk.ERR_NO_PAGES, lambda: c.append([0, 1], [0, 5, 13], z[:13], z[:13]))   # needs 1 + 2 pages, 2 free
    fails(pk.ERR_UNKNOWN_TASK, lambda: c.release(2))
    fails(pk.ERR_INVALID_ARG, lambda: c.truncate(0, 4))
    fails(pk.ERR_CTX_RANGE, lambda: c.check_rows([(0, 1, 4)]))
    fails(pk.ERR_CTX_RANGE, lambda: c.check_rows([(0, 0, 2)]))
    fails(pk.ERR_CTX_RANGE, lambda: c.check_rows([(0, 3, 2)]))
    c.alloc(2, reserve_tokens=8)   # exactly the headroom: admitted
    c.append([1], [0, 0], z[:0], z[:0])  # zero-length append is a no-op
    assert c.task_len(1) == 0 and list(c.page_table(1)) == []


def test_prune_keeps_prefix_and_tail_and_reuses_pages():
    # sliding-window pruning: tokens [0, keep) and [tail_begin, len) survive, in order, and the task ends up with
    # exactly the pages a task of the new length needs, the first of them unchanged
    rng = np.random.default_rng(17)
    c = PagedKVOracle(20, 4, 2, 4, 3, 12, free_order=rng.permutation(20))
    k = rng.integers(0, 65536, size=(30, 2, 4)).astype(np.uint16)
    v = rng.integers(0, 65536, size=(30, 2, 4)).astype(np.uint16)
    c.alloc(0)
    c.alloc(1)
    c.append([0], [0, 30], k, v)
    c.append([1], [0, 5], k[:5], v[:5])
    before = list(c.page_table(0))
    free_before = c.free_pages()
    c.prune(0, 6, 17)                      # drop positions 6..16
    gk, gv = c.read(0)
    assert c.task_len(0) == 6 + 13
    assert np.array_equal(gk, np.concatenate([k[:6], k[17:]])) and np.array_equal(gv, np.concatenate([v[:6], v[17:]]))
    assert list(c.page_table(0)) == before[:5]          # ceil(19 / 4) = 5 pages, the same ones in the same order
    assert c.free_pages() == free_before + 3
    assert np.array_equal(c.read(1)[0], k[:5])          # the neighbour is untouched
    c.prune(0, 19, 19)                                  # nothing dropped: no-op
    assert c.task_len(0) == 19
    c.prune(0, 0, 19)                                   # everything dropped
    assert c.task_len(0) == 0 and list(c.page_table(0)) == []
    with pytest.raises(OracleError):
        c.prune(1, 3, 2)
    c.release_many([0, 1])
    assert c.free_pages() == 20 and not c.live
    c.alloc(2)
    with pytest.raises(OracleError) as e:
        c.release_many([2, 2])
    assert e.value.code == pk.ERR_DUPLICATE_TASK and 2 in c.live
