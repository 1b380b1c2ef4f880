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


def test_fork_shares_full_pages_and_copies_the_partial_one():
    # hand trace, page size 4, pool of 8 handed out in order 0..7
    c = PagedKVOracle(8, 4, 1, 2, 4, 6)
    k = np.arange(40 * 2, dtype=np.uint16).reshape(40, 1, 2)
    v = k + np.uint16(1000)
    c.alloc(0)
    c.append([0], [0, 10], k[:10], v[:10])                 # pages [0,1,2], the last one partial (2 of 4 slots)
    c.fork(0, 1)                                           # child: shares 0,1; page 3 is a copy of page 2
    assert list(c.page_table(1)) == [0, 1, 3] and list(c.page_refs(1)) == [2, 2, 1]
    assert list(c.page_refs(0)) == [2, 2, 1] and c.free_pages() == 4
    assert np.array_equal(c.read(1)[0], k[:10]) and np.array_equal(c.read(1)[1], v[:10])
    # the two diverge: each appends into its own partial page, then takes fresh pages
    c.append([0, 1], [0, 3, 9], k[10:19], v[10:19])         # parent +3 (fills page 2, pops 4), child +6 (fills 3, pops 5)
    assert list(c.page_table(0)) == [0, 1, 2, 4] and list(c.page_table(1)) == [0, 1, 3, 5]
    assert np.array_equal(c.read(0)[0], np.concatenate([k[:10], k[10:13]]))
    assert np.array_equal(c.read(1)[0], np.concatenate([k[:10], k[13:19]]))
    # fork on a page boundary copies nothing
    c.truncate(1, 8)
    assert list(c.page_table(1)) == [0, 1] and c.free_stack_top_first()[:2] == [3, 5]
    c.fork(1, 2)
    assert list(c.page_table(2)) == [0, 1] and list(c.page_refs(2)) == [3, 3] and c.free_pages() == 4
    # releasing the parent keeps the shared pages alive; the last holder frees them, last page first
    c.release(0)
    assert c.free_stack_top_first()[:2] == [2, 4] and list(c.page_refs(1)) == [2, 2]
    c.release(1)
    c.release(2)
    assert c.free_pages() == 8 and c.free_stack_top_first()[:2] == [0, 1] and not c.ref


def test_append_into_a_shared_partial_page_takes_a_private_copy_first():
    c = PagedKVOracle(8, 4, 1, 2, 4, 6)
    k = np.arange(40 * 2, dtype=np.uint16).reshape(40, 1, 2)
    c.alloc(0)
    c.append([0], [0, 8], k[:8], k[:8])                    # pages [0,1], both full
    c.fork(0, 1)                                           # child shares both
    c.truncate(1, 6)                                       # child now ends INSIDE shared page 1
    assert list(c.page_table(1)) == [0, 1] and c.ref[1] == 2
    c.append([1], [0, 3], k[20:23], k[20:23])              # private copy of page 1 (pops 2), then one more page (3)
    assert list(c.page_table(1)) == [0, 2, 3] and c.ref[1] == 1 and c.ref[2] == 1
    assert np.array_equal(c.read(1)[0], np.concatenate([k[:6], k[20:23]]))
    assert np.array_equal(c.read(0)[0], k[:8])             # the parent still sees its own tokens 6 and 7
    # the extra page counts in the all-or-nothing check: 4 pages free, child 2 needs a copy + 4 new pages
    c.fork(0, 2)
    c.truncate(2, 5)
    before = c.state_hash()
    with pytest.raises(OracleError) as e:
        c.append([2], [0, 16], k[:16], k[:16])             # ceil(21/4) - 2 = 4 new pages + 1 copy = 5 > 4 free
    assert e.value.code == pk.ERR_NO_PAGES and c.state_hash() == before
    with pytest.raises(OracleError) as e:
        c.fork(0, 1)
    assert e.value.code == pk.ERR_TASK_EXISTS


def test_refcount_conservation_under_random_ops_with_forks():
    rng = np.random.default_rng(31)
    P, S = 48, 4
    c = PagedKVOracle(P, S, 1, 2, max_tasks=10, max_pages_per_task=12, free_order=rng.permutation(P))
    shadow = {}
    counter = 0
    for _ in range(600):
        r = rng.random()
        live = sorted(c.live)
        try:
            if r < 0.15:
                t = int(rng.integers(0, 10))
                c.alloc(t)
                shadow[t] = []
            elif r < 0.3 and live:
                a, b = int(rng.choice(live)), int(rng.integers(0, 10))
                c.fork(a, b)
                shadow[b] = list(shadow[a])
            elif r < 0.7 and live:
                t = int(rng.choice(live))
                n = int(rng.integers(0, 9))
                kk = (np.arange(n * 2, dtype=np.uint32) + counter).astype(np.uint16).reshape(n, 1, 2)
                counter += 2 * n
                c.append([t], [0, n], kk, kk ^ np.uint16(0xAAAA))
                shadow[t].extend(kk[i].copy() for i in range(n))
            elif r < 0.85 and live:
                t = int(rng.choice(live))
                nl = int(rng.integers(0, c.task_len(t) + 1))
                c.truncate(t, nl)
                shadow[t] = shadow[t][:nl]
            elif live:
                t = int(rng.choice(live))
                c.release(t)
                del shadow[t]
        except OracleError:
            pass
        held = {}
        for t in c.live:
            assert len(c.pages[t]) == -(-c.len[t] // S)
            for p in c.pages[t]:
                held[p] = held.get(p, 0) + 1
        assert held == c.ref, "reference counts disagree with the page tables"
        assert not set(held) & set(c.free) and len(held) + c.free_pages() == P
    for t in c.live:
        kk, _ = c.read(t)
        assert kk.shape[0] == len(shadow[t])
        for pos, row in enumerate(shadow[t]):
            assert np.array_equal(kk[pos], row)


def test_reset_flushes_everything_and_primes_the_stack_in_the_given_order():
    """Hand trace on the 6-page pool (page size 4): after a reset the pool behaves like a fresh one created with
    that order - pages come out as order[0], order[1], ... - whatever was resident before (the flush that follows
    a weight synchronisation, Section 5.2)."""
    def rows(n):
        k = np.arange(n * 2, dtype=np.uint16).reshape(n, 1, 2)
        return k, k + np.uint16(9)

    c = PagedKVOracle(6, 4, 1, 2, max_tasks=4, max_pages_per_task=6, free_order=[3, 0, 5, 1, 4, 2])
    for t in (0, 1):
        c.alloc(t)
    c.append([0, 1], [0, 9, 14], *rows(14))                  # 3 + 2 pages: [3, 0, 5] and [1, 4]
    c.fork(1, 2)                                             # shares page 1, copies the partial page 4 into page 2
    assert c.free_pages() == 0 and list(c.page_table(2)) == [1, 2]
    c.reset([2, 4, 0, 5, 1, 3])
    assert c.free_pages() == 6 and c.used_tokens() == 0 and c.ref == {} and c.live == {}
    assert c.free_stack_top_first() == [2, 4, 0, 5, 1, 3]
    for t in (0, 1, 2):
        with pytest.raises(OracleError) as e:                # every task is unknown afterwards
            c.task_len(t)
        assert e.value.code == pk.ERR_UNKNOWN_TASK
    c.alloc(1)
    c.alloc(0)
    c.append([1], [0, 5], *rows(5))
    assert list(c.page_table(1)) == [2, 4]
    c.append([0, 1], [0, 1, 5], *rows(5))                    # task 0 takes the next page, task 1 fills page 4 and takes one more
    assert list(c.page_table(0)) == [0] and list(c.page_table(1)) == [2, 4, 5]
    assert c.free_stack_top_first() == [1, 3]
    # same content as a fresh pool created with that order and given the same calls
    f = PagedKVOracle(6, 4, 1, 2, max_tasks=4, max_pages_per_task=6, free_order=[2, 4, 0, 5, 1, 3])
    f.alloc(1)
    f.alloc(0)
    f.append([1], [0, 5], *rows(5))
    f.append([0, 1], [0, 1, 5], *rows(5))
    assert f.state_hash() == c.state_hash()
    for t in (0, 1):
        assert all(np.array_equal(a, b) for a, b in zip(c.read(t), f.read(t)))
    # no order = identity: pages 0, 1, 2, ...
    c.reset()
    assert c.free_stack_top_first() == [0, 1, 2, 3, 4, 5]
    c.alloc(3)
    c.append([3], [0, 9], *rows(9))
    assert list(c.page_table(3)) == [0, 1, 2]
    # an order that is not a permutation is refused and changes nothing
    before = c.state_hash()
    for bad in ([0, 1, 2, 3, 4, 4], [0, 1, 2, 3, 4], [0, 1, 2, 3, 4, 6]):
        with pytest.raises(OracleError) as e:
            c.reset(bad)
        assert e.value.code == pk.ERR_INVALID_ARG
        assert c.state_hash() == before and c.task_len(3) == 9
