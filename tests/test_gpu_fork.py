"""Group-shared prefix pages on the GPU against the oracle (tide_kv_fork, reference-counted pages, the private
copy an append takes before writing into a shared page).  A GRPO group rolls out G trajectories from one prompt
(paper Section 2.1) and CTB keeps the group on the rank that holds its shared prefix (end of Section 4)."""
import math

import numpy as np
import pytest

from oracle import cbuild
from oracle.paged_kv import OracleError, PagedKVOracle
from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu

HQ, HKV, D, S = 28, 4, 128, 16


def _same(kv, orc, tasks):
    for t in tasks:
        assert kv.task_len(t) == orc.task_len(t)
        assert np.array_equal(kv.page_table(t), orc.page_table(t)), f"page table of task {t}"
        assert np.array_equal(kv.page_refs(t), orc.page_refs(t)), f"reference counts of task {t}"
        gk, gv = kv.read(t)
        ok, ov = orc.read(t)
        assert np.array_equal(H.from_dev(gk), ok) and np.array_equal(H.from_dev(gv), ov), f"cache bits of task {t}"
    assert kv.usage() == (orc.used_tokens(), orc.free_pages())


def test_grpo_group_shares_its_prompt_pages():
    import torch
    from paper_2608_10402_b200 import tide
    rng = np.random.default_rng(77)
    P, G = 400, 8
    order = rng.permutation(P).astype(np.int32)
    kv = tide.TideKV(HQ, HKV, D, S, P, 16, 128, 16, 4096, free_order=order)
    orc = PagedKVOracle(P, S, HKV, D, 16, 128, free_order=order)
    scale = 1.0 / math.sqrt(D)
    # the prompt is prefilled once ...
    L0 = 1000 + 7                                            # ends inside a page: the partial page must be copied
    pk_, pv_ = inputs.normal_bf16(rng, (L0, HKV, D)), inputs.normal_bf16(rng, (L0, HKV, D))
    for o in (kv, orc):
        o.alloc(0)
    kv.append([0], [0, L0], H.to_dev(pk_, torch), H.to_dev(pv_, torch))
    orc.append([0], [0, L0], pk_, pv_)
    free_after_prompt = orc.free_pages()
    # ... and the other G-1 trajectories fork from it
    for c in range(1, G):
        kv.fork(0, c)
        orc.fork(0, c)
    assert orc.free_pages() == free_after_prompt - (G - 1)   # one copied page per child, nothing else
    _same(kv, orc, range(G))
    # every trajectory continues on its own: a first action (decode), then an observation of its own length
    for n_new in ([1] * G, [int(x) for x in rng.integers(20, 300, size=G)]):
        indptr = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
        T = int(indptr[-1])
        nk, nv, q = (inputs.normal_bf16(rng, (T, HKV, D)), inputs.normal_bf16(rng, (T, HKV, D)),
                     inputs.normal_bf16(rng, (T, HQ, D)))
        kv.append(list(range(G)), indptr, H.to_dev(nk, torch), H.to_dev(nv, torch))
        orc.append(list(range(G)), indptr, nk, nv)
        rows = [(t, n_new[t], orc.task_len(t)) for t in range(G)]
        out = torch.zeros((T, HQ, D), dtype=torch.int16, device="cuda")
        lse = torch.zeros((T, HQ), dtype=torch.float32, device="cuda")
        kv.attend(rows, H.to_dev(q, torch), scale, out, lse)
        assert kv.status() == tide.OK
        ref_o, ref_l = cbuild.attend_paged(orc, rows, q, scale)
        H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ref_o, ref_l, "group step")
        _same(kv, orc, range(G))
    # the prompt's pages survive until the last trajectory of the group is released
    shared = set(int(p) for p in orc.page_table(0)[: L0 // S])
    kv.release_many(list(range(G - 1)))
    orc.release_many(list(range(G - 1)))
    assert shared <= set(int(p) for p in orc.page_table(G - 1)) and not shared & set(orc.free)
    _same(kv, orc, [G - 1])
    kv.release(G - 1)
    orc.release(G - 1)
    assert kv.usage() == (0, P)
    kv.close()


def test_random_ops_with_forks_match_the_oracle_bit_for_bit():
    import torch
    from paper_2608_10402_b200 import tide
    rng = np.random.default_rng(5)
    P, NT = 96, 10
    order = rng.permutation(P).astype(np.int32)
    kv = tide.TideKV(8, 2, 64, 16, P, NT, 12, NT, 512, free_order=order)
    orc = PagedKVOracle(P, 16, 2, 64, NT, 12, free_order=order)
    codes = {"fork": 0, "append": 0, "truncate": 0, "release": 0, "errors": 0}
    for step in range(250):
        live = sorted(orc.live)
        r = rng.random()
        op = None
        if r < 0.15 or not live:
            t = int(rng.integers(0, NT))
            op = ("alloc", lambda o, t=t: o.alloc(t))
        elif r < 0.35:
            a, b = int(rng.choice(live)), int(rng.integers(0, NT))
            op = ("fork", lambda o, a=a, b=b: o.fork(a, b))
        elif r < 0.7:
            t, n = int(rng.choice(live)), int(rng.integers(0, 40))
            nk, nv = inputs.normal_bf16(rng, (n, 2, 64)), inputs.normal_bf16(rng, (n, 2, 64))
            op = ("append", lambda o, t=t, n=n, nk=nk, nv=nv: o.append([t], [0, n], *((H.to_dev(nk, torch), H.to_dev(nv, torch)) if o is kv else (nk, nv))))
        elif r < 0.85:
            t = int(rng.choice(live))
            nl = int(rng.integers(0, orc.task_len(t) + 1))
            op = ("truncate", lambda o, t=t, nl=nl: o.truncate(t, nl))
        else:
            t = int(rng.choice(live))
            op = ("release", lambda o, t=t: o.release(t))
        name, fn = op
        want = None
        try:
            fn(orc)
        except OracleError as e:
            want = e.code
        if want is None:
            fn(kv)
            codes[name] = codes.get(name, 0) + 1
        else:
            with pytest.raises(tide.TideError) as e:
                fn(kv)
            assert e.value.code == want, (name, e.value.code, want)
            codes["errors"] += 1
        if step % 10 == 9:
            _same(kv, orc, sorted(orc.live))
    _same(kv, orc, sorted(orc.live))
    assert codes["fork"] > 5 and codes["errors"] > 3, codes
    kv.close()


@pytest.mark.parametrize("geom", [(28, 4, 128, 16), (8, 2, 64, 16), (16, 1, 128, 32), (4, 4, 64, 32)])
def test_decode_rows_of_forked_groups_read_their_shared_pages_once(geom):
    """Groups of trajectories forked from one prompt, then decoding: the planner must treat each group's shared
    pages as one multi-query range (tide_last_sharing), and every row's result must still be plain attention over
    its whole context.  Group sizes around what one work item holds, members with and without tokens of their
    own, one unshared task in between, a context that ends inside the shared pages."""
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S = geom
    rng = np.random.default_rng(HQ + D + S)
    scale = 1.0 / math.sqrt(D)
    NT = 40
    kv = tide.TideKV(HQ, HKV, D, S, 2000, NT, 200, NT, 64)
    kv.tune(tide.TUNE_MIN_SAVED_BYTES, 0)      # small test batches: no minimum saving per batch
    orc = PagedKVOracle(2000, S, HKV, D, NT, 200)

    def app(ts, cnt):
        ip = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
        T = int(ip[-1])
        k, v = inputs.normal_bf16(rng, (T, HKV, D)), inputs.normal_bf16(rng, (T, HKV, D))
        kv.append(ts, ip, H.to_dev(k, torch), H.to_dev(v, torch))
        orc.append(ts, ip, k, v)

    task = 0
    rows_tasks = []
    for prompt, members, own in [(1500, 8, True), (700, 3, True), (4 * S * 16, 12, False), (300, 2, True)]:
        lead = task
        for o in (kv, orc):
            o.alloc(lead)
        app([lead], [prompt])
        ids = [lead]
        for _ in range(members - 1):
            task += 1
            kv.fork(lead, task)
            orc.fork(lead, task)
            ids.append(task)
        task += 1
        if own:
            app(ids, [int(rng.integers(1, 90)) for _ in ids])      # every trajectory continues on its own
        rows_tasks += ids
        if members == 3:                                            # an unshared task between two groups
            for o in (kv, orc):
                o.alloc(task)
            app([task], [900])
            rows_tasks.append(task)
            task += 1
    # one decode step: every task appends a token
    app(rows_tasks, [1] * len(rows_tasks))
    rows = [(t, 1, orc.task_len(t)) for t in rows_tasks]
    q = inputs.normal_bf16(rng, (len(rows), HQ, D))
    out = torch.zeros((len(rows), HQ, D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((len(rows), HQ), dtype=torch.float32, device="cuda")
    kv.attend(rows, H.to_dev(q, torch), scale, out, lse)
    assert kv.status() == tide.OK
    ref_o, ref_l = cbuild.attend_paged(orc, rows, q, scale)
    H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ref_o, ref_l, f"grouped decode {geom}")
    sharing = kv.last_sharing()
    assert sharing["groups"] >= 3 and sharing["rows"] >= 8 + 3 + 4, sharing
    # a window that ends inside the shared pages, and windows shorter than the shared range, still come out right
    rows2 = [(t, 1, max(1, min(orc.task_len(t), int(rng.integers(1, 1600))))) for t in rows_tasks]
    kv.attend(rows2, H.to_dev(q, torch), scale, out, lse)
    assert kv.status() == tide.OK
    ref_o, ref_l = cbuild.attend_paged(orc, rows2, q, scale)
    H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ref_o, ref_l, f"grouped decode, windows {geom}")
    # with the caller's own page table there is no grouping, and the result is the same attention
    table = torch.zeros((NT, 200), dtype=torch.int32, device="cuda")
    for t in rows_tasks:
        pt = orc.page_table(t)
        table[t, :len(pt)] = torch.from_numpy(pt).cuda()
    kv.attend(rows, H.to_dev(q, torch), scale, out, lse, page_table=table)
    assert kv.last_sharing()["groups"] == 0
    ref_o, ref_l = cbuild.attend_paged(orc, rows, q, scale)
    H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ref_o, ref_l, f"own table {geom}")
    kv.close()


def test_step_planned_before_its_append_does_not_share_a_page_that_is_about_to_be_copied():
    """Forked tasks rolled back to one token short of a page edge INSIDE their shared pages, then stepped by one
    token through tide_step_begin: the step is planned before the tokens are appended, the append gives each such
    task a private copy of that last page, so the page must not be planned as part of the group's shared range -
    otherwise every member but the first would read the first member's new token instead of its own."""
    import torch
    from paper_2608_10402_b200 import tide
    rng = np.random.default_rng(2024)
    P = 200
    order = rng.permutation(P).astype(np.int32)
    kv = tide.TideKV(HQ, HKV, D, S, P, 8, 64, 8, 64, free_order=order)
    kv.tune(tide.TUNE_MIN_SAVED_BYTES, 0)
    orc = PagedKVOracle(P, S, HKV, D, 8, 64, free_order=order)
    scale = 1.0 / math.sqrt(D)
    L0 = 20 * S
    pk_, pv_ = inputs.normal_bf16(rng, (L0, HKV, D)), inputs.normal_bf16(rng, (L0, HKV, D))
    for o in (kv, orc):
        o.alloc(0)
    kv.append([0], [0, L0], H.to_dev(pk_, torch), H.to_dev(pv_, torch))
    orc.append([0], [0, L0], pk_, pv_)
    for c in (1, 2, 3):
        kv.fork(0, c)
        orc.fork(0, c)
    for c in (1, 2):                                         # 18 pages kept, the last one a shared page with one free slot
        kv.truncate(c, 18 * S - 1)
        orc.truncate(c, 18 * S - 1)
    tasks = [1, 2, 3, 0]
    rows = [(t, 1, orc.task_len(t) + 1) for t in tasks]
    nk, nv, q = (inputs.normal_bf16(rng, (4, HKV, D)), inputs.normal_bf16(rng, (4, HKV, D)), inputs.normal_bf16(rng, (4, HQ, D)))
    # make the new tokens matter: each task's own new key is the one its query likes best
    qf = inputs.bf16_bits_to_f32(q)
    for i in range(4):
        for g in range(HKV):
            nk[i, g] = inputs.f32_to_bf16_bits(qf[i, g * (HQ // HKV)] * 0.5)
    out = torch.zeros((4, HQ, D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((4, HQ), dtype=torch.float32, device="cuda")
    kv.step_begin(rows)
    kv.step_layer(0, H.to_dev(nk, torch), H.to_dev(nv, torch), H.to_dev(q, torch), scale, out, lse)
    assert kv.status() == tide.OK
    assert kv.last_sharing()["groups"] >= 1, "the case is meant to be planned as a sharing group"
    orc.append(tasks, np.arange(5), nk, nv)
    _same(kv, orc, tasks)
    ref_o, ref_l = cbuild.attend_paged(orc, rows, q, scale)
    H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ref_o, ref_l, "step over a rolled-back group")
    kv.close()
