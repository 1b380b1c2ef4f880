"""Random sequences of cache operations on a multi-layer cache against the layered oracle: alloc, fork, append
(extend + per-layer write), truncate, prune, release, on small pools so that pages are shared, copied on write, run
out and come back.  After every few operations page tables, reference counts, usage and the cache bits of every
layer are compared; every refusal must carry the oracle's error code.  The one refusal the oracle does not have
(a prune whose tail would have to be staged whole but exceeds max_batch_tokens) must be justified by the state."""
import math

import numpy as np
import pytest

from oracle import cbuild
from oracle.layers import LayeredKVOracle
from oracle.paged_kv import OracleError
from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _run(seed, n_ops, tide, torch):
    rng = np.random.default_rng(seed)
    L = int(rng.integers(1, 4)); S = int(rng.choice([16, 32])); HKV = 2; D = 64; HQ = 4
    P, NT, MAXP = 120, 10, 14
    CAP = int(rng.choice([24, 64, 512]))
    order = rng.permutation(P).astype(np.int32)
    kv = tide.TideKV(HQ, HKV, D, S, P, NT, MAXP, NT, CAP, free_order=order, num_layers=L)
    orc = LayeredKVOracle(L, num_pages=P, page_size=S, num_kv_heads=HKV, head_dim=D, max_tasks=NT, max_pages_per_task=MAXP, free_order=order)
    stats = {}
    def same(tasks):
        for t in tasks:
            assert kv.task_len(t) == orc.task_len(t), ("len", t)
            assert np.array_equal(kv.page_table(t), orc.page_table(t)), ("table", t)
            assert np.array_equal(kv.page_refs(t), orc.page_refs(t)), ("refs", t)
            for l in range(L):
                gk, gv = kv.read(t, layer=l); ok, ov = orc.read(l, t)
                assert np.array_equal(H.from_dev(gk), ok) and np.array_equal(H.from_dev(gv), ov), ("bits", l, t)
        assert kv.usage() == (orc.used_tokens(), orc.free_pages())
    for step in range(n_ops):
        live = sorted(orc.layer(0).live)
        r = rng.random()
        if r < 0.12 or not live:
            t = int(rng.integers(0, NT)); name = "alloc"
            fk = lambda: kv.alloc(t); fo = lambda: orc.alloc(t)
        elif r < 0.30:
            a, b = int(rng.choice(live)), int(rng.integers(0, NT)); name = "fork"
            fk = lambda: kv.fork(a, b); fo = lambda: orc.fork(a, b)
        elif r < 0.62:
            k = int(rng.integers(1, min(3, len(live)) + 1))
            ts = [int(x) for x in rng.choice(live, size=k, replace=False)]
            cnt = [int(rng.integers(0, 50)) for _ in ts]
            ip = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32); T = int(ip[-1])
            nk = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)]); nv = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
            name = "append"
            def fk():
                kv.extend(ts, ip)
                for l in range(L): kv.write(l, ts, ip, H.to_dev(nk[l], torch), H.to_dev(nv[l], torch))
            fo = lambda: orc.append(ts, ip, nk, nv)
        elif r < 0.72:
            t = int(rng.choice(live)); nl = int(rng.integers(0, orc.task_len(t) + 1)); name = "truncate"
            fk = lambda: kv.truncate(t, nl); fo = lambda: orc.truncate(t, nl)
        elif r < 0.90:
            t = int(rng.choice(live)); n = orc.task_len(t)
            a = int(rng.integers(0, n + 1)); b = int(rng.integers(a, n + 1)); name = "prune"
            fk = lambda: kv.prune(t, a, b); fo = lambda: orc.prune(t, a, b)
        else:
            t = int(rng.choice(live)); name = "release"
            fk = lambda: kv.release(t); fo = lambda: orc.release(t)
        try:
            fk(); ok = True
        except tide.TideError as e:
            ok = False; code = e.code
        if ok:
            fo()
            stats[name] = stats.get(name, 0) + 1
        elif code == tide.ERR_WORKSPACE and name == "prune":
            n = orc.task_len(t); pages = orc.page_table(t); refs = orc.page_refs(t)
            assert n - b > CAP and (refs[a // S:] > 1).any(), ("workspace refusal not justified", n, a, b, CAP, refs)
            stats["prune_ws"] = stats.get("prune_ws", 0) + 1
        else:
            try:
                fo(); raise AssertionError(f"{name}: library refused ({code}) what the oracle accepts")
            except OracleError as e:
                assert e.code == code, (name, e.code, code)
            stats["errors"] = stats.get("errors", 0) + 1
        if step % 7 == 6: same(sorted(orc.layer(0).live))
    same(sorted(orc.layer(0).live))
    assert kv.status() == tide.OK
    kv.close()
    return stats


def test_random_multi_layer_sequences_match_the_oracle():
    import torch
    from paper_2608_10402_b200 import tide
    total = {}
    for seed in range(8):
        for k, v in _run(seed, 220, tide, torch).items():
            total[k] = total.get(k, 0) + v
    assert total.get("prune", 0) > 100 and total.get("fork", 0) > 50 and total.get("errors", 0) > 100, total


def _run_steps(seed, n_ops, tide, torch):
    rng = np.random.default_rng(seed)
    L = int(rng.integers(1, 3)); S = int(rng.choice([16, 32])); D = int(rng.choice([64, 128]))
    HKV = int(rng.choice([1, 2, 4])); G = int(rng.choice([1, 4, 7, 8])); HQ = HKV * G
    P, NT, MAXP = 400, 8, 60
    order = rng.permutation(P).astype(np.int32)
    kv = tide.TideKV(HQ, HKV, D, S, P, NT, MAXP, 2 * NT, 4096, free_order=order, num_layers=L)
    # odd seeds: no minimum saving per batch, so that forked rows are planned as sharing groups whenever they can be
    kv.tune(tide.TUNE_MIN_SAVED_BYTES, 0 if seed % 2 else 64 << 20)
    orc = LayeredKVOracle(L, num_pages=P, page_size=S, num_kv_heads=HKV, head_dim=D, max_tasks=NT, max_pages_per_task=MAXP, free_order=order)
    scale = 1 / math.sqrt(D)
    n_att = 0
    for step in range(n_ops):
        live = sorted(orc.layer(0).live)
        r = rng.random()
        try:
            if r < 0.15 or not live:
                t = int(rng.integers(0, NT)); orc.alloc(t); kv.alloc(t)
            elif r < 0.30:
                a, b = int(rng.choice(live)), int(rng.integers(0, NT)); orc.fork(a, b); kv.fork(a, b)
            elif r < 0.60:
                k = int(rng.integers(1, min(4, len(live)) + 1))
                ts = [int(x) for x in rng.choice(live, size=k, replace=False)]
                cnt = [int(rng.choice([1, 1, int(rng.integers(2, 300))])) for _ in ts]
                ip = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32); T = int(ip[-1])
                nk = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)]); nv = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
                q = np.stack([inputs.normal_bf16(rng, (T, HQ, D)) for _ in range(L)])
                orc.append(ts, ip, nk, nv)       # raises first if it cannot be done
                rows = [(t, c, orc.task_len(t)) for t, c in zip(ts, cnt)]
                out = torch.zeros((L, T, HQ, D), dtype=torch.int16, device="cuda"); lse = torch.zeros((L, T, HQ), dtype=torch.float32, device="cuda")
                dk, dv, dq = H.to_dev(nk, torch), H.to_dev(nv, torch), H.to_dev(q, torch)
                kv.step_begin(rows)
                for l in range(L): kv.step_layer(l, dk[l], dv[l], dq[l], scale, out[l], lse[l])
                assert kv.status() == tide.OK
                for l in range(L):
                    ro, rl = cbuild.attend_paged(orc.layer(l), rows, q[l], scale)
                    H.check_outputs(H.from_dev(out[l]), lse[l].cpu().numpy(), ro, rl, f"seed {seed} step {step} layer {l}")
                n_att += 1
            elif r < 0.70:
                t = int(rng.choice(live)); nl = int(rng.integers(0, orc.task_len(t) + 1)); orc.truncate(t, nl); kv.truncate(t, nl)
            elif r < 0.85:
                t = int(rng.choice(live)); n = orc.task_len(t); a = int(rng.integers(0, n + 1)); b = int(rng.integers(a, n + 1))
                orc.prune(t, a, b); kv.prune(t, a, b)
            elif r < 0.93:
                # attention over arbitrary windows of live tasks (ctx_len below the resident length, a task twice)
                cand = [t for t in live if orc.task_len(t) > 0]
                if cand:
                    rows = []
                    for t in rng.choice(cand, size=min(len(cand), 5)):
                        n = orc.task_len(int(t)); c = int(rng.integers(1, n + 1)); ql = int(rng.integers(1, min(c, 200) + 1))
                        rows.append((int(t), ql, c))
                    l = int(rng.integers(0, L)); T = sum(r_[1] for r_ in rows)
                    q = inputs.normal_bf16(rng, (T, HQ, D))
                    out = torch.zeros((T, HQ, D), dtype=torch.int16, device="cuda"); lse = torch.zeros((T, HQ), dtype=torch.float32, device="cuda")
                    kv.attend(rows, H.to_dev(q, torch), scale, out, lse, layer=l)
                    assert kv.status() == tide.OK
                    ro, rl = cbuild.attend_paged(orc.layer(l), rows, q, scale)
                    H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ro, rl, f"seed {seed} step {step} windows")
                    n_att += 1
            else:
                t = int(rng.choice(live)); orc.release(t); kv.release(t)
        except OracleError:
            pass      # the oracle refused before the library was called: nothing happened on either side
        for t in sorted(orc.layer(0).live):
            assert kv.task_len(t) == orc.task_len(t) and np.array_equal(kv.page_table(t), orc.page_table(t)), (seed, step, t)
    kv.close()
    return n_att


def test_random_steps_and_windows_match_the_oracle():
    """Random geometries (head counts, head size, page size, layers); steps through tide_step_begin /
    tide_step_layer with decode and resume rows, attention over arbitrary windows of live tasks, interleaved with
    forks, truncates, prunes and releases; every attention result against the float64 oracle."""
    import torch
    from paper_2608_10402_b200 import tide
    checks = 0
    for seed in range(8):
        checks += _run_steps(seed, 80, tide, torch)
    assert checks > 100
