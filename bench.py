#!/usr/bin/env python
"""Benchmark of one CTB step (page append + mixed-batch attention) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl ours|reference]

A step = tide_kv_append of every row's new tokens + tide_attend of the whole batch, on a synthetic batch
shaped like the paper's workloads (see paper_2608_10402_b200/inputs.py).  Prints ONE JSON line.
`value` is the KV-read rate of the decode rows inside the mixed step (their KV bytes / the device time of
the decode-style kernel in that step); `append_prefill_tflops` is the other half of the metric (flops of
the resume rows / device time of the tile kernel).  Multi-GPU runs are independent replicas (tasks never
move between ranks), launched with torch.distributed.run.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "mixed resume batch: KV-read GB/s vs HBM peak; append-prefill TFLOP/s vs peak"
# DRAM traffic per unit of algorithmic work, from the ncu captures summarised under profiles/ (reduced cases,
# scaled by the units one launch processes): decode kernel dram bytes / algorithmic KV bytes; tcgen05 kernel
# dram bytes per flop of resume-row attention.
NCU_DECODE_TRAFFIC_RATIO = 1.011
NCU_UMMA_DRAM_BYTES_PER_FLOP = 348.6e6 / 863.8e9
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for name, val in zip(names, f[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------------------------------------
def build_state(w, torch, tide, seed):
    """Cache with every task's preserved prefix resident, plus this step's device inputs."""
    total_q = int(w.n_new.sum())
    kv = tide.TideKV(w.Hq, w.Hkv, w.D, w.S, w.num_pages, w.max_tasks, w.max_pages_per_task,
                     max_batch_rows=w.B, max_batch_tokens=total_q, free_order=w.free_order)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    for b in range(w.B):
        kv.alloc(int(w.task[b]))
    for b in range(w.B):
        p = int(w.prefix[b])
        k = torch.randn((p, w.Hkv, w.D), device="cuda", generator=gen).to(torch.bfloat16)
        v = torch.randn((p, w.Hkv, w.D), device="cuda", generator=gen).to(torch.bfloat16)
        kv.append([int(w.task[b])], [0, p], k, v)
    torch.cuda.synchronize()
    sig = torch.ones((total_q, 1, 1), device="cuda")
    off = 0
    for b in range(w.B):            # image tokens of a multimodal chunk: K/V ~ N(0, 1.5)
        ni = int(w.n_image[b])
        if ni:
            sig[off:off + ni] = w.image_sigma
        off += int(w.n_new[b])
    new_k = (torch.randn((total_q, w.Hkv, w.D), device="cuda", generator=gen) * sig).to(torch.bfloat16)
    new_v = (torch.randn((total_q, w.Hkv, w.D), device="cuda", generator=gen) * sig).to(torch.bfloat16)
    q = torch.randn((total_q, w.Hq, w.D), device="cuda", generator=gen).to(torch.bfloat16)
    out = torch.empty_like(q)
    lse = torch.empty((total_q, w.Hq), device="cuda", dtype=torch.float32)
    return kv, new_k, new_v, q, out, lse


def multi_layer_leg(args, w, torch, tide, seed):
    """The same step over `--layers` K/V stores (one per model layer) that share one page table: device time per
    layer when every layer is driven by its own write + attend calls (the work is planned once per layer), when
    the step is planned once (tide_step_begin) and every layer only launches kernels (tide_step_layer), and when
    those launches are replayed from a CUDA graph captured for this step."""
    L = args.layers
    total_q = int(w.n_new.sum())
    kv = tide.TideKV(w.Hq, w.Hkv, w.D, w.S, w.num_pages, w.max_tasks, w.max_pages_per_task, max_batch_rows=w.B,
                     max_batch_tokens=total_q, free_order=w.free_order, num_layers=L)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    for b in range(w.B):
        kv.alloc(int(w.task[b]))
    for b in range(w.B):
        p = int(w.prefix[b])
        k = torch.randn((p, w.Hkv, w.D), device="cuda", generator=gen).to(torch.bfloat16)
        v = torch.randn((p, w.Hkv, w.D), device="cuda", generator=gen).to(torch.bfloat16)
        kv.extend([int(w.task[b])], [0, p])
        for l in range(L):
            kv.write(l, [int(w.task[b])], [0, p], k, v)
    new_k = torch.randn((L, total_q, w.Hkv, w.D), device="cuda", generator=gen).to(torch.bfloat16)
    new_v = torch.randn((L, total_q, w.Hkv, w.D), device="cuda", generator=gen).to(torch.bfloat16)
    q = torch.randn((L, total_q, w.Hq, w.D), device="cuda", generator=gen).to(torch.bfloat16)
    out = torch.empty_like(q)
    lse = torch.empty((L, total_q, w.Hq), device="cuda", dtype=torch.float32)
    rows = tide.rows_array(w.rows())
    ids = np.asarray(w.task, dtype=np.int32)
    indptr = np.concatenate([[0], np.cumsum(w.n_new)]).astype(np.int32)
    order_back = [(int(w.task[b]), int(w.prefix[b])) for b in reversed(range(w.B))]
    stream = torch.cuda.Stream()

    def rollback():
        for t, p in order_back:
            kv.truncate(t, p)

    def per_layer_calls():
        kv.extend(ids, indptr, stream=stream)
        for l in range(L):
            kv.write(l, ids, indptr, new_k[l], new_v[l], stream=stream)
            kv.attend(rows, q[l], w.scale, out[l], lse[l], layer=l, stream=stream)

    def planned():
        kv.step_begin(rows, stream=stream)
        for l in range(L):
            kv.step_layer(l, new_k[l], new_v[l], q[l], w.scale, out[l], lse[l], stream=stream)

    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        kv.step_begin(rows, stream=stream)
        t0 = time.perf_counter()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for l in range(L):
                kv.step_layer(l, new_k[l], new_v[l], q[l], w.scale, out[l], lse[l], stream=torch.cuda.current_stream())
        capture_ms = (time.perf_counter() - t0) * 1e3
        rollback()

        def from_graph():
            kv.step_begin(rows, stream=stream)      # the same rows give the same plan at the same place
            graph.replay()

        res = {}
        for name, fn in (("per_layer_calls", per_layer_calls), ("planned", planned), ("graph", from_graph)):
            for _ in range(3):
                fn()
                rollback()
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.steps):
                fn()
                rollback()
            e1.record(stream)
            stream.synchronize()
            host = []
            for _ in range(args.steps):          # host time to enqueue one step on an idle stream
                t0 = time.perf_counter()
                fn()
                host.append((time.perf_counter() - t0) * 1e3)
                rollback()
                stream.synchronize()
            res[name] = {"device_ms_per_layer": e0.elapsed_time(e1) / args.steps / L,
                         "host_enqueue_ms_per_step": float(np.median(host))}
        # the same with launch shapes fixed at twice what this step plans: ONE graph then serves every later step
        # whose plan stays below those maxima (surplus thread blocks leave at once)
        kv.step_begin(rows, stream=stream)
        pl = kv.last_plan()
        rollback()
        n_dec = sum(1 for (_, n, _) in w.rows() if n * (w.Hq // w.Hkv) <= 16)
        kv.step_fix_grids(max_decode_items=2 * pl["decode_items"] + 64,
                          max_tile_items=0 if w.D == 128 else 2 * pl["prefill_items"] + 64,
                          max_umma_items=2 * pl["prefill_items"] + 64 if w.D == 128 and n_dec < w.B else 0,
                          max_merge_rows=min(2 * pl["merge_rows"] + 64, total_q * w.Hq), max_tokens=total_q)
        kv.step_begin(rows, stream=stream)
        graph2 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph2, stream=stream):
            for l in range(L):
                kv.step_layer(l, new_k[l], new_v[l], q[l], w.scale, out[l], lse[l], stream=torch.cuda.current_stream())
        rollback()

        def from_fixed_graph():
            kv.step_begin(rows, stream=stream)
            graph2.replay()

        for _ in range(3):
            from_fixed_graph()
            rollback()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            from_fixed_graph()
            rollback()
        e1.record(stream)
        stream.synchronize()
        res["graph_fixed_shapes"] = {"device_ms_per_layer": e0.elapsed_time(e1) / args.steps / L}
        assert kv.status(stream=stream) == tide.OK
    kv.close()
    return {"layers": L, "graph_capture_ms": capture_ms, **res}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2608_10402_b200 import inputs, replicas, tide

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()

    w = inputs.make_workload(args.config, seed=replicas.rank_seed(1000 + args.config, rank), n_tasks=args.tasks, len_div=args.len_div,
                              pool_factor=args.pool_factor)
    kv, new_k, new_v, q, out, lse = build_state(w, torch, tide, seed=rank)
    rows = tide.rows_array(w.rows())
    ids = np.asarray(w.task, dtype=np.int32)
    indptr = np.concatenate([[0], np.cumsum(w.n_new)]).astype(np.int32)
    order_back = [(int(w.task[b]), int(w.prefix[b])) for b in reversed(range(w.B))]

    def step():
        kv.append(ids, indptr, new_k, new_v)
        kv.attend(rows, q, w.scale, out, lse)

    def rollback():
        for t, p in order_back:       # host only: every task back to its prefix, pages return in LIFO order
            kv.truncate(t, p)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
        rollback()
    assert kv.status() == tide.OK
    launches_per_step = kv.last_plan()["kernel_launches"]
    plan = kv.last_plan()

    # ---- timed region 1: K whole steps, device time ----
    barrier()
    sampler.lines.clear()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step()
        rollback()
    ev1.record()
    barrier()
    step_ms = ev0.elapsed_time(ev1) / args.steps

    # ---- timed region 2: the same steps with per-phase events (append / decode kernel / tile kernel / merge) ----
    kv.set_profiling(True)
    phases = {"append": [], "decode": [], "tile": [], "merge": []}
    for _ in range(args.steps):
        step()
        ph = kv.phase_ms()
        rollback()
        for k in phases:
            phases[k].append(ph[k])
    kv.set_profiling(False)
    clocks = sampler.stop()
    ph_ms = {k: float(np.mean(v)) for k, v in phases.items()}
    assert kv.status() == tide.OK

    # ---- timed region 3: end to end from pinned HOST buffers through tide_step_host ----
    hk, hv, hq = new_k.cpu().pin_memory(), new_v.cpu().pin_memory(), q.cpu().pin_memory()
    hout = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    hlse = torch.empty(lse.shape, dtype=lse.dtype).pin_memory()
    for _ in range(2):
        kv.step_host(rows, hk, hv, hq, w.scale, hout, hlse)
        rollback()
    barrier()
    e2e_steps = max(1, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        kv.step_host(rows, hk, hv, hq, w.scale, hout, hlse)
        rollback()
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps

    # ---- numbers ----
    dec_bytes = w.decode_kv_bytes()
    res_flops = w.resume_flops()
    (step_ms, dec_ms, tile_ms, app_ms, mrg_ms, e2e_ms), (dec_bytes_all, res_flops_all) = replicas.reduce_step_stats(
        [step_ms, ph_ms["decode"], ph_ms["tile"], ph_ms["append"], ph_ms["merge"], e2e_ms], [dec_bytes, res_flops],
        world, dist, "cuda")
    kv_gbs = replicas.whole_job_rate(dec_bytes_all, dec_ms) / 1e9
    tflops = replicas.whole_job_rate(res_flops_all, tile_ms) / 1e12

    multi_layer = None
    if args.layers > 1:
        kv.close()
        kv.pool = kv.workspace = None
        del new_k, new_v, q, out, lse
        torch.cuda.empty_cache()
        multi_layer = multi_layer_leg(args, w, torch, tide, seed=rank)

    if rank == 0:
        reduced = args.tasks is not None or args.len_div != 1 or args.pool_factor is not None
        n_app = int(w.n_new.sum())
        app_bytes = 2 * w.kv_bytes_per_token() * n_app
        use_tensor = res_flops > 0 and tile_ms >= dec_ms
        sustained = step_ms * args.steps > 1000.0
        tpeak = peaks["bf16_tflops_sustained" if sustained else "bf16_tflops"]
        roof_tensor = {"bound": "tensor", "kernel": "attend tile kernel (resume rows)",
                       "achieved": res_flops / (ph_ms["tile"] * 1e-3) / 1e12 if ph_ms["tile"] > 0 else 0.0,
                       "peak": tpeak, "unit": "TFLOP/s", "traffic": res_flops * NCU_UMMA_DRAM_BYTES_PER_FLOP,
                       "traffic_note": "dram read+write bytes of a reduced-case ncu capture scaled by flops (see profiles/)",
                       "peak_source": f"{peaks['_source']} ({'sustained' if sustained else 'burst'} bf16)"}
        roof_tensor["frac"] = roof_tensor["achieved"] / tpeak
        roof_hbm = {"bound": "hbm", "kernel": "attend decode kernel (decode rows)",
                    "achieved": dec_bytes / (ph_ms["decode"] * 1e-3) / 1e9 if ph_ms["decode"] > 0 else 0.0,
                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "traffic": dec_bytes * NCU_DECODE_TRAFFIC_RATIO,
                    "traffic_note": "ncu dram read+write of a reduced case / its algorithmic bytes, scaled (see profiles/)",
                    "peak_source": f"{peaks['_source']} (copy)"}
        roof_hbm["frac"] = roof_hbm["achieved"] / peaks["hbm_gbs"]
        line = {
            "metric": METRIC, "value": kv_gbs, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "append_prefill_tflops": tflops,
            "phase_ms": {"append": app_ms, "decode_kernel": dec_ms, "tile_kernel": tile_ms, "merge": mrg_ms},
            "append_gbs": app_bytes / (ph_ms["append"] * 1e-3) / 1e9 if ph_ms["append"] > 0 else 0.0,
            "config": {"workload": f"configs[{args.config - 1}]: {w.name}" + (" (REDUCED for a profiler capture)" if reduced else ""),
                       "tasks": w.B,
                       "decode_rows": int((w.n_new == 1).sum()), "resume_rows": int((w.n_new > 1).sum()),
                       "new_tokens": n_app, "prefix_tokens": int(w.prefix.sum()),
                       "heads": f"{w.Hq}q/{w.Hkv}kv", "head_dim": w.D, "page_size": w.S,
                       "decode_kv_bytes": dec_bytes, "resume_flops": res_flops,
                       "l2": "inputs larger than L2 (no flush)" if dec_bytes + app_bytes > 2 * 126e6 else "smaller than L2",
                       "parallelism": f"replicas x{world}", "plan": plan},
            "roofline": roof_tensor if use_tensor else roof_hbm,
            "roofline_decode": roof_hbm, "roofline_prefill": roof_tensor,
            "e2e": {"value": dec_bytes_all / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e2e_ms,
                    "definition": "decode-row KV bytes / whole host-buffer step (H2D new K,V,Q + append + attend + D2H out,lse)",
                    "h2d_bytes_per_step": int(hk.numel() * 2 * 2 + hq.numel() * 2),
                    "d2h_bytes_per_step": int(hout.numel() * 2 + hlse.numel() * 4)},
            "gpu_launches": int(launches_per_step * args.steps),
            "clocks": clocks,
        }
        if multi_layer is not None:
            line["multi_layer"] = multi_layer
        line["cpu_baseline"] = cpu_baseline(args.config, budget_s=args.cpu_budget)
        print(json.dumps(line))
    kv.close()
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------------------
def _oracle_sample(config, n_decode=12, n_resume_q=48):
    """A bounded sample of the workload for the CPU oracle: a few decode rows and a few queries of one
    resume row, with their whole contexts resident in an oracle cache."""
    from oracle.paged_kv import PagedKVOracle
    from paper_2608_10402_b200 import inputs
    w = inputs.make_workload(config)
    dec = [b for b in range(w.B) if w.n_new[b] == 1][:n_decode]
    res = [b for b in range(w.B) if w.n_new[b] > 1][:1]
    picked = dec + res
    pages = int(sum((int(w.ctx[b]) + w.S - 1) // w.S for b in picked)) + 4
    c = PagedKVOracle(pages, w.S, w.Hkv, w.D, w.max_tasks, w.max_pages_per_task,
                      free_order=np.random.default_rng(5).permutation(pages))
    rows, qs, items = [], [], []
    for r, b in enumerate(picked):
        k, v = w.task_kv(b)
        t = int(w.task[b])
        c.alloc(t)
        c.append([t], [0, k.shape[0]], k, v)
        rows.append(w.rows()[b])
        qs.append(w.task_q(b))
        n = int(w.n_new[b])
        if n == 1:
            items.append((r, 0))
        else:
            items.extend((r, int(i)) for i in np.linspace(0, n - 1, n_resume_q).astype(int))
    kv_bytes = sum(w.kv_bytes_per_token() * (rows[r][2] - rows[r][1] + i + 1) for r, i in items)
    return w, c, rows, np.concatenate(qs), items, kv_bytes


def cpu_baseline(config, budget_s=20.0):
    """The oracle as it stands, timed on this machine's host cores on a bounded sample of the workload."""
    from oracle import cbuild
    w, c, rows, q, items, kv_bytes = _oracle_sample(config)
    t0 = time.perf_counter()
    reps = 0
    while True:
        cbuild.attend_paged(c, rows, q, w.scale, items=items)
        reps += 1
        dt = time.perf_counter() - t0
        if dt > budget_s * 0.5:
            break
    return {"value": kv_bytes * reps / dt / 1e9, "unit": "GB/s", "cores": cbuild.threads(), "kind": "oracle",
            "sample": f"{len(items)} (row, query) items of configs[{config - 1}] ({sum(1 for r in rows if r[1] == 1)} decode rows + "
                      f"sampled queries of 1 resume row), KV bytes visible to each item / oracle seconds, {reps} passes",
            "seconds": dt}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import cbuild
    w, c, rows, q, items, kv_bytes = _oracle_sample(args.config)
    for _ in range(max(1, min(args.warmup, 2))):
        cbuild.attend_paged(c, rows, q, w.scale, items=items)
    steps = max(1, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(steps):
        cbuild.attend_paged(c, rows, q, w.scale, items=items)
    dt = (time.perf_counter() - t0) / steps
    val = kv_bytes / dt / 1e9
    sample = f"each step = {len(items)} (row, query) items of configs[{args.config - 1}] through the float64 oracle"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": steps, "warmup": max(1, min(args.warmup, 2)), "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"configs[{args.config - 1}]: {w.name}", "sample": sample},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": cbuild.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=3, help="BASELINE.json configs[config-1]; default the mixed resume batch")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--tasks", type=int, default=None, help="fewer tasks (profiler captures only)")
    ap.add_argument("--len-div", type=int, default=1, help="divide every length bound (profiler captures only)")
    ap.add_argument("--pool-factor", type=float, default=None, help="pool pages / live pages (profiler captures only)")
    ap.add_argument("--layers", type=int, default=1,
                    help="> 1 adds a leg that steps this many layers over one page table (planned once, CUDA graph)")
    ap.add_argument("--cpu-budget", type=float, default=20.0, help="seconds of oracle time for cpu_baseline")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
