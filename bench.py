#!/usr/bin/env python
"""Benchmark of one CTB step (page append + mixed-batch attention) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl ours|reference]

A step = tide_kv_append of every row's new tokens + tide_attend of the whole batch, on a synthetic batch
shaped like the paper's workloads (see paper_2608_10402_b200/inputs.py).  Prints ONE JSON line.
`value` is the KV-read rate of the decode rows inside the mixed step (their KV bytes / the device time of
the decode-style kernel in that step); `append_prefill_tflops` is the other half of the metric (flops of
the resume rows / device time of the tile kernel).  Multi-GPU runs are independent replicas (tasks never
move between ranks): `--gpus N` started as a plain process launches itself N times under torch.distributed.run
(one rank per GPU); started under torch.distributed.run it takes its rank from the environment.
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
# dram bytes / algorithmic bytes of its launch (K and V of every resume row once + Q + O).
NCU_DECODE_TRAFFIC_RATIO = 1.012
NCU_UMMA_TRAFFIC_RATIO = 1155.1e6 / 1153.2e6     # one-pass capture of the full-size mixed batch
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
def rooflines(peaks, dec_bytes, dec_ms, res_flops, tile_ms, timed_ms, res_bytes):
    """The two roofline objects of a step: decode rows against the measured HBM copy rate (algorithmic KV bytes of
    the decode rows / device time of the decode-style kernel) and resume rows against the measured bf16 tensor rate
    (algorithmic flops / device time of the tile kernels; the burst peak unless the timed region is over a second)."""
    use_tensor = res_flops > 0 and tile_ms >= dec_ms
    sustained = timed_ms > 1000.0
    tpeak = peaks["bf16_tflops_sustained" if sustained else "bf16_tflops"]
    roof_tensor = {"bound": "tensor", "kernel": "attend tile kernel (resume rows)",
                   "achieved": res_flops / (tile_ms * 1e-3) / 1e12 if tile_ms > 0 else 0.0,
                   "peak": tpeak, "unit": "TFLOP/s", "traffic": res_bytes * NCU_UMMA_TRAFFIC_RATIO,
                   "traffic_note": "ncu dram read+write of one full-size launch / its algorithmic bytes (K,V of the resume rows once + Q + O), times this launch's algorithmic bytes (see profiles/)",
                   "peak_source": f"{peaks['_source']} ({'sustained' if sustained else 'burst'} bf16)"}
    roof_tensor["frac"] = roof_tensor["achieved"] / tpeak
    roof_hbm = {"bound": "hbm", "kernel": "attend decode kernel (decode rows)",
                "achieved": dec_bytes / (dec_ms * 1e-3) / 1e9 if dec_ms > 0 else 0.0,
                "peak": peaks["hbm_gbs"], "unit": "GB/s", "traffic": dec_bytes * NCU_DECODE_TRAFFIC_RATIO,
                "traffic_note": "ncu dram read+write of a reduced case / its algorithmic bytes, scaled (see profiles/)",
                "peak_source": f"{peaks['_source']} (copy)"}
    roof_hbm["frac"] = roof_hbm["achieved"] / peaks["hbm_gbs"]
    return use_tensor, roof_hbm, roof_tensor


def sample_rows(w, n_decode=12):
    """Batch rows whose values come from the workload's own seeded bits (the others are drawn on the device): a few
    decode rows and one resume row.  The CPU oracle computes exactly these rows, so its outputs check the timed run."""
    dec = [b for b in range(w.B) if w.n_new[b] == 1][:n_decode]
    res = [b for b in range(w.B) if w.n_new[b] > 1][:1]
    return dec + res


def build_state(w, torch, tide, seed, picked=(), tune=()):
    """Cache with every task's preserved prefix resident, plus this step's device inputs."""
    def dev_bits(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.bfloat16)

    total_q = int(w.n_new.sum())
    kv = tide.TideKV(w.Hq, w.Hkv, w.D, w.S, w.num_pages, w.max_tasks, w.max_pages_per_task,
                     max_batch_rows=w.B, max_batch_tokens=total_q, free_order=w.free_order)
    for knob, value in tune:
        kv.tune(knob, value)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    for b in range(w.B):
        kv.alloc(int(w.task[b]))
    bits = {b: (w.task_kv(b), w.task_q(b)) for b in picked}
    for b in range(w.B):
        p = int(w.prefix[b])
        if b in bits:
            k, v = dev_bits(bits[b][0][0][:p]), dev_bits(bits[b][0][1][:p])
        else:
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
    qoff = np.concatenate([[0], np.cumsum(w.n_new)])
    for b, ((kb, vb), qb) in bits.items():
        a, e, p = int(qoff[b]), int(qoff[b + 1]), int(w.prefix[b])
        new_k[a:e], new_v[a:e], q[a:e] = dev_bits(kb[p:]), dev_bits(vb[p:]), dev_bits(qb)
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
    picked = sample_rows(w) if rank == 0 else []
    tune = [tuple(int(x) for x in kvs.split("=")) for kvs in args.tune]
    kv, new_k, new_v, q, out, lse = build_state(w, torch, tide, seed=rank, picked=picked, tune=tune)
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
    parity_failed = False
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
    # what the last timed step left in `out` / `lse`, for the rows the CPU oracle will recompute
    qoff = np.concatenate([[0], np.cumsum(w.n_new)])
    _, sample_items = oracle_items(w, picked)
    sample_idx = torch.tensor([int(qoff[picked[r]]) + i for r, i in sample_items], dtype=torch.long, device="cuda")
    got_o = out[sample_idx].view(torch.int16).cpu().numpy().view(np.uint16) if picked else None
    got_l = lse[sample_idx].cpu().numpy() if picked else None

    # ---- timed region 2: the same steps with per-phase events (append / decode kernel / tile kernel / merge) ----
    kv.set_profiling(True)
    phases = {"append": [], "decode": [], "tile": [], "merge": []}
    for _ in range(args.steps):
        # two steps ahead of the measured one keep the device busy while the host enqueues it, so that the phase
        # events bracket device time only (after a synchronisation the host's own enqueue time would sit inside them)
        for _ in range(2):
            step()
            rollback()
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
        res_rows = w.n_new > 1
        res_bytes = int(w.kv_bytes_per_token() * int(w.ctx[res_rows].sum()) + int(w.n_new[res_rows].sum()) * w.Hq * w.D * 4)
        use_tensor, roof_hbm, roof_tensor = rooflines(peaks, dec_bytes, ph_ms["decode"], res_flops, ph_ms["tile"],
                                                      step_ms * args.steps, res_bytes)
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
                       "parallelism": f"replicas x{world}", "plan": plan, **({"tune": args.tune} if args.tune else {})},
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
        line["kv_read_gbs_with_merge"] = dec_bytes_all / ((dec_ms + mrg_ms) * 1e-3) / 1e9 if dec_ms + mrg_ms > 0 else 0.0
        base, ref_o, ref_l = cpu_baseline(w, picked, args.config, budget_s=args.cpu_budget)
        line["cpu_baseline"] = base
        line["parity_sample"] = parity_of_sample(got_o, got_l, ref_o, ref_l, len(sample_items))
        print(json.dumps(line))
        parity_failed = not line["parity_sample"]["within_tolerance"]
    kv.close()
    if world > 1:
        dist.destroy_process_group()
    if rank == 0 and parity_failed:
        raise SystemExit("bench.py: the timed run's outputs are outside the tolerance against the oracle")


# ---------------------------------------------------------------------------------------------------------
def oracle_items(w, picked, n_resume_q=48):
    """The (sample row, query) items the oracle computes: every decode row's query and n_resume_q evenly spaced
    queries of the resume row.  Returns the rows re-numbered as tasks 0.. of a small oracle cache, and the items."""
    rows, items = [], []
    for r, b in enumerate(picked):
        n = int(w.n_new[b])
        rows.append((r, n, int(w.ctx[b])))
        if n == 1:
            items.append((r, 0))
        else:
            items.extend((r, int(i)) for i in np.unique(np.linspace(0, n - 1, n_resume_q).astype(int)))
    return rows, items


def _oracle_sample(w, picked):
    """A bounded sample of the workload for the CPU oracle, with the sampled rows' whole contexts resident in an
    oracle cache (the same seeded bits the timed run holds for these rows)."""
    from oracle.paged_kv import PagedKVOracle
    pages = int(sum((int(w.ctx[b]) + w.S - 1) // w.S for b in picked)) + 4
    c = PagedKVOracle(pages, w.S, w.Hkv, w.D, max(len(picked), 1), w.max_pages_per_task,
                      free_order=np.random.default_rng(5).permutation(pages))
    rows, items = oracle_items(w, picked)
    qs = []
    for r, b in enumerate(picked):
        k, v = w.task_kv(b)
        c.alloc(r)
        c.append([r], [0, k.shape[0]], k, v)
        qs.append(w.task_q(b))
    kv_bytes = sum(w.kv_bytes_per_token() * (rows[r][2] - rows[r][1] + i + 1) for r, i in items)
    return c, rows, np.concatenate(qs), items, kv_bytes


def cpu_baseline(w, picked, config, budget_s=20.0):
    """The oracle as it stands, timed on this machine's host cores on a bounded sample of the workload.  Also returns
    the oracle's outputs for the sample, which are the expected values of the timed run's outputs for those rows."""
    from oracle import cbuild
    c, rows, q, items, kv_bytes = _oracle_sample(w, picked)
    t0 = time.perf_counter()
    reps = 0
    while True:
        ref_o, ref_l = cbuild.attend_paged(c, rows, q, w.scale, items=items, n_threads=host_threads())
        reps += 1
        dt = time.perf_counter() - t0
        if dt > budget_s * 0.5:
            break
    base = {"value": kv_bytes * reps / dt / 1e9, "unit": "GB/s", "cores": cbuild.threads(), "kind": "oracle",
            "sample": f"{len(items)} (row, query) items of configs[{config - 1}] ({sum(1 for r in rows if r[1] == 1)} decode rows + "
                      f"sampled queries of 1 resume row), KV bytes visible to each item / oracle seconds, {reps} passes",
            "seconds": dt}
    return base, ref_o, ref_l


def host_threads() -> int:
    """Cores this process may use (torch.distributed.run sets OMP_NUM_THREADS=1; the oracle leg runs on rank 0 alone
    while the other ranks idle, so it takes the cores the process is allowed)."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def parity_of_sample(got_bits, got_lse, ref_o, ref_lse, n_items, atol=1e-2, rtol=1e-2, lse_tol=1e-3, rel_fro_max=5e-3):
    """The timed run's outputs for the sampled rows against the oracle's: |gpu - oracle| <= atol + rtol |oracle|,
    LSE within lse_tol, relative Frobenius error within rel_fro_max (the tolerances of the parity tests)."""
    got = (got_bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    err = np.abs(got - ref_o)
    worst = float((err / (atol + rtol * np.abs(ref_o))).max())
    rel_fro = float(np.linalg.norm(got - ref_o) / max(np.linalg.norm(ref_o), 1e-300))
    lse_err = float(np.abs(got_lse.astype(np.float64) - ref_lse).max())
    ok = bool(np.isfinite(got).all() and worst <= 1.0 and lse_err <= lse_tol and rel_fro <= rel_fro_max)
    return {"items": int(n_items), "worst_ratio": worst, "lse_err": lse_err, "rel_fro": rel_fro, "within_tolerance": ok,
            "what": "outputs of the last timed step for the sampled rows vs the float64 oracle (the cpu_baseline leg's outputs)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import cbuild
    from paper_2608_10402_b200 import inputs
    w = inputs.make_workload(args.config, n_tasks=args.tasks, len_div=args.len_div, pool_factor=args.pool_factor)
    c, rows, q, items, kv_bytes = _oracle_sample(w, sample_rows(w))
    warmup = max(1, min(args.warmup, 2))
    steps = max(1, min(args.steps, 10))
    for _ in range(warmup):
        cbuild.attend_paged(c, rows, q, w.scale, items=items, n_threads=host_threads())
    t0 = time.perf_counter()
    for _ in range(steps):
        cbuild.attend_paged(c, rows, q, w.scale, items=items, n_threads=host_threads())
    dt = (time.perf_counter() - t0) / steps
    val = kv_bytes / dt / 1e9
    sample = f"each step = {len(items)} (row, query) items of configs[{args.config - 1}] through the float64 oracle"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"configs[{args.config - 1}]: {w.name}", "sample": sample,
                   "requested": {"steps": args.steps, "warmup": args.warmup},
                   "clamp": "the oracle arm runs at most 10 timed and 2 warm-up steps (each step is seconds of CPU work)"},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": cbuild.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---------------------------------------------------------------------------------------------------------
def run_long_horizon(args):
    """configs[4] as it is worded: a pool sized for ~150 GB of bf16 KV holds the state of ALL resident tasks (most
    of them paused), every step batches 256 of them (230 decode rows, 26 resume rows appending 500..4000 tokens), and
    between steps 26 tasks are released and as many new ones admitted into the freed pages.  Every timed step is a
    different batch.  K/V values are a reproducible integer hash of (task, position), so the rows the oracle
    recomputes need no copy of the pool."""
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
    HQ, HKV, D, S, XM, CAP = 28, 4, 128, 32, 1024, 128 * 1024
    free_b, _ = torch.cuda.mem_get_info()
    page_bytes = HKV * 2 * D * S * 2
    pool_bytes = min(args.resident_gb * 1e9, 0.85 * free_b - 8e9)
    num_pages = int(pool_bytes // page_bytes)
    rng = np.random.default_rng(replicas.rank_seed(1005, rank))

    def draw_len():
        return int(np.clip(round(XM * (1.0 - rng.random()) ** (-1.0 / 1.5)), XM, CAP))

    lens, used = [], 0
    while True:
        L = CAP if not lens else draw_len()
        if used + -(-L // S) > 0.9 * num_pages:
            break
        lens.append(L)
        used += -(-L // S)
    warmup, steps = max(args.warmup, 3), max(args.steps, 8)
    e2e_steps = 4
    n_steps_all = warmup + steps + e2e_steps
    max_tasks = len(lens) + n_steps_all * 32 + 8
    max_pages_per_task = -(-(CAP + 4000 + n_steps_all) // S) + 1
    max_batch_tokens = 230 + 26 * 4000
    kv = tide.TideKV(HQ, HKV, D, S, num_pages, max_tasks, max_pages_per_task, 256, max_batch_tokens,
                     free_order=rng.permutation(num_pages).astype(np.int32))

    def filler(task, start, count):
        return (inputs.hashed_bf16_bits_torch(torch, task, start, count, HKV, D, 0),
                inputs.hashed_bf16_bits_torch(torch, task, start, count, HKV, D, 1))

    def admit(task, L):
        kv.alloc(task, L)
        k, v = filler(task, 0, L)
        kv.append([task], [0, L], k, v)

    t0 = time.time()
    length = {}
    for t, L in enumerate(lens):
        admit(t, L)
        length[t] = L
    torch.cuda.synchronize()
    fill_s = time.time() - t0
    next_task = len(lens)
    scale = 1.0 / math.sqrt(D)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(rank)

    def make_batch():
        live = np.array(sorted(length))
        batch = rng.choice(live, size=256, replace=False)
        n_new = np.concatenate([np.ones(230, np.int64), rng.integers(500, 4001, size=26)])[rng.permutation(256)]
        n_new = np.array([min(int(n), max_pages_per_task * S - length[int(t)]) for t, n in zip(batch, n_new)])
        indptr = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
        total = int(indptr[-1])
        nk = torch.empty((total, HKV, D), dtype=torch.int16, device="cuda")
        nv = torch.empty_like(nk)
        for j, (t, n) in enumerate(zip(batch, n_new)):
            nk[indptr[j]:indptr[j + 1]], nv[indptr[j]:indptr[j + 1]] = filler(int(t), length[int(t)], int(n))
        q = torch.randn((total, HQ, D), device="cuda", generator=gen).to(torch.bfloat16)
        rows = [(int(t), int(n), length[int(t)] + int(n)) for t, n in zip(batch, n_new)]
        return batch, n_new, indptr, nk, nv, q, rows

    def churn(batch):
        """Release 26 tasks of the batch and admit as many new ones: their pages are handed out again at once."""
        nonlocal next_task
        for t in rng.choice(batch, size=26, replace=False):
            kv.release(int(t))
            del length[int(t)]
        for _ in range(26):
            L = draw_len()
            if -(-L // S) > kv.usage()[1]:
                continue
            admit(next_task, L)
            length[next_task] = L
            next_task += 1

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    kv.set_profiling(True)
    sampler = ClockSampler(local)
    sampler.start()
    tot = {"ms": 0.0, "append": 0.0, "decode": 0.0, "tile": 0.0, "merge": 0.0, "dec_bytes": 0.0, "flops": 0.0, "res_bytes": 0.0, "tokens": 0, "launches": 0}
    step_ms_list, last = [], None
    for it in range(warmup + steps):
        batch, n_new, indptr, nk, nv, q, rows = make_batch()
        out = torch.empty_like(q)
        lse = torch.empty((q.shape[0], HQ), dtype=torch.float32, device="cuda")
        if it == warmup:
            barrier()
            sampler.lines.clear()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        kv.append([int(t) for t in batch], indptr, nk, nv)
        kv.attend(rows, q, scale, out, lse)
        e1.record()
        torch.cuda.synchronize()
        ph = kv.phase_ms()
        for t, n in zip(batch, n_new):
            length[int(t)] += int(n)
        if it >= warmup:
            ms = e0.elapsed_time(e1)
            step_ms_list.append(ms)
            tot["ms"] += ms
            for k in ("append", "decode", "tile", "merge"):
                tot[k] += ph[k]
            tot["dec_bytes"] += HKV * D * 4 * sum(r[2] for r in rows if r[1] == 1)
            tot["flops"] += 4 * D * HQ * sum(r[1] * (r[2] - r[1]) + r[1] * (r[1] + 1) // 2 for r in rows if r[1] > 1)
            tot["res_bytes"] += sum(HKV * D * 4 * r[2] + r[1] * HQ * D * 4 for r in rows if r[1] > 1)
            tot["tokens"] += int(indptr[-1])
            tot["launches"] += kv.last_plan()["kernel_launches"]
            last = (rows, indptr, q, out, lse)
        churn(batch)
    barrier()
    clocks = sampler.stop()
    kv.set_profiling(False)
    assert kv.status() == tide.OK
    plan = kv.last_plan()

    # ---- the oracle's sample of the LAST timed step: three decode rows and sampled queries of one resume row ----
    parity, base = None, None
    if rank == 0:
        from oracle import cbuild
        from oracle.paged_kv import PagedKVOracle
        rows, indptr, q, out, lse = last
        picks = [j for j in range(256) if rows[j][1] == 1 and rows[j][2] <= 40000][:3] + [j for j in range(256) if rows[j][1] > 1][:1]
        val = PagedKVOracle(sum(-(-rows[j][2] // S) for j in picks) + 2, S, HKV, D, len(picks), max_pages_per_task)
        srows, sq, items, idx = [], [], [], []
        for r, j in enumerate(picks):
            t, n, L = rows[j]
            val.alloc(r)
            val.append([r], [0, L], inputs.hashed_bf16_bits(t, 0, L, HKV, D, 0), inputs.hashed_bf16_bits(t, 0, L, HKV, D, 1))
            srows.append((r, n, L))
            sq.append(q[int(indptr[j]):int(indptr[j + 1])].view(torch.int16).cpu().numpy().view(np.uint16))
            qs = [0] if n == 1 else sorted({int(i) for i in np.linspace(0, n - 1, 24)})
            items.extend((r, i) for i in qs)
            idx.extend(int(indptr[j]) + i for i in qs)
        sq = np.concatenate(sq)
        t0 = time.perf_counter()
        ref_o, ref_l = cbuild.attend_paged(val, srows, sq, scale, items=items, n_threads=host_threads())
        dt = time.perf_counter() - t0
        sel = torch.tensor(idx, dtype=torch.long, device="cuda")
        parity = parity_of_sample(out[sel].view(torch.int16).cpu().numpy().view(np.uint16), lse[sel].cpu().numpy(), ref_o, ref_l, len(items))
        vis = sum(HKV * D * 4 * (srows[r][2] - srows[r][1] + i + 1) for r, i in items)
        base = {"value": vis / dt / 1e9, "unit": "GB/s", "cores": cbuild.threads(), "kind": "oracle", "seconds": dt,
                "sample": f"{len(items)} (row, query) items of the last timed step (3 decode rows + sampled queries of 1 resume row), one pass"}

    # ---- end to end: further different steps through tide_step_host from pinned host buffers ----
    e2e_ms, h2d, d2h = 0.0, 0, 0
    for it in range(e2e_steps):
        batch, n_new, indptr, nk, nv, q, rows = make_batch()
        hk, hv, hq = nk.cpu().pin_memory(), nv.cpu().pin_memory(), q.cpu().pin_memory()
        hout = torch.empty(q.shape, dtype=q.dtype).pin_memory()
        hlse = torch.empty((q.shape[0], HQ), dtype=torch.float32).pin_memory()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        kv.step_host(rows, hk, hv, hq, scale, hout, hlse)
        dt = (time.perf_counter() - t0) * 1e3
        for t, n in zip(batch, n_new):
            length[int(t)] += int(n)
        if it > 0:                                            # the first one creates the copy streams
            e2e_ms += dt
            h2d += hk.numel() * 2 * 2 + hq.numel() * 2
            d2h += hout.numel() * 2 + hlse.numel() * 4
            e2e_dec = HKV * D * 4 * sum(r[2] for r in rows if r[1] == 1)
            tot.setdefault("e2e_dec_bytes", 0.0)
            tot["e2e_dec_bytes"] += e2e_dec
        churn(batch)
    n_e2e = e2e_steps - 1
    (step_ms, dec_ms, tile_ms, app_ms, mrg_ms, e2e_ms), (dec_bytes_all, flops_all, e2e_bytes_all) = replicas.reduce_step_stats(
        [tot["ms"], tot["decode"], tot["tile"], tot["append"], tot["merge"], e2e_ms],
        [tot["dec_bytes"], tot["flops"], tot["e2e_dec_bytes"]], world, dist, "cuda")
    if rank == 0:
        use_tensor, roof_hbm, roof_tensor = rooflines(peaks, tot["dec_bytes"], tot["decode"], tot["flops"], tot["tile"], tot["ms"],
                                                      tot["res_bytes"])
        line = {
            "metric": METRIC, "value": replicas.whole_job_rate(dec_bytes_all, dec_ms) / 1e9, "unit": "GB/s", "n_gpus": world,
            "steps": steps, "warmup": warmup, "ms_per_step": step_ms / steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "append_prefill_tflops": replicas.whole_job_rate(flops_all, tile_ms) / 1e12,
            "phase_ms": {"append": app_ms / steps, "decode_kernel": dec_ms / steps, "tile_kernel": tile_ms / steps, "merge": mrg_ms / steps},
            "append_gbs": 2 * HKV * D * 4 * tot["tokens"] / (tot["append"] * 1e-3) / 1e9 if tot["append"] > 0 else 0.0,
            "kv_read_gbs_with_merge": dec_bytes_all / ((dec_ms + mrg_ms) * 1e-3) / 1e9,
            "config": {"workload": "configs[4]: long-horizon stress batch, resident population (every timed step a different batch; "
                                   "26 tasks released and 26 admitted into the freed pages between steps)",
                       "pool_gb": num_pages * page_bytes / 1e9, "num_pages": num_pages, "residents": len(lens),
                       "fill_seconds": fill_s, "tasks": 256, "decode_rows": 230, "resume_rows": 26,
                       "new_tokens_per_step": tot["tokens"] / steps, "heads": f"{HQ}q/{HKV}kv", "head_dim": D, "page_size": S,
                       "step_ms": [round(x, 3) for x in step_ms_list], "l2": "inputs larger than L2 (no flush)",
                       "parallelism": f"replicas x{world}", "plan_of_last_step": plan},
            "roofline": roof_tensor if use_tensor else roof_hbm, "roofline_decode": roof_hbm, "roofline_prefill": roof_tensor,
            "e2e": {"value": e2e_bytes_all / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e2e_ms / n_e2e,
                    "definition": "decode-row KV bytes / whole host-buffer step (H2D new K,V,Q + append + attend + D2H out,lse)",
                    "h2d_bytes_per_step": int(h2d / n_e2e), "d2h_bytes_per_step": int(d2h / n_e2e)},
            "gpu_launches": int(tot["launches"]), "clocks": clocks, "cpu_baseline": base, "parity_sample": parity,
        }
        print(json.dumps(line))
    kv.close()
    if world > 1:
        dist.destroy_process_group()
    if rank == 0 and not parity["within_tolerance"]:
        raise SystemExit("bench.py: the timed run's outputs are outside the tolerance against the oracle")


def relaunch_as_replicas(n: int):
    """`--gpus N` from a plain process: the same command again under torch.distributed.run, one rank per GPU."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=3, help="workload 1..5 (configs[config-1]); default the mixed resume batch")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--tasks", type=int, default=None, help="fewer tasks (profiler captures only)")
    ap.add_argument("--len-div", type=int, default=1, help="divide every length bound (profiler captures only)")
    ap.add_argument("--pool-factor", type=float, default=None, help="pool pages / live pages (profiler captures only)")
    ap.add_argument("--layers", type=int, default=1,
                    help="> 1 adds a leg that steps this many layers over one page table (planned once, CUDA graph)")
    ap.add_argument("--cpu-budget", type=float, default=20.0, help="seconds of oracle time for cpu_baseline")
    ap.add_argument("--tune", action="append", default=[], metavar="KNOB=VALUE",
                    help="tide_tune setting for the handle, by the knob's number (see tide_tune_t); may be repeated")
    ap.add_argument("--resident-gb", type=float, default=0.0,
                    help="--config 5 only: GB of KV pool that holds a resident population (150 = the workload as quoted); every "
                         "timed step is then a different batch with releases and admissions in between.  0 = one fixed batch")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        relaunch_as_replicas(args.gpus)
    if args.impl == "reference":
        run_reference(args)
    elif args.config == 5 and args.resident_gb > 0:
        run_long_horizon(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
