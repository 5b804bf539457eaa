#!/usr/bin/env python
"""Benchmark of the decode-attention hot path: step plan + KV append + attention, per decode step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line.  A step is one decode step of the whole batch: every active thread appends
one token (pasta_step_begin + pasta_kv_append) and attends (pasta_decode_attn: tensor-core pass over
shared streams, warp-shuffle pass over private ones, merge).  Metric: thread-tokens per second
(one thread-token = one (request, thread) query through attention in every layer of the workload).

Workloads (synthetic, seeded; shapes of the five configurations):
  long_shared_prefix  8 requests x 32768-token prefix x 16 forks (chunks U[50,400]), 1 layer      [default]
  batched             64 requests, prefix U[256,2048], forks geometric, chunks U[10,300], 32 layers
  single_request      1 request, 768-token prefix, 4 forks, 1 layer (cache resident: a latency case)
  trace               synthetic interpreter trace (cfg5): 256 requests x 32 layers, promises / forks / syncs as they
                      come; every op of the trace is executed (step plan, append, attention, spawn, finish, sync merge);
                      --steps decode steps are timed after --warmup untimed ones (--size small: 64 requests x 8 layers)
With N > 1 (torchrun) every rank runs its own copy of the workload on its own GPU: requests are
independent, there is no exchange between ranks ("weak" scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "decode-attn thread-tokens/s"
UNIT = "thread-tokens/s"
NOMINAL_HBM_GBS = 8000.0
SEED_EXTRAS = 2502115
FALLBACK_HBM_GBS = 6650.0
# dram bytes (read + write) of one launch of the dominant kernel from an ncu capture of this workload,
# or None when no capture matches the current kernel
# Per-kernel events inside the timed region: a timing event between two kernels delays the second by a few microseconds
# (10 % of a 0.2 ms step with all four events on every step), so only every eighth step carries them.
PROFILE_STRIDE = 8
NCU_TRAFFIC_BYTES = {("long_shared_prefix", "full"): 1.2111e9, ("long_shared_prefix", "small"): 3.945e8}   # see profiles/


def make_script(workload: str, size: str = "full"):
    from pasta_workloads import cfg2_single_request, cfg3_batched, cfg4_long_prefix
    if workload == "long_shared_prefix":
        return cfg4_long_prefix() if size == "full" else cfg4_long_prefix(prefix=8192)
    if workload == "batched":
        return cfg3_batched() if size == "full" else cfg3_batched(n_layers=4)
    if workload == "single_request":
        script = cfg2_single_request("a")
        last = next(i for i, op in enumerate(script.ops) if op[0] == "step")
        script.ops = script.ops[:last + 1]          # step A: four forks and the main thread
        return script
    raise SystemExit(f"unknown workload {workload}")


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(device_index), f"--query-gpu=timestamp,{self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t0: float, t1: float):
        """Samples whose wall-clock time lies in [t0, t1] (the timed region); falls back to all samples."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        rows = []
        import datetime
        for line in open(self.file.name):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]), parts[4:9]))
            except Exception:
                continue
        os.unlink(self.file.name)
        inside = [r for r in rows if t0 <= r[0] <= t1]
        out["window"] = "timed region" if inside else "whole run (timed region shorter than the sampling period)"
        use = inside or rows
        if not use:
            return out
        out["samples"] = len(use)
        out["sm_mhz"] = float(np.median([r[1] for r in use]))
        out["sm_max_mhz"] = float(max(r[2] for r in use))
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        seen = set()
        for r in use:
            for name, flag in zip(names, r[3][1:]):
                if flag.lower().startswith("active"):
                    seen.add(name)
        out["reasons"] = sorted(seen)
        return out


# ------------------------------------------------------------------------------------------------ our arm
def build_state(script, device, seed_offset=0, grow_tokens=640, flags=0):
    """Replays the set-up part of the script (everything before its final step) with device-generated
    bf16 N(0,1) tensors.  Returns the pool and the final step's entries."""
    import torch
    from paper_2502_11517_b200 import binding
    geo = script.geometry
    # room for the tokens the benchmark appends: every entry may grow by up to `grow` tokens
    entries = list(script.ops[-1][1])
    grow_pages = len(entries) * (grow_tokens // 16 + 2)
    order = np.concatenate([script.free_order, np.arange(script.n_pages, script.n_pages + grow_pages, dtype=np.int32)])
    pool = binding.Pool(geo.n_layers, geo.n_q_heads, geo.n_kv_heads, geo.head_dim, script.n_pages + grow_pages,
                        script.max_requests, script.max_threads_per_request, script.max_segments_per_thread,
                        free_order=order, max_step_queries=len(entries), max_layers_per_launch=geo.n_layers,
                        flags=flags, device=device.index or 0)
    gen = torch.Generator(device=device)
    gen.manual_seed(script.seed + 977 * seed_offset)

    def randn(shape):
        return torch.randn(shape, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)

    for op in script.ops[:-1]:
        kind = op[0]
        if kind == "begin":
            assert pool.request_begin() == op[1]
        elif kind == "spawn":
            assert pool.thread_spawn(op[1]) == op[2]
        elif kind == "finish":
            pool.thread_finish(op[1], op[2])
        elif kind == "merge":
            pool.sync_merge(op[1], None if op[2] is None else list(op[2]))
        elif kind == "run":
            m = op[3]
            done = 0
            while done < m:                      # bounded transient memory for many-layer pools
                cnt = min(m - done, 4096)
                shape = (geo.n_layers, cnt, geo.n_kv_heads, geo.head_dim)
                pool.kv_append_run(op[1], op[2], cnt, randn(shape), randn(shape))
                done += cnt
        else:
            raise ValueError(kind)
    torch.cuda.synchronize(device)
    return pool, entries, randn


def build_state_naive_rows(script, device, seed_offset=0, grow_tokens=640):
    """The same set-up in the comparison layout of the paper's Appendix B: every thread a dense row of its own, the
    main thread's row duplicated into each fork's row at spawn (paper_2502_11517_b200/naive_rows.py).  Returns the
    pool, the final step's entries (one fork-less request per thread) and the bytes duplicated."""
    import torch
    from paper_2502_11517_b200 import binding
    from paper_2502_11517_b200.naive_rows import NaiveRows
    geo = script.geometry
    entries = list(script.ops[-1][1])
    n_rows = sum(op[0] in ("begin", "spawn") for op in script.ops)
    main_len, own_len = {}, {}
    for op in script.ops[:-1]:
        if op[0] == "run":
            (main_len if op[2] == 0 else own_len)[(op[1], op[2])] = (main_len if op[2] == 0 else own_len).get((op[1], op[2]), 0) + op[3]
    longest = max(main_len.values()) + max(own_len.values(), default=0) + grow_tokens + 32
    n_pages = n_rows * (longest // 16 + 2)
    pool = binding.Pool(geo.n_layers, geo.n_q_heads, geo.n_kv_heads, geo.head_dim, n_pages, n_rows, 1, 4,
                        max_step_queries=len(entries), max_layers_per_launch=geo.n_layers, device=device.index or 0)
    gen = torch.Generator(device=device)
    gen.manual_seed(script.seed + 977 * seed_offset)

    def randn(shape):
        return torch.randn(shape, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)

    rows = NaiveRows(pool)
    for op in script.ops[:-1]:
        kind = op[0]
        if kind == "begin":
            rows.begin(op[1])
        elif kind == "spawn":
            rows.spawn(op[1], op[2])
        elif kind == "finish":
            pass
        elif kind == "merge":
            rows.merge(op[1], [] if op[2] is None else list(op[2]))
        elif kind == "run":
            done = 0
            while done < op[3]:
                cnt = min(op[3] - done, 4096)
                shape = (geo.n_layers, cnt, geo.n_kv_heads, geo.head_dim)
                rows.run(op[1], op[2], cnt, randn(shape), randn(shape))
                done += cnt
        else:
            raise ValueError(kind)
    torch.cuda.synchronize(device)
    row_entries = [(rows.row[(req, t)], 0, n) for req, t, n in entries]
    return pool, row_entries, randn, rows.bytes_copied_at_spawn


def unique_tokens(pool, entries):
    """Per request, the union of what the step's threads see (a shared prefix counts once); and the part of
    it that the tensor-core kernel reads: everything, for requests whose stacked query rows fit one MMA tile."""
    dump = pool.dump()
    by_req = {}
    for req, t, _ in entries:
        by_req.setdefault(req, []).append(t)
    total = shared = 0
    for req, threads in by_req.items():
        seen = {}
        for t in threads:
            vis = {}
            for s, a, n in dump["requests"][req]["threads"][t]["view"]:
                vis[s] = max(vis.get(s, 0), a + n)
            for s, v in vis.items():
                seen.setdefault(s, []).append(v)
        on_tensor = (pool.head_dim == 128 and len(threads) * (pool.n_q_heads // pool.n_kv_heads) <= 128
                     and len(seen) <= 255)
        for s, vs in seen.items():
            total += max(vs)
            if on_tensor:
                shared += max(vs)
    return total, shared


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2502_11517_b200.build import build
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    if rank == 0:
        build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    script = make_script(args.workload, args.size)
    geo = script.geometry
    e2e_steps = max(3, min(args.steps, 50))
    grow = args.steps + max(args.warmup, 3) + e2e_steps + 3
    spawn_copy_bytes = None
    if args.layout == "naive_rows":
        pool, entries, randn, spawn_copy_bytes = build_state_naive_rows(script, device, seed_offset=rank, grow_tokens=grow)
    else:
        from paper_2502_11517_b200 import binding as _b
        pool, entries, randn = build_state(script, device, seed_offset=rank, grow_tokens=grow,
                                           flags=_b.FLAG_OUT_BF16 if args.out_dtype == "bf16" else 0)
    n = len(entries)
    reqs = np.asarray([e[0] for e in entries], dtype=np.int32); thr = np.asarray([e[1] for e in entries], dtype=np.int32)
    ones = np.ones(n, dtype=np.int32)
    L = geo.n_layers
    k_new = randn((L, n, geo.n_kv_heads, geo.head_dim)); v_new = randn((L, n, geo.n_kv_heads, geo.head_dim))
    q = randn((L, n, geo.n_q_heads, geo.head_dim))
    out_dtype = torch.bfloat16 if (args.out_dtype == "bf16" and args.layout == "pool") else torch.float32
    out = torch.empty(q.shape, dtype=out_dtype, device=device)
    stream = torch.cuda.current_stream(device)

    sh = stream.cuda_stream                   # the stream's handle, looked up once

    def step():                               # plan + append + attention of all layers, one library call
        pool.step_device(reqs, thr, ones, k_new, v_new, q, out, stream=sh)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize(device)
    tok0, shared0 = unique_tokens(pool, entries)
    launches0 = pool.launch_count()
    stride = min(PROFILE_STRIDE, max(1, args.steps // 4))      # short runs still get at least four timed steps
    pool.profile_enable(stride)
    sampler = ClockSampler(local) if rank == 0 else None
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(device)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    torch.cuda.synchronize(device)
    t_wall1 = time.time()
    if world > 1:
        dist.barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    kernel_ms, kernel_launches = pool.profile_read()
    pool.profile_enable(False)
    launches = pool.launch_count() - launches0
    tok1, shared1 = unique_tokens(pool, entries)
    assert pool.status() == 0, "a kernel reported an error"
    from paper_2502_11517_b200.sharding import aggregate
    all_tokens, worst_s = aggregate(float(n * args.steps), ms * 1e-3)    # every rank runs its own requests
    ms = worst_s * 1e3

    # ---- end to end: the same step through the host-buffer entry point (copies inside the timed region)
    k_h = k_new.cpu().pin_memory(); v_h = v_new.cpu().pin_memory(); q_h = q.cpu().pin_memory()
    out_h = torch.empty(q.shape, dtype=out_dtype).pin_memory()
    staging = torch.empty(pool.step_host_bytes(n), dtype=torch.uint8, device=device)
    for _ in range(3):
        pool.step_host(reqs, thr, ones, k_h, v_h, q_h, out_h, staging)
    torch.cuda.synchronize(device)
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        pool.step_host(reqs, thr, ones, k_h, v_h, q_h, out_h, staging)
    torch.cuda.synchronize(device)
    e2e_s = time.perf_counter() - t0
    e2e_tokens, e2e_s = aggregate(float(n * e2e_steps), e2e_s)
    h2d = k_h.numel() * 2 * 2 + q_h.numel() * 2
    d2h = out_h.numel() * out_h.element_size()

    # ---- host-only cost of a <sync/> merge (no kernel, no copy): a scratch pool with 16 finished forks
    merge_us = time_sync_merge()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    B_tok = geo.kv_bytes_per_token
    # unique KV bytes of the average step (every step adds one token per entry); all layers
    avg_tokens = (tok0 + tok1) / 2.0 + n / 2.0
    step_bytes = avg_tokens * B_tok * L
    shared_bytes = (shared0 + shared1) / 2.0 * B_tok * L      # what one tensor-core launch... per step
    peak, peak_kind = measured_peak()
    timed_steps = max(1, max(kernel_launches))                 # one launch of each kernel per step
    dom = 0 if kernel_launches[0] else 1                       # tensor-core kernel when the workload has shared streams
    dom_name = ["attn_tensor_kernel", "attn_warp_kernel"][dom]
    # the per-kernel events bracket every PROFILE_STRIDE-th step of the timed region, up to a bounded number of them,
    # and every step lengthens each stream by one token: bytes of the average step of the range they cover
    frac_timed = min(1.0, timed_steps * stride / max(1, args.steps))
    tok_p = tok0 + (tok1 - tok0) * frac_timed
    shared_p = shared0 + (shared1 - shared0) * frac_timed
    prof_step_bytes = ((tok0 + tok_p) / 2.0 + n / 2.0) * B_tok * L
    prof_shared_bytes = (shared0 + shared_p) / 2.0 * B_tok * L
    dom_bytes_per_launch = prof_shared_bytes if dom == 0 else prof_step_bytes - prof_shared_bytes
    dom_ms = kernel_ms[dom] / max(1, kernel_launches[dom])
    achieved = dom_bytes_per_launch / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 else 0.0
    value = all_tokens / (ms * 1e-3)
    step_gbs = step_bytes / (ms / args.steps * 1e-3) / 1e9
    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": args.workload, "size": args.size, "layout": args.layout, "out_dtype": args.out_dtype,
            "script": script.name, "requests": len(set(reqs)), "thread_tokens_per_step": n,
            "layers": L, "n_q_heads": geo.n_q_heads, "n_kv_heads": geo.n_kv_heads, "head_dim": geo.head_dim,
            "page_size": geo.page_size, "unique_kv_tokens_per_layer": avg_tokens,
            "unique_kv_bytes_per_step": step_bytes, "l2": "inputs larger than L2" if step_bytes / L > 126e6 * 1.5 else
            "working set fits L2 (latency case)",
            "step_hbm_gbs": step_gbs, "step_frac_of_measured_peak": step_gbs / peak,
            "step_frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS,
            "kernel_ms_per_step": {"tensor": kernel_ms[0] / timed_steps, "warp": kernel_ms[1] / timed_steps,
                                   "merge": kernel_ms[2] / timed_steps, "steps_timed": timed_steps,
                                   "every": stride},
            "sync_merge_host_us": merge_us,
            **({"bytes_duplicated_at_spawn": spawn_copy_bytes} if spawn_copy_bytes is not None else {}),
        },
        "clocks": clocks,
        "e2e": {"value": e2e_tokens / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "kernel": dom_name, "achieved": achieved, "peak": peak, "peak_kind": peak_kind,
                     "unit": "GB/s", "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                     "traffic": NCU_TRAFFIC_BYTES.get((args.workload, args.size)) if dom == 0 and args.layout == "pool" else None, "bytes_per_launch": dom_bytes_per_launch,
                     "ms_per_launch": dom_ms},
        "cpu_baseline": oracle_sample(args.workload, budget_s=20.0) if world == 1 and not args.no_cpu_baseline else None,
    }
    print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def unique_tokens_per_step(script):
    """Bookkeeping-only replay (a host-only pool): unique visible tokens of every step of a trace script."""
    from paper_2502_11517_b200 import binding
    geo = script.geometry
    pool = binding.Pool(1, geo.n_q_heads, geo.n_kv_heads, geo.head_dim, script.n_pages, script.max_requests,
                        script.max_threads_per_request, script.max_segments_per_thread, free_order=script.free_order,
                        flags=binding.FLAG_HOST_ONLY)
    lens, seen_by = {}, {}      # (req, stream) -> length; req -> set of streams somebody of the request can see
    out = []
    for op in script.ops:
        kind = op[0]
        if kind == "begin":
            pool.request_begin(); lens[(op[1], 0)] = 0; seen_by[op[1]] = {0}
        elif kind == "run":
            pool.kv_append_run(op[1], op[2], op[3]); lens[(op[1], op[2])] = lens.get((op[1], op[2]), 0) + op[3]
        elif kind == "spawn":
            pool.thread_spawn(op[1]); lens[(op[1], op[2])] = 0
        elif kind == "finish":
            pool.thread_finish(op[1], op[2])
        elif kind == "merge":
            pool.sync_merge(op[1], None if op[2] is None else list(op[2])); seen_by[op[1]].update(op[2] or [])
        elif kind == "step":
            total = 0
            reqs = {}
            for r, t, n in op[1]:
                lens[(r, t)] += n
                reqs.setdefault(r, set()).add(t)
            for r, ts in reqs.items():
                total += sum(lens[(r, st)] for st in (seen_by[r] | ts))
            out.append(total)
    pool.close()
    return out


def run_trace(args):
    import torch
    from paper_2502_11517_b200 import binding
    from paper_2502_11517_b200.build import build
    from paper_2502_11517_b200.sharding import aggregate
    from pasta_workloads import cfg5_trace
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0")); world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    if rank == 0:
        build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local)); dist.barrier()
    device = torch.device("cuda", local); torch.cuda.set_device(device)
    warm = max(args.warmup, 3)
    n_req, n_layers = (256, 32) if args.size == "full" else (64, 8)
    script = cfg5_trace(n_requests=n_req, n_steps=args.steps + warm, n_layers=n_layers)
    geo = script.geometry
    uniq = unique_tokens_per_step(script)
    max_n = max(len(op[1]) for op in script.ops if op[0] == "step")
    pool = binding.Pool(geo.n_layers, geo.n_q_heads, geo.n_kv_heads, geo.head_dim, script.n_pages, script.max_requests,
                        script.max_threads_per_request, script.max_segments_per_thread, free_order=script.free_order,
                        max_step_queries=max_n, max_layers_per_launch=geo.n_layers, device=local)
    gen = torch.Generator(device=device); gen.manual_seed(script.seed + 977 * rank)

    def randn(shape):
        return torch.randn(shape, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)

    L = geo.n_layers
    kv_pool = randn((L * max_n * geo.n_kv_heads * geo.head_dim,)); kv_pool2 = randn(kv_pool.shape)
    q_pool = randn((L * max_n * geo.n_q_heads * geo.head_dim,))
    out = torch.empty((L * max_n * geo.n_q_heads * geo.head_dim,), dtype=torch.float32, device=device)
    stream = torch.cuda.current_stream(device)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step_i = 0; tokens = 0; bytes_ = 0.0; merges = 0; host_s = 0.0
    t_wall0 = t_wall1 = None; sampler = None; launches0 = 0
    for op in script.ops:
        kind = op[0]
        if kind == "begin":
            assert pool.request_begin() == op[1]
        elif kind == "run":
            done = 0
            while done < op[3]:
                cnt = min(op[3] - done, 2048)
                shape = (L, cnt, geo.n_kv_heads, geo.head_dim)
                pool.kv_append_run(op[1], op[2], cnt, randn(shape), randn(shape)); done += cnt
        elif kind == "spawn":
            assert pool.thread_spawn(op[1]) == op[2]
        elif kind == "finish":
            pool.thread_finish(op[1], op[2])
        elif kind == "merge":
            pool.sync_merge(op[1], None if op[2] is None else list(op[2])); merges += step_i >= warm
        elif kind == "step":
            if step_i == warm:
                torch.cuda.synchronize(device)
                if world > 1:
                    dist.barrier()
                launches0 = pool.launch_count()
                pool.profile_enable(True)
                sampler = ClockSampler(local) if rank == 0 else None
                t_wall0 = time.time(); ev0.record(stream)
            n = len(op[1])
            h0 = time.perf_counter()
            pool.step_begin([e[0] for e in op[1]], [e[1] for e in op[1]], [e[2] for e in op[1]])
            host_s += (time.perf_counter() - h0) if step_i >= warm else 0.0
            kn = kv_pool[:L * n * geo.n_kv_heads * geo.head_dim]; vn = kv_pool2[:kn.numel()]
            pool.kv_append(kn, vn)
            pool.decode_attn(q_pool[:L * n * geo.n_q_heads * geo.head_dim], out)
            if step_i >= warm:
                tokens += n; bytes_ += uniq[step_i] * geo.kv_bytes_per_token * L
            step_i += 1
    ev1.record(stream); torch.cuda.synchronize(device); t_wall1 = time.time()
    if world > 1:
        dist.barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    launches = pool.launch_count() - launches0
    kernel_ms, kernel_launches = pool.profile_read()
    timed_calls = max(1, max(kernel_launches))
    assert pool.status() == 0, "a kernel reported an error"
    all_tokens, worst_s = aggregate(float(tokens), ms * 1e-3)
    if rank == 0:
        peak, peak_kind = measured_peak()
        gbs = bytes_ / (ms * 1e-3) / 1e9
        print(json.dumps({
            "metric": METRIC, "value": all_tokens / worst_s, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
            "ms_per_step": worst_s * 1e3 / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "trace", "size": args.size, "script": script.name, "requests": n_req, "layers": L,
                       "thread_tokens_timed": tokens, "max_thread_tokens_per_step": max_n, "sync_merges_timed": int(merges),
                       "pool_pages": script.n_pages, "pool_gb": script.n_pages * 65536 * L / 1e9,
                       "unique_kv_bytes_timed": bytes_, "l2": "inputs larger than L2",
                       "step_hbm_gbs": gbs, "step_frac_of_measured_peak": gbs / peak, "step_frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS,
                       "kernel_ms_per_step": {"tensor": kernel_ms[0] / timed_calls, "warp": kernel_ms[1] / timed_calls,
                                              "merge": kernel_ms[2] / timed_calls, "steps_timed": timed_calls},
                       "step_begin_call_ms": host_s * 1e3 / args.steps,
                       "step_begin_note": "wall time inside pasta_step_begin; includes waiting for the device when the host runs ahead"},
            "clocks": clocks, "e2e": None, "gpu_launches": launches,
            "roofline": {"bound": "hbm", "kernel": "whole step (tensor + warp + merge + append)", "achieved": gbs, "peak": peak,
                         "peak_kind": peak_kind, "unit": "GB/s", "frac": gbs / peak, "traffic": None},
            "cpu_baseline": None}))
    if world > 1:
        dist.destroy_process_group()


def run_extras(args):
    """Measurements of the steps around the decode path: rotary embedding fused into the append, the host
    interpreter's cost per step, a prompt fed in chunks of several tokens per step.  One JSON line; `value` is the
    chunked-prefill rate in thread-tokens/s (one query per prompt token)."""
    import torch
    from paper_2502_11517_b200 import binding
    from paper_2502_11517_b200.build import build
    from paper_2502_11517_b200.interpreter import Interpreter, Tags
    build()
    device = torch.device("cuda", 0); torch.cuda.set_device(device)
    gen = torch.Generator(device=device); gen.manual_seed(SEED_EXTRAS)

    def randn(shape):
        return torch.randn(shape, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)

    def timed(fn, reps):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        torch.cuda.synchronize(); ev[0].record(); [fn() for _ in range(reps)]; ev[1].record(); torch.cuda.synchronize()
        return ev[0].elapsed_time(ev[1]) / reps

    # ---- 1. append with and without the rotary embedding: 512 threads x 8 layers, one token each
    L, Hq, Hkv, d, n = 8, 32, 8, 128, 512
    pool = binding.Pool(L, Hq, Hkv, d, 4096, n, 1, 2, max_step_queries=n)
    reqs = [pool.request_begin() for _ in range(n)]
    for r in reqs:
        pool.kv_append_run(r, 0, 16, randn((L, 16, Hkv, d)), randn((L, 16, Hkv, d)))
    k, v = randn((L, n, Hkv, d)), randn((L, n, Hkv, d))
    append_us = {}
    for name, call in (("plain", lambda: pool.kv_append(k, v)), ("rope", lambda: pool.kv_append_rope(k, v, 10000.0))):
        def one():
            pool.step_begin(reqs, [0] * n, [1] * n)
            call()
        for _ in range(3):
            one()
        both = timed(one, 20)
        plan_only = timed(lambda: pool.step_begin(reqs, [0] * n, [0] * n), 20)
        append_us[name] = (both - plan_only) * 1e3
    append_bytes = 2 * L * n * Hkv * d * 2 * 2              # K and V, read and written
    pool.close()

    # ---- 2. the host interpreter alone (host-only pool): 64 responses of three forks each
    tags = Tags(1, 2, 3, 4)
    hp = binding.Pool(1, Hq, Hkv, d, 8192, 64, 8, 16, flags=binding.FLAG_HOST_ONLY, max_step_queries=512)
    it = Interpreter(hp, tags, predicted_length=lambda r, kk: 40)
    main = [1, 1, 1] + [50] * 40 + [4] + [51] * 8
    forks = {1: [60] * 30 + [3], 2: [61] * 45 + [3], 3: [62] * 20 + [3]}
    for _ in range(64):
        it.add_request(list(range(100, 400)))
    count = {}
    t0 = time.perf_counter(); steps = 0; fed = 0
    while steps < 60:
        entries = it.begin_step()
        nxt = []
        for req, t, _tok in entries:
            kk = count.get((req, t), 0); count[(req, t)] = kk + 1
            src = main if t == 0 else forks[t]
            nxt.append(src[kk] if kk < len(src) else 52)
        it.end_step(nxt)
        steps += 1; fed += len(entries)
    interp_s = time.perf_counter() - t0
    hp.close()

    # ---- 3. a prompt of 8192 tokens fed 32 tokens per step (128 stacked rows on the tensor-core path), 1 layer
    prompt, chunk = 8192, 32
    pool = binding.Pool(1, Hq, Hkv, d, 1024, 1, 1, 2, max_step_queries=chunk)
    r = pool.request_begin()
    kc, vc, qc = randn((1, chunk, Hkv, d)), randn((1, chunk, Hkv, d)), randn((1, chunk, Hq, d))
    out = torch.empty((1, chunk, Hq, d), dtype=torch.float32, device=device)

    def feed(m):
        pool.step_begin([r], [0], [m])
        pool.kv_append(kc[:, :m], vc[:, :m])
        pool.decode_attn(qc[:, :m], out[:, :m])

    for _ in range(4):
        feed(chunk)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_chunks = prompt // chunk - 4
    torch.cuda.synchronize(); ev0.record()
    for _ in range(n_chunks):
        feed(chunk)
    ev1.record(); torch.cuda.synchronize()
    chunk_ms = ev0.elapsed_time(ev1)
    pool.close()
    pool = binding.Pool(1, Hq, Hkv, d, 1024, 1, 1, 2, max_step_queries=chunk)
    r = pool.request_begin()
    for _ in range(8):
        feed(1)
    torch.cuda.synchronize(); ev0.record()
    for _ in range(512):
        feed(1)
    ev1.record(); torch.cuda.synchronize()
    single_ms = ev0.elapsed_time(ev1)
    assert pool.status() == 0
    pool.close()
    chunk_rate = n_chunks * chunk / (chunk_ms * 1e-3)
    print(json.dumps({
        "metric": METRIC, "value": chunk_rate, "unit": UNIT, "n_gpus": 1, "steps": n_chunks, "warmup": 4,
        "ms_per_step": chunk_ms / n_chunks, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": "extras",
                   "chunked_prefill": {"prompt_tokens": prompt, "tokens_per_step": chunk, "layers": 1,
                                       "thread_tokens_per_s": chunk_rate, "ms_per_step": chunk_ms / n_chunks,
                                       "one_token_per_step_thread_tokens_per_s": 512 / (single_ms * 1e-3),
                                       "one_token_per_step_ms": single_ms / 512},
                   "rope_append": {"threads": n, "layers": L, "plain_us": append_us["plain"], "rope_us": append_us["rope"],
                                   "bytes_moved": append_bytes,
                                   "rope_gbs": append_bytes / (append_us["rope"] * 1e-6) / 1e9},
                   "interpreter_host_only": {"responses": 64, "steps": steps, "thread_tokens_fed": fed,
                                             "us_per_step": interp_s / steps * 1e6,
                                             "thread_tokens_per_s": fed / interp_s}},
        "clocks": None, "e2e": None, "gpu_launches": None, "roofline": None, "cpu_baseline": None}))


def time_sync_merge():
    from paper_2502_11517_b200 import binding
    best = None
    for _ in range(5):
        pool = binding.Pool(1, 32, 8, 128, 4096, 1, 32, 64, flags=binding.FLAG_HOST_ONLY)
        r = pool.request_begin()
        pool.kv_append_run(r, 0, 768)
        forks = [pool.thread_spawn(r) for _ in range(16)]
        for t in forks:
            pool.kv_append_run(r, t, 100); pool.thread_finish(r, t)
        t0 = time.perf_counter()
        pool.sync_merge(r)
        dt = (time.perf_counter() - t0) * 1e6
        best = dt if best is None else min(best, dt)
        pool.close()
    return best


# ------------------------------------------------------------------------------------------------ oracle arm
_ORACLE_STATE = {}


def _oracle_state(workload: str):
    """The oracle replayed up to the workload's last step (bookkeeping and append done once), kept for reuse."""
    if workload in _ORACLE_STATE:
        return _ORACLE_STATE[workload]
    from oracle import OracleReplay
    from pasta_workloads import cfg2_single_request, cfg3_batched, cfg4_long_prefix, step_tensors
    if workload == "long_shared_prefix":
        script = cfg4_long_prefix(n_requests=1); passes = 4
        sample = "the 17 thread-tokens of 1 of 8 requests (32768-token prefix, 16 forks), 1 layer, 4 passes"
    elif workload == "batched":
        script = cfg3_batched(n_layers=1); passes = 8
        sample = "all thread-tokens of the 64 requests, 1 of 32 layers, 8 passes (time scaled by 32 layers)"
    else:
        script = cfg2_single_request("a"); script.ops = script.ops[:11]; passes = 50
        sample = "step A: 5 thread-tokens of the request, 1 layer, 50 passes"
    rep = OracleReplay(script)
    last = len(script.ops) - 1
    for i in range(last):
        rep.apply(i, attend=False)
    op = script.ops[last]
    k, v, q = step_tensors(script, last, 0)
    slots = [s for s in rep.model.reserve(op[1]) if s is not None]
    rep.stores[0].write(slots, k, v)
    queries = [(e[0], e[1]) for e in op[1]]
    _ORACLE_STATE[workload] = (rep, queries, q, sample, passes)
    return _ORACLE_STATE[workload]


def oracle_sample(workload: str, budget_s: float = 20.0, steps: int = 1):
    """Times the fp64 CPU oracle, as it stands, on a bounded sample of the workload: the queries of the
    workload's first request(s), in layer 0 (the attention is what is timed).  Returns the cpu_baseline object."""
    from oracle import decode_attention
    rep, queries, q, sample, passes = _oracle_state(workload)
    steps = max(steps, passes)
    times = []
    t_all = time.perf_counter()
    for _ in range(steps):
        t0 = time.perf_counter()
        done = 0
        for i, qq in enumerate(queries):
            decode_attention(rep.model, rep.stores[0], [qq], q[i:i + 1])
            done += 1
            if time.perf_counter() - t_all > budget_s:
                break
        times.append((time.perf_counter() - t0, done))
        if time.perf_counter() - t_all > budget_s:
            break
    dt = sum(t for t, _ in times); done = sum(d for _, d in times)
    layers = 32 if workload == "batched" else 1
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = 1
    return {"value": done / (dt * layers), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{done} thread-tokens: {sample}", "seconds": dt}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    t0 = time.perf_counter()
    _oracle_state(args.workload)                       # set-up once, outside the steps
    per_step = max(0.25, min(20.0, 150.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(args.workload, budget_s=per_step)
    res = [oracle_sample(args.workload, budget_s=per_step) for _ in range(args.steps)]
    secs = sum(r["seconds"] for r in res)
    done = sum(float(r["sample"].split()[0]) for r in res)
    layers = 32 if args.workload == "batched" else 1
    value = done / (secs * layers)
    base = dict(res[-1]); base["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs / max(1, args.steps) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload}, "cpu_baseline": base,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "wall_s": time.perf_counter() - t0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="long_shared_prefix")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--out-dtype", default="fp32", choices=["fp32", "bf16"],
                    help="type of the attention output (bf16 halves the device-to-host bytes of the end-to-end path)")
    ap.add_argument("--layout", default="pool", choices=["pool", "naive_rows"],
                    help="pool: the library's shared paged pool (default).  naive_rows: the comparison layout of the "
                         "paper's Appendix B (one dense row per thread, prefix duplicated), on the same kernels")
    ap.add_argument("--size", default="full", choices=["full", "small"],
                    help="small: a reduced copy of the workload for profiler captures (prefix 8192 / 4 layers)")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps == 200:
            args.steps, args.warmup = 3, 1
        run_reference(args)
    elif args.workload == "trace":
        run_trace(args)
    elif args.workload == "extras":
        run_extras(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
