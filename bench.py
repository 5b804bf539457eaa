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
# The per-kernel events are kept out of the timed region (a timing event between two kernels holds the second back
# by a few microseconds): the kernels are timed in a loop of their own right after it, every launch, at least this many.
PROFILE_STEPS = 24
# DRAM bytes (read + write) of one launch of the tensor-core kernel from the ncu captures summarised under profiles/,
# as a ratio to the launch's algorithmic bytes (reads grow with the bytes read; the partial-row writes are added as
# they are).  Valid for the kernel source it was captured from only: its hash is checked at run time.
NCU_TRAFFIC = {"attn_tensor_sha256_16": "843a495e04b30a5e", "read_ratio": 1.0135, "write_bytes": 4.3e6}


def kernel_source_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in ("attn_tensor.cu", "device_common.cuh", "pasta_plan.h"):
        with open(os.path.join(ROOT, "paper_2502_11517_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


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
    """SM clock, power and throttle reasons of one GPU while a region runs: read through NVML from a thread of this
    process every millisecond or so (reading only; no setting is touched), or, without the NVML module, from an
    `nvidia-smi` child that samples every 20 ms."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        import threading
        self.rows = []          # (wall time, sm MHz, reasons bit mask, watts)
        self.now = lambda: None  # one reading taken by the caller's thread (NVML only)
        self.sm_max = None
        self.proc = self.file = self.thread = None
        self._stop = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            index = int(visible.split(",")[device_index]) if visible and visible.split(",")[device_index].isdigit() else device_index
            handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
            reasons = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or pynvml.nvmlDeviceGetCurrentClocksThrottleReasons

            def loop():
                while not self._stop.is_set():
                    try:
                        self.rows.append((time.time(), float(pynvml.nvmlDeviceGetClockInfo(handle, pynvml.NVML_CLOCK_SM)),
                                          int(reasons(handle)), pynvml.nvmlDeviceGetPowerUsage(handle) / 1000.0))
                    except Exception:
                        pass
                    time.sleep(0.001)

            def now():
                self.rows.append((time.time(), float(pynvml.nvmlDeviceGetClockInfo(handle, pynvml.NVML_CLOCK_SM)),
                                  int(reasons(handle)), pynvml.nvmlDeviceGetPowerUsage(handle) / 1000.0))

            self.now = now
            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
            self.how = "nvml: a thread about 1 ms apart, plus one reading as the region's last kernel ends"
        except Exception:
            self.how = "nvidia-smi, 20 ms apart"
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            try:
                self.proc = subprocess.Popen(
                    ["nvidia-smi", "-i", str(device_index), f"--query-gpu=timestamp,{self.QUERY}",
                     "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.file, stderr=subprocess.DEVNULL)
            except Exception:
                self.proc = None

    def _finish(self):
        if self.thread is not None:
            self._stop.set()
            self.thread.join(timeout=2)
            self.thread = None
        if self.proc is not None:
            import datetime
            time.sleep(0.05)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self.proc = None
            self.file.flush()
            bits = {v: k for k, v in self.REASONS.items()}
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            for line in open(self.file.name):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    mask = sum(bits[n] for n, flag in zip(names, parts[5:9]) if flag.lower().startswith("active"))
                    self.rows.append((ts, float(parts[1]), mask, float(parts[3])))
                    self.sm_max = max(self.sm_max or 0.0, float(parts[2]))
                except Exception:
                    continue
            os.unlink(self.file.name)

    def window(self, t0: float, t1: float):
        """Summary of the samples taken in [t0, t1] (wall clock); all samples so far when none fell inside."""
        out = {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "samples": 0, "how": self.how}
        rows = list(self.rows)
        inside = [r for r in rows if t0 <= r[0] <= t1]
        out["window"] = "timed region" if inside else "whole run (no sample fell inside the timed region)"
        use = inside or rows
        if not use:
            return out
        out["samples"] = len(use)
        out["sm_mhz"] = float(np.median([r[1] for r in use]))
        out["power_w"] = float(np.median([r[3] for r in use]))
        seen = set()
        for r in use:
            seen.update(name for bit, name in self.REASONS.items() if r[2] & bit)
        out["reasons"] = sorted(seen)
        return out

    def stop(self, t0: float, t1: float):
        self._finish()
        return self.window(t0, t1)


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


def unique_tokens(pool, entries, tensor=True):
    """Tokens of the step, three ways: (a) per request, the union of what the step's threads see (a shared prefix counts
    once); (b) the part of (a) that the tensor-core kernel reads: everything, for requests whose stacked query rows fit
    one MMA tile; (c) what the warp-shuffle kernel reads for the other requests: every query's own visible tokens,
    a shared prefix once per thread that sees it (that kernel shares nothing between queries)."""
    dump = pool.dump()
    by_req = {}
    for req, t, _ in entries:
        by_req.setdefault(req, []).append(t)
    total = shared = per_query = 0
    for req, threads in by_req.items():
        seen = {}
        for t in threads:
            vis = {}
            for s, a, n in dump["requests"][req]["threads"][t]["view"]:
                vis[s] = max(vis.get(s, 0), a + n)
            for s, v in vis.items():
                seen.setdefault(s, []).append(v)
        on_tensor = (tensor and pool.head_dim == 128 and len(threads) * (pool.n_q_heads // pool.n_kv_heads) <= 128
                     and len(seen) <= 4095)
        for s, vs in seen.items():
            total += max(vs)
            if on_tensor:
                shared += max(vs)
            else:
                per_query += sum(vs)
    return total, shared, per_query


def measure_steady(args, workload, size, steps, warmup, device, rank, world, local, *, layout="pool",
                   out_dtype_name="fp32", with_e2e=True, flags=0):
    """One workload whose step repeats (every entry appends a token and attends): builds the state, times `steps`
    steps after `warmup`, then times the kernels in a loop of their own and, if asked, the host-buffer path."""
    import torch
    import torch.distributed as dist
    from paper_2502_11517_b200 import binding as _b
    from paper_2502_11517_b200.sharding import aggregate
    script = make_script(workload, size)
    geo = script.geometry
    warmup = max(warmup, 3)
    prof_steps = PROFILE_STEPS
    e2e_steps = max(8, min(steps, 50)) if with_e2e else 0
    grow = steps + warmup + prof_steps + 2 * e2e_steps + 16
    spawn_copy_bytes = None
    if layout == "naive_rows":
        pool, entries, randn, spawn_copy_bytes = build_state_naive_rows(script, device, seed_offset=rank, grow_tokens=grow)
    else:
        pool, entries, randn = build_state(script, device, seed_offset=rank, grow_tokens=grow,
                                           flags=flags | (_b.FLAG_OUT_BF16 if out_dtype_name == "bf16" else 0))
    if getattr(args, "tail", None):
        pool.debug_set_tail(*[int(v) for v in args.tail.split(",")])
    n = len(entries)
    reqs = np.asarray([e[0] for e in entries], dtype=np.int32); thr = np.asarray([e[1] for e in entries], dtype=np.int32)
    ones = np.ones(n, dtype=np.int32)
    L = geo.n_layers
    k_new = randn((L, n, geo.n_kv_heads, geo.head_dim)); v_new = randn((L, n, geo.n_kv_heads, geo.head_dim))
    q = randn((L, n, geo.n_q_heads, geo.head_dim))
    out_dtype = torch.bfloat16 if (out_dtype_name == "bf16" and layout == "pool") else torch.float32
    out = torch.empty(q.shape, dtype=out_dtype, device=device)
    stream = torch.cuda.current_stream(device)
    sh = stream.cuda_stream                   # the stream's handle, looked up once

    def step():                               # plan + append + attention of all layers, one library call
        pool.step_device(reqs, thr, ones, k_new, v_new, q, out, stream=sh)

    sampler = ClockSampler(local) if rank == 0 else None      # started early: its first readings take a while
    for _ in range(warmup):
        step()
    torch.cuda.synchronize(device)
    on_tensor = not (flags & _b.FLAG_NO_TENSOR_PATH)
    tok0, _, _ = unique_tokens(pool, entries, on_tensor)
    launches0 = pool.launch_count()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(device)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    ev0.record(stream)
    for _ in range(steps):
        step()
    ev1.record(stream)
    torch.cuda.synchronize(device)
    if sampler:
        sampler.now()                         # the GPU was under load until a few microseconds ago
    t_wall1 = time.time()
    if world > 1:
        dist.barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.window(t_wall0, t_wall1) if sampler else None
    launches = pool.launch_count() - launches0
    tok1, shared1, warp1 = unique_tokens(pool, entries, on_tensor)
    all_tokens, worst_s = aggregate(float(n * steps), ms * 1e-3)    # every rank runs its own requests
    ms = worst_s * 1e3

    # ---- the kernels, timed one by one (events around every launch) in the steps that follow the timed region
    pool.profile_enable(1)
    t_prof0 = time.time()
    for _ in range(prof_steps):
        step()
    torch.cuda.synchronize(device)
    if sampler:
        sampler.now()
    t_prof1 = time.time()
    kernel_ms, kernel_launches = pool.profile_read()
    pool.profile_enable(False)
    prof_clocks = sampler.window(t_prof0, t_prof1) if sampler else None
    tok2, shared2, warp2 = unique_tokens(pool, entries, on_tensor)
    assert pool.status() == 0, "a kernel reported an error"

    # ---- what a read-only kernel gets on this GPU, same run: the pool's KV memory read by bulk copies and by loads
    ceilings = {}
    if layout == "pool" and pool.kv.numel() > 256e6:
        for name, mode in (("bulk_copy", 1), ("bulk_copy_scattered_8k", 2), ("vector_loads", 0)):
            for _ in range(2):
                nbytes = pool.debug_stream_read(None, mode, stream=sh)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = 8
            e0.record(stream)
            for _ in range(reps):
                pool.debug_stream_read(None, mode, stream=sh)
            e1.record(stream)
            torch.cuda.synchronize(device)
            ceilings[name] = nbytes * reps / (e0.elapsed_time(e1) * 1e-3) / 1e9
        assert pool.status() == 0

    # ---- end to end: the same step through the host-buffer entry points (copies inside the timed region)
    e2e = None
    if with_e2e:
        k_h = k_new.cpu().pin_memory(); v_h = v_new.cpu().pin_memory(); q_h = q.cpu().pin_memory()
        out_h = [torch.empty(q.shape, dtype=out_dtype).pin_memory() for _ in range(3)]
        staging = torch.empty(3 * pool.step_host_bytes(n), dtype=torch.uint8, device=device)
        for _ in range(3):
            pool.step_host(reqs, thr, ones, k_h, v_h, q_h, out_h[0], staging)
        torch.cuda.synchronize(device)
        if world > 1:
            dist.barrier()
        # (a) one step after the other, each waited for before the next begins
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            pool.step_host(reqs, thr, ones, k_h, v_h, q_h, out_h[0], staging)
        serial_s = time.perf_counter() - t0
        # (b) three steps in flight: the copies and the planning of a step overlap the kernels of its neighbours
        torch.cuda.synchronize(device)
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            pool.step_host_begin(reqs, thr, ones, k_h, v_h, q_h, out_h[i % 3], staging)
            if i >= 2:
                pool.step_host_wait()
        for _ in range(min(2, e2e_steps)):
            pool.step_host_wait()
        piped_s = time.perf_counter() - t0
        torch.cuda.synchronize(device)
        assert pool.status() == 0
        e2e_tokens, piped_s = aggregate(float(n * e2e_steps), piped_s)
        _, serial_s = aggregate(float(n * e2e_steps), serial_s)
        e2e = {"value": e2e_tokens / piped_s, "unit": UNIT, "h2d_bytes_per_step": k_h.numel() * 2 * 2 + q_h.numel() * 2,
               "d2h_bytes_per_step": out_h[0].numel() * out_h[0].element_size(), "steps": e2e_steps,
               "how": "pasta_step_host_begin / _wait, three steps in flight, pinned host buffers",
               "one_step_at_a_time": e2e_tokens / serial_s}
    if sampler:
        sampler.stop(0, 0)

    B_tok = geo.kv_bytes_per_token
    avg_tokens = (tok0 + tok1) / 2.0 + n / 2.0                 # unique KV tokens of the average timed step
    step_bytes = avg_tokens * B_tok * L
    timed = max(1, max(kernel_launches))
    dom = 0 if kernel_launches[0] else 1                       # tensor-core kernel when the plan has t-units
    prof_tokens = (tok1 + tok2) / 2.0 + n / 2.0
    prof_shared = (shared1 + shared2) / 2.0
    # the warp-shuffle kernel's algorithmic bytes are per query (it is the path for what is not shared): K and V of
    # every token each of its queries sees; the tensor-core kernel's are the unique tokens of its requests
    dom_bytes = (prof_shared if dom == 0 else (warp1 + warp2) / 2.0 + n / 2.0) * B_tok * L
    dom_ms = kernel_ms[dom] / max(1, kernel_launches[dom])
    res = {
        "script": script, "geo": geo, "n": n, "L": L, "requests": len(set(reqs.tolist())),
        "value": all_tokens / (ms * 1e-3), "ms_per_step": ms / steps, "steps": steps, "warmup": warmup,
        "launches": launches, "clocks": clocks, "avg_tokens": avg_tokens, "step_bytes": step_bytes,
        "step_gbs": step_bytes / (ms / steps * 1e-3) / 1e9,
        "kernel_ms_per_step": {"tensor": kernel_ms[0] / timed, "warp": kernel_ms[1] / timed, "merge": kernel_ms[2] / timed,
                               "launches_timed": timed, "where": "every launch of the %d steps after the timed region" % prof_steps,
                               "clocks": prof_clocks},
        "dom": ["attn_tensor_kernel", "attn_warp_kernel"][dom], "dom_bytes": dom_bytes, "dom_ms": dom_ms,
        "dom_gbs": dom_bytes / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 else 0.0,
        "ceilings": ceilings, "e2e": e2e, "spawn_copy_bytes": spawn_copy_bytes,
    }
    pool.close()
    del pool, out, q, k_new, v_new
    torch.cuda.empty_cache()
    return res


def run_dense_mask(args):
    """The workload in the paper's own layout (paper_2502_11517_b200/dense_mask.py): one dense pool per response filled
    in decode order, a boolean mask row per thread, every query reading its response's whole pool.  One layer."""
    import torch
    from paper_2502_11517_b200.build import build
    from paper_2502_11517_b200.dense_mask import DensePool
    build()
    device = torch.device("cuda", 0); torch.cuda.set_device(device)
    script = make_script(args.workload, args.size)
    geo = script.geometry
    warm = max(args.warmup, 3)
    entries = [(r, t, 1) for r, t, _n in script.ops[-1][1]]
    n = len(entries)
    per_req = {}
    for op in script.ops[:-1]:
        if op[0] == "run":
            per_req[op[1]] = per_req.get(op[1], 0) + op[3]
    max_slots = max(per_req.values()) + (args.steps + warm + 2) * max(sum(e[0] == r for e in entries) for r in per_req) + 64
    dp = DensePool(geo.n_q_heads, geo.n_kv_heads, geo.head_dim, max_slots, script.max_threads_per_request, device=device)
    gen = torch.Generator(device=device); gen.manual_seed(script.seed)

    def randn(shape):
        return torch.randn(shape, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)

    for op in script.ops[:-1]:
        if op[0] == "begin":
            dp.begin(op[1])
        elif op[0] == "spawn":
            dp.spawn(op[1], op[2])
        elif op[0] == "run":
            done = 0
            while done < op[3]:
                cnt = min(op[3] - done, 4096)
                dp.run(op[1], op[2], cnt, randn((cnt, geo.n_kv_heads, geo.head_dim)), randn((cnt, geo.n_kv_heads, geo.head_dim)))
                done += cnt
        elif op[0] == "merge":
            dp.merge(op[1], list(op[2] or []))
    k_new, v_new = randn((n, geo.n_kv_heads, geo.head_dim)), randn((n, geo.n_kv_heads, geo.head_dim))
    q = randn((n, geo.n_q_heads, geo.head_dim))
    out = torch.empty(q.shape, dtype=torch.float32, device=device)
    for _ in range(warm):
        dp.step(entries, k_new, v_new, q, out)
    torch.cuda.synchronize(device)
    sampler = ClockSampler(0)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time(); ev0.record()
    read = 0
    for _ in range(args.steps):
        dp.step(entries, k_new, v_new, q, out)
        read += dp.bytes_read_last_step
    ev1.record(); torch.cuda.synchronize(device); sampler.now(); t1 = time.time()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop(t0, t1)
    peak, peak_kind = measured_peak()
    gbs = read / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": METRIC, "value": n * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "size": args.size, "layout": "dense_mask", "script": script.name,
                   "requests": len(per_req), "thread_tokens_per_step": n, "layers": 1,
                   "bytes_read_per_step": read / args.steps, "l2": "inputs larger than L2",
                   "note": "every query reads every slot of its response's pool (K, V and a mask byte per slot)"},
        "clocks": clocks, "e2e": None, "gpu_launches": args.steps * 3 * len(per_req),
        "roofline": {"bound": "hbm", "kernel": "dense_mask_attn_kernel", "achieved": gbs, "peak": peak, "peak_kind": peak_kind,
                     "unit": "GB/s", "frac": gbs / peak, "traffic": None,
                     "note": "bytes the kernel asks for per second (a response's pool is re-read by each of its threads; "
                             "what of that the L2 serves is not DRAM traffic)"},
        "cpu_baseline": None}))


def summary_of(m, peak):
    """The figures of a secondary workload that go under config.other_workloads."""
    return {"workload": m["script"].name, "thread_tokens_per_step": m["n"], "layers": m["L"], "steps": m["steps"],
            "warmup": m["warmup"], "ms_per_step": m["ms_per_step"], "thread_tokens_per_s": m["value"],
            "unique_kv_bytes_per_step": m["step_bytes"],
            "l2": "inputs larger than L2" if m["step_bytes"] / m["L"] > 126e6 * 1.5 else "working set fits L2 (latency case)",
            "step_hbm_gbs": m["step_gbs"], "step_frac_of_measured_peak": m["step_gbs"] / peak,
            "kernel": m["dom"], "kernel_gbs": m["dom_gbs"], "kernel_frac_of_measured_peak": m["dom_gbs"] / peak,
            "kernel_ms_per_step": m["kernel_ms_per_step"], "clocks": m["clocks"], "gpu_launches": m["launches"]}


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
    from paper_2502_11517_b200 import binding as _b
    flags = _b.FLAG_NO_TENSOR_PATH if args.kernel == "warp" else 0
    m = measure_steady(args, args.workload, args.size, args.steps, args.warmup, device, rank, world, local,
                       layout=args.layout, out_dtype_name=args.out_dtype, flags=flags)
    merge_us = time_sync_merge()              # host-only cost of a <sync/> merge (no kernel, no copy)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_kind = measured_peak()
    others = []
    if world == 1 and args.others and args.workload == "long_shared_prefix" and args.layout == "pool" and args.kernel == "auto":
        # the other configurations, same protocol, shorter: their figures ride along under config.other_workloads
        for wl, size, st, wu in (("batched", "full", 12, 3), ("single_request", "full", 200, 10)):
            try:
                others.append(summary_of(measure_steady(args, wl, size, st, wu, device, rank, world, local, with_e2e=False), peak))
            except Exception as exc:           # e.g. not enough free memory on a shared GPU
                others.append({"workload": wl, "error": repr(exc)[:200]})
        try:
            tr = trace_measure(device, rank, world, local, size="small", steps=40, warmup=4)
            others.append({k: tr[k] for k in ("workload", "steps", "warmup", "ms_per_step", "thread_tokens_per_s", "layers",
                                              "requests", "step_hbm_gbs", "step_frac_of_measured_peak", "kernel_ms_per_step",
                                              "clocks", "gpu_launches", "sync_merges_timed")})
        except Exception as exc:
            others.append({"workload": "trace", "error": repr(exc)[:200]})
    geo, L = m["geo"], m["L"]
    traffic = None
    if m["dom"] == "attn_tensor_kernel" and args.layout == "pool" and NCU_TRAFFIC["attn_tensor_sha256_16"] == kernel_source_hash():
        traffic = m["dom_bytes"] * NCU_TRAFFIC["read_ratio"] + NCU_TRAFFIC["write_bytes"]
    result = {
        "metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": m["warmup"], "ms_per_step": m["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": args.workload, "size": args.size, "layout": args.layout, "out_dtype": args.out_dtype,
            "kernel_path": args.kernel,
            "script": m["script"].name, "requests": m["requests"], "thread_tokens_per_step": m["n"],
            "layers": L, "n_q_heads": geo.n_q_heads, "n_kv_heads": geo.n_kv_heads, "head_dim": geo.head_dim,
            "page_size": geo.page_size, "unique_kv_tokens_per_layer": m["avg_tokens"],
            "unique_kv_bytes_per_step": m["step_bytes"],
            "l2": "inputs larger than L2" if m["step_bytes"] / L > 126e6 * 1.5 else "working set fits L2 (latency case)",
            "step_hbm_gbs": m["step_gbs"], "step_frac_of_measured_peak": m["step_gbs"] / peak,
            "step_frac_of_nominal_8TBs": m["step_gbs"] / NOMINAL_HBM_GBS,
            "kernel_ms_per_step": m["kernel_ms_per_step"],
            "read_ceiling_gbs": m["ceilings"],
            "sync_merge_host_us": merge_us,
            **({"bytes_duplicated_at_spawn": m["spawn_copy_bytes"]} if m["spawn_copy_bytes"] is not None else {}),
            **({"other_workloads": others} if others else {}),
        },
        "clocks": m["clocks"],
        "e2e": m["e2e"],
        "gpu_launches": m["launches"],
        "roofline": {"bound": "hbm", "kernel": m["dom"], "achieved": m["dom_gbs"], "peak": peak, "peak_kind": peak_kind,
                     "unit": "GB/s", "frac": m["dom_gbs"] / peak, "frac_of_nominal_8TBs": m["dom_gbs"] / NOMINAL_HBM_GBS,
                     "traffic": traffic, "bytes_per_launch": m["dom_bytes"], "ms_per_launch": m["dom_ms"],
                     "launches_timed": m["kernel_ms_per_step"]["launches_timed"]},
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


def trace_measure(device, rank, world, local, size="full", steps=200, warmup=3):
    """Replays the synthetic interpreter trace op by op (step plan, append, attention of every layer, spawn, finish,
    sync merge) and times `steps` decode steps after `warmup`.  Returns the figures as a dict."""
    import torch
    import torch.distributed as dist
    from paper_2502_11517_b200 import binding
    from paper_2502_11517_b200.sharding import aggregate
    from pasta_workloads import cfg5_trace
    warm = max(warmup, 3)
    n_req, n_layers = (256, 32) if size == "full" else (64, 8)
    script = cfg5_trace(n_requests=n_req, n_steps=steps + warm, n_layers=n_layers)
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
                pool.profile_enable(8)
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
    peak, peak_kind = measured_peak()
    gbs = bytes_ / (ms * 1e-3) / 1e9
    res = {"workload": script.name, "size": size, "script": script, "steps": steps, "warmup": warm,
           "value": all_tokens / worst_s, "thread_tokens_per_s": all_tokens / worst_s, "ms_per_step": worst_s * 1e3 / steps,
           "requests": n_req, "layers": L, "thread_tokens_timed": tokens, "max_thread_tokens_per_step": max_n,
           "sync_merges_timed": int(merges), "pool_pages": script.n_pages, "pool_gb": script.n_pages * 65536 * L / 1e9,
           "unique_kv_bytes_timed": bytes_, "step_hbm_gbs": gbs, "step_frac_of_measured_peak": gbs / peak,
           "kernel_ms_per_step": {"tensor": kernel_ms[0] / timed_calls, "warp": kernel_ms[1] / timed_calls,
                                  "merge": kernel_ms[2] / timed_calls, "launches_timed": timed_calls,
                                  "where": "every eighth step of the timed region"},
           "step_begin_call_ms": host_s * 1e3 / steps, "clocks": clocks, "gpu_launches": launches, "peak": peak,
           "peak_kind": peak_kind}
    pool.close()
    del pool, out, kv_pool, kv_pool2, q_pool
    torch.cuda.empty_cache()
    return res


def run_trace(args):
    import torch
    import torch.distributed as dist
    from paper_2502_11517_b200.build import build
    rank = int(os.environ.get("RANK", "0")); world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    if rank == 0:
        build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local)); dist.barrier()
    device = torch.device("cuda", local); torch.cuda.set_device(device)
    r = trace_measure(device, rank, world, local, size=args.size, steps=args.steps, warmup=args.warmup)
    if rank == 0:
        peak, gbs = r["peak"], r["step_hbm_gbs"]
        print(json.dumps({
            "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": r["warmup"],
            "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "trace", "size": args.size, "script": r["workload"], "requests": r["requests"],
                       "layers": r["layers"], "thread_tokens_timed": r["thread_tokens_timed"],
                       "max_thread_tokens_per_step": r["max_thread_tokens_per_step"],
                       "sync_merges_timed": r["sync_merges_timed"], "pool_pages": r["pool_pages"], "pool_gb": r["pool_gb"],
                       "unique_kv_bytes_timed": r["unique_kv_bytes_timed"], "l2": "inputs larger than L2",
                       "step_hbm_gbs": gbs, "step_frac_of_measured_peak": gbs / peak,
                       "step_frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS, "kernel_ms_per_step": r["kernel_ms_per_step"],
                       "step_begin_call_ms": r["step_begin_call_ms"],
                       "step_begin_note": "wall time inside pasta_step_begin; includes waiting for the device when the host runs ahead"},
            "clocks": r["clocks"], "e2e": None, "gpu_launches": r["gpu_launches"],
            "roofline": {"bound": "hbm", "kernel": "whole step (tensor + warp + merge + append)", "achieved": gbs, "peak": peak,
                         "peak_kind": r["peak_kind"], "unit": "GB/s", "frac": gbs / peak, "traffic": None},
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
ORACLE_WORKER_GB = {"long_shared_prefix": 1.3, "batched": 1.2, "single_request": 0.3}   # resident + transient, per worker


def _oracle_script(workload: str):
    """The bounded sample of a workload that the oracle is timed on: (script, what it is, layers it stands for)."""
    from pasta_workloads import cfg2_single_request, cfg3_batched, cfg4_long_prefix
    if workload == "long_shared_prefix":
        return (cfg4_long_prefix(n_requests=1),
                "the 17 thread-tokens of 1 of the 8 requests (32768-token prefix, 16 forks), 1 layer", 1)
    if workload == "batched":
        return cfg3_batched(n_layers=1), "all thread-tokens of the 64 requests, 1 of 32 layers (time scaled by 32)", 32
    script = cfg2_single_request("a")
    script.ops = script.ops[:11]
    return script, "step A: the 5 thread-tokens of the request, 1 layer", 1


def _oracle_state(workload: str):
    """The oracle replayed up to the workload's last step (bookkeeping and append done once), kept for reuse."""
    if workload in _ORACLE_STATE:
        return _ORACLE_STATE[workload]
    from oracle import OracleReplay
    from pasta_workloads import step_tensors
    script, _, _ = _oracle_script(workload)
    rep = OracleReplay(script)
    last = len(script.ops) - 1
    for i in range(last):
        rep.apply(i, attend=False)
    op = script.ops[last]
    k, v, q = step_tensors(script, last, 0)
    slots = [s for s in rep.model.reserve(op[1]) if s is not None]
    rep.stores[0].write(slots, k, v)
    queries = [(e[0], e[1]) for e in op[1]]
    _ORACLE_STATE[workload] = (rep, queries, q)
    return _ORACLE_STATE[workload]


def _oracle_worker_init(workload, root, ready):
    """Runs once in every worker process: one compute thread, its own copy of the oracle's state."""
    if root not in sys.path:
        sys.path.insert(0, root)
    try:
        import torch
        torch.set_num_threads(1)
    except Exception:
        pass
    try:
        from threadpoolctl import threadpool_limits
        threadpool_limits(1)
    except Exception:
        pass
    _oracle_state(workload)
    with ready.get_lock():
        ready.value += 1


def _oracle_worker_query(task):
    """One query of the sample through the oracle, as it stands; returns the seconds it took in this worker."""
    workload, i = task
    from oracle import decode_attention
    rep, queries, q = _oracle_state(workload)
    t0 = time.perf_counter()
    decode_attention(rep.model, rep.stores[0], [queries[i]], q[i:i + 1])
    return time.perf_counter() - t0


class OraclePool:
    """The fp64 oracle on the host's cores: one single-threaded worker process per core the process may use (fewer when
    memory is short), each with its own copy of the state; queries of the sample are independent and are handed out one
    by one.  Workers are spawned, not forked: this process may already hold a CUDA context."""

    def __init__(self, workload: str):
        import multiprocessing as mp
        self.workload = workload
        self.script, self.what, self.layers = _oracle_script(workload)
        self.n_queries = len(self.script.ops[-1][1])
        self.cores_available = len(os.sched_getaffinity(0))
        workers = self.cores_available
        try:
            import psutil
            room = psutil.virtual_memory().available / 2**30 * 0.5
            workers = max(1, min(workers, int(room / ORACLE_WORKER_GB.get(workload, 1.0))))
        except Exception:
            workers = min(workers, 16)
        self.workers = min(workers, 96)
        ctx = mp.get_context("spawn")
        ready = ctx.Value("i", 0)
        saved = {k: os.environ.get(k) for k in ("OMP_NUM_THREADS", "OPENBLAS_NUM_THREADS", "MKL_NUM_THREADS")}
        os.environ.update({k: "1" for k in saved})           # inherited by the workers: one thread each
        try:
            self.pool = ctx.Pool(self.workers, initializer=_oracle_worker_init, initargs=(workload, ROOT, ready))
        finally:
            for k, v in saved.items():
                if v is None:
                    os.environ.pop(k, None)
                else:
                    os.environ[k] = v
        t0 = time.time()
        while ready.value < self.workers and time.time() - t0 < 300:
            time.sleep(0.05)
        if ready.value < self.workers:
            raise RuntimeError(f"only {ready.value} of {self.workers} oracle workers came up")
        self.one_query_s = None

    def one_core(self, repeats: int = 6) -> float:
        """Seconds per query with a single worker busy (the fastest of a few: the first calls of a worker are cold)."""
        ts = [self.pool.apply(_oracle_worker_query, ((self.workload, i % self.n_queries),)) for i in range(repeats)]
        self.one_query_s = float(min(ts))
        return self.one_query_s

    def sample(self, budget_s: float):
        """Hands whole passes over the sample's queries to the workers for about budget_s seconds of wall time."""
        if self.one_query_s is None:
            self.one_core()
        per_pass = self.n_queries * self.one_query_s / min(self.workers, self.n_queries)
        passes = int(max(1, min(256, budget_s / max(per_pass, 1e-6))))
        # enough queries in the air to keep every worker busy
        passes = max(passes, -(-self.workers // self.n_queries))
        tasks = [(self.workload, i) for _ in range(passes) for i in range(self.n_queries)]
        t0 = time.perf_counter()
        self.pool.map(_oracle_worker_query, tasks, chunksize=1)
        wall = time.perf_counter() - t0
        return {"value": len(tasks) / (wall * self.layers), "unit": UNIT, "cores": self.workers,
                "cores_available": self.cores_available, "kind": "oracle",
                "sample": f"{len(tasks)} thread-tokens ({passes} passes over {self.what})", "seconds": wall,
                "one_core_value": 1.0 / (self.one_query_s * self.layers), "thread_tokens": len(tasks)}

    def close(self):
        self.pool.close()
        self.pool.join()


def oracle_sample(workload: str, budget_s: float = 20.0):
    """The cpu_baseline object: the oracle, as it stands, on a bounded sample of the workload, over the host's cores."""
    pool = OraclePool(workload)
    try:
        return pool.sample(budget_s)
    finally:
        pool.close()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    t0 = time.perf_counter()
    pool = OraclePool(args.workload)                   # set-up once, outside the steps
    try:
        per_step = max(0.5, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
        for _ in range(args.warmup):
            pool.sample(per_step)
        res = [pool.sample(per_step) for _ in range(args.steps)]
    finally:
        pool.close()
    secs = sum(r["seconds"] for r in res)
    done = sum(r["thread_tokens"] for r in res)
    value = done / (secs * pool.layers)
    base = {"value": value, "unit": UNIT, "cores": pool.workers, "cores_available": pool.cores_available, "kind": "oracle",
            "sample": f"{done} thread-tokens in {args.steps} steps, each step whole passes over {pool.what}",
            "seconds": secs, "one_core_value": res[-1]["one_core_value"]}
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
    ap.add_argument("--no-others", dest="others", action="store_false",
                    help="skip the shorter runs of the other configurations that ride along with the default workload")
    ap.add_argument("--kernel", default="auto", choices=["auto", "warp"],
                    help="warp: send every stream through the warp-shuffle kernel (PASTA_FLAG_NO_TENSOR_PATH)")
    ap.add_argument("--tail", default=None, metavar="PERCENT,TILES",
                    help="share of the short runs' tiles that the tensor-core kernel's CTAs share out at run time, and the "
                         "tiles per shared unit (pasta_debug_set_tail; the library's default when not given)")
    ap.add_argument("--no-launch-overlap", action="store_true",
                    help="launch the kernels of a step strictly one after the other (pasta_debug_set_launch_overlap(0)) "
                         "instead of letting each set itself up while the one ahead drains")
    ap.add_argument("--out-dtype", default="fp32", choices=["fp32", "bf16"],
                    help="type of the attention output (bf16 halves the device-to-host bytes of the end-to-end path)")
    ap.add_argument("--layout", default="pool", choices=["pool", "naive_rows", "dense_mask"],
                    help="pool: the library's shared paged pool (default).  naive_rows: the comparison layout of the "
                         "paper's Appendix B (one dense row per thread, prefix duplicated), on the same kernels.  "
                         "dense_mask: the paper's own layout (one dense pool per response in decode order, a boolean "
                         "mask row per thread), one layer, plain CUDA-core kernels")
    ap.add_argument("--size", default="full", choices=["full", "small"],
                    help="small: a reduced copy of the workload for profiler captures (prefix 8192 / 4 layers)")
    args = ap.parse_args()
    if args.no_launch_overlap and args.impl != "reference":
        from paper_2502_11517_b200 import binding as _binding
        from paper_2502_11517_b200.build import build as _build
        _build()
        _binding.Pool.debug_set_launch_overlap(False)
    if args.impl == "reference":
        if args.steps == 200:
            args.steps, args.warmup = 3, 1
        run_reference(args)
    elif args.workload == "trace":
        run_trace(args)
    elif args.workload == "extras":
        run_extras(args)
    elif args.layout == "dense_mask":
        run_dense_mask(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
