"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: all layers in one
pasta_decode_attn call, one step of all threads.  The oracle evaluates a sample of the queries one by one."""
import numpy as np
import pytest

from oracle import KVStore, PoolModel, decode_attention
from pasta_workloads import cfg3_batched, cfg4_long_prefix, run_tensors, step_tensors

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 1e-2, 1e-3


def _replay_both(script, oracle_layers, torch, binding):
    """Applies the script to the library (all layers; layers outside `oracle_layers` get device-generated
    data) and to the oracle (bookkeeping + the chosen layers).  Returns pool, model, stores, final-step tensors."""
    geo = script.geometry
    pool = binding.Pool(geo.n_layers, geo.n_q_heads, geo.n_kv_heads, geo.head_dim, script.n_pages,
                        script.max_requests, script.max_threads_per_request, script.max_segments_per_thread,
                        free_order=script.free_order, max_layers_per_launch=geo.n_layers)
    model = PoolModel(script.n_pages, geo.page_size, script.free_order)
    stores = {l: KVStore(script.n_pages, geo.page_size, geo.n_kv_heads, geo.head_dim) for l in oracle_layers}
    gen = torch.Generator(device="cuda"); gen.manual_seed(1)

    last = len(script.ops) - 1
    for i, op in enumerate(script.ops):
        kind = op[0]
        if kind == "begin":
            assert pool.request_begin() == op[1] == model.request_begin()
        elif kind == "spawn":
            assert pool.thread_spawn(op[1]) == op[2] == model.thread_spawn(op[1])
        elif kind == "run":
            m = op[3]
            slots = model.append_run(op[1], op[2], m)
            k = torch.empty((geo.n_layers, m, geo.n_kv_heads, geo.head_dim), dtype=torch.bfloat16, device="cuda")
            k.copy_(torch.randn(k.shape, generator=gen, device="cuda", dtype=torch.float32))
            v = torch.empty_like(k)
            v.copy_(torch.randn(v.shape, generator=gen, device="cuda", dtype=torch.float32))
            for l in oracle_layers:
                kc, vc = run_tensors(script, i, l)
                k[l].copy_(kc); v[l].copy_(vc)
                stores[l].write(slots, kc, vc)
            pool.kv_append_run(op[1], op[2], m, k, v)
        elif kind == "step":
            assert i == last
            entries = op[1]
            slots = [s for s in model.reserve(entries) if s is not None]
            n = len(entries); n_app = len(slots)
            k = torch.zeros((geo.n_layers, n_app, geo.n_kv_heads, geo.head_dim), dtype=torch.bfloat16, device="cuda")
            v = torch.zeros_like(k)
            q = torch.empty((geo.n_layers, n, geo.n_q_heads, geo.head_dim), dtype=torch.bfloat16, device="cuda")
            q.copy_(torch.randn(q.shape, generator=gen, device="cuda", dtype=torch.float32))
            q_cpu = {}
            for l in oracle_layers:
                kc, vc, qc = step_tensors(script, i, l)
                if n_app:
                    k[l].copy_(kc); v[l].copy_(vc)
                q[l].copy_(qc); q_cpu[l] = qc
                stores[l].write(slots, kc, vc)
            pool.step_begin([e[0] for e in entries], [e[1] for e in entries], [e[2] for e in entries])
            got_slots = [None if s[0] < 0 else (int(s[0]), int(s[1])) for s in pool.step_slots()]
            assert [s for s in got_slots if s is not None] == slots
            pool.kv_append(k, v)
            out = torch.empty(q.shape, dtype=torch.float32, device="cuda")
            lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
            pool.decode_attn(q, out, lse)
            torch.cuda.synchronize()
            return pool, model, stores, entries, q_cpu, out, lse
        else:
            raise AssertionError(kind)


def _check_sample(model, stores, entries, q_cpu, out, lse, sample, layers):
    worst = (0.0, 0.0)
    for l in layers:
        for i in sample:
            want, want_lse = decode_attention(model, stores[l], [(entries[i][0], entries[i][1])], q_cpu[l][i:i + 1])
            got = out[l, i].double().cpu().numpy()
            err = np.abs(got - want[0])
            assert np.all(np.isfinite(got))
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (l, i, err.max(), err.mean())
            assert np.abs(lse[l, i].double().cpu().numpy() - want_lse[0]).max() <= 1e-2
            worst = (max(worst[0], err.max()), max(worst[1], err.mean()))
    return worst


def test_long_shared_prefix_full_size():
    """cfg4 as benchmarked: 8 requests x 32768-token prefix x 16 forks; 12 sampled queries (forks and main threads)."""
    import torch
    from paper_2502_11517_b200 import binding, build
    build()
    script = cfg4_long_prefix(n_new=1)
    pool, model, stores, entries, q_cpu, out, lse = _replay_both(script, [0], torch, binding)
    assert pool.dump() == model.dump()
    rng = np.random.default_rng(0)
    mains = [i for i, e in enumerate(entries) if e[1] == 0]
    forks = [i for i, e in enumerate(entries) if e[1] != 0]
    sample = list(rng.choice(mains, 3, replace=False)) + list(rng.choice(forks, 9, replace=False))
    worst = _check_sample(model, stores, entries, q_cpu, out, lse, sample, [0])
    assert torch.isfinite(out).all()
    assert pool.status() == 0
    print("cfg4 full size: worst max-abs %.2e mean-abs %.2e over %d sampled queries" % (worst + (len(sample),)))
    pool.close()


def test_batched_full_size():
    """cfg3 as benchmarked: 64 requests x 32 layers in one call; the oracle holds layers 0 and 31 and checks
    40 sampled queries in each; every other layer must at least be finite."""
    import torch
    from paper_2502_11517_b200 import binding, build
    build()
    script = cfg3_batched(n_new=1)
    layers = [0, script.geometry.n_layers - 1]
    pool, model, stores, entries, q_cpu, out, lse = _replay_both(script, layers, torch, binding)
    assert pool.dump() == model.dump()
    rng = np.random.default_rng(1)
    sample = list(rng.choice(len(entries), 40, replace=False))
    worst = _check_sample(model, stores, entries, q_cpu, out, lse, sample, layers)
    assert torch.isfinite(out).all() and torch.isfinite(lse).all()
    assert pool.status() == 0
    print("cfg3 full size: worst max-abs %.2e mean-abs %.2e" % worst)
    pool.close()


def test_interpreter_trace_at_size():
    """cfg5 with its stated statistics (promise probability 0.02, chunks of mean 80, groups of 2 to 6 forks) at
    64 requests x 8 layers x 128 decode steps.  Indexing (slots of every step, the whole bookkeeping state after every
    step) must equal the oracle's exactly.  Attention is checked against the oracle in layers 0 and 7: every query of
    every 32nd step and of the last step, and, in the step that follows a spawn or a merge, every query of the
    requests that spawned or merged."""
    import torch
    from paper_2502_11517_b200 import binding, build
    from pasta_workloads import cfg5_trace
    build()
    script = cfg5_trace(n_requests=64, n_steps=128, n_layers=8)
    geo = script.geometry
    layers = [0, geo.n_layers - 1]
    pool = binding.Pool(geo.n_layers, geo.n_q_heads, geo.n_kv_heads, geo.head_dim, script.n_pages,
                        script.max_requests, script.max_threads_per_request, script.max_segments_per_thread,
                        free_order=script.free_order, max_layers_per_launch=geo.n_layers,
                        max_step_queries=max(len(op[1]) for op in script.ops if op[0] == "step"))
    model = PoolModel(script.n_pages, geo.page_size, script.free_order, script.max_requests,
                      script.max_threads_per_request, script.max_segments_per_thread)
    stores = {l: KVStore(script.n_pages, geo.page_size, geo.n_kv_heads, geo.head_dim) for l in layers}
    gen = torch.Generator(device="cuda"); gen.manual_seed(5)

    def noise(shape):
        t = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
        t.copy_(torch.randn(shape, generator=gen, device="cuda", dtype=torch.float32))
        return t

    n_steps = sum(op[0] == "step" for op in script.ops)
    step_no = queries_checked = steps_checked = spawns = merges = 0
    touched = set()
    worst = (0.0, 0.0)
    for i, op in enumerate(script.ops):
        kind = op[0]
        if kind == "begin":
            assert pool.request_begin() == op[1] == model.request_begin()
        elif kind == "spawn":
            assert pool.thread_spawn(op[1]) == op[2] == model.thread_spawn(op[1], 0, 0)
            touched.add(op[1]); spawns += 1
        elif kind == "finish":
            pool.thread_finish(op[1], op[2]); model.thread_finish(op[1], op[2])
        elif kind == "merge":
            pool.sync_merge(op[1], list(op[2])); model.sync_merge(op[1], list(op[2]))
            touched.add(op[1]); merges += 1
        elif kind == "run":
            m = op[3]
            slots = model.append_run(op[1], op[2], m)
            k, v = noise((geo.n_layers, m, geo.n_kv_heads, geo.head_dim)), noise((geo.n_layers, m, geo.n_kv_heads, geo.head_dim))
            for l in layers:
                kc, vc = run_tensors(script, i, l)
                k[l].copy_(kc); v[l].copy_(vc)
                stores[l].write(slots, kc, vc)
            pool.kv_append_run(op[1], op[2], m, k, v)
        elif kind == "step":
            entries = op[1]
            n = len(entries)
            slots = [s for s in model.reserve(entries) if s is not None]
            k, v = noise((geo.n_layers, n, geo.n_kv_heads, geo.head_dim)), noise((geo.n_layers, n, geo.n_kv_heads, geo.head_dim))
            q = noise((geo.n_layers, n, geo.n_q_heads, geo.head_dim))
            q_cpu = {}
            for l in layers:
                kc, vc, qc = step_tensors(script, i, l)
                k[l].copy_(kc); v[l].copy_(vc); q[l].copy_(qc); q_cpu[l] = qc
                stores[l].write(slots, kc, vc)
            pool.step_begin([e[0] for e in entries], [e[1] for e in entries], [e[2] for e in entries])
            assert [(int(s[0]), int(s[1])) for s in pool.step_slots()] == slots, ("slots", step_no)
            pool.kv_append(k, v)
            out = torch.empty(q.shape, dtype=torch.float32, device="cuda")
            lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
            pool.decode_attn(q, out, lse)
            assert pool.dump() == model.dump(), ("bookkeeping", step_no)
            if step_no % 32 == 0 or step_no == n_steps - 1:
                sample = list(range(n))
            else:
                sample = [j for j, e in enumerate(entries) if e[0] in touched]
            if sample:
                w = _check_sample(model, stores, entries, q_cpu, out, lse, sample, layers)
                worst = (max(worst[0], w[0]), max(worst[1], w[1]))
                queries_checked += len(sample) * len(layers); steps_checked += 1
            touched.clear()
            step_no += 1
        else:
            raise AssertionError(kind)
    assert pool.status() == 0
    assert step_no == 128 and spawns >= 100 and merges >= 10 and steps_checked >= 60
    print("cfg5 at size: %d steps, %d spawns, %d merges; attention checked on %d (query, layer) pairs in %d steps, "
          "worst max-abs %.2e mean-abs %.2e; bookkeeping equal after every step"
          % (step_no, spawns, merges, queries_checked, steps_checked, worst[0], worst[1]))
    pool.close()
