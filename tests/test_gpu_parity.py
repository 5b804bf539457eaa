"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded inputs.

Indexing (slots, page tables, segment lists, the appended bits) must be bit-exact.  Attention must be
within max-abs 1e-2 and mean-abs 1e-3 of the oracle (the stated target; bf16 inputs, bf16 softmax
weights on the tensor-core path, fp32 accumulation)."""
import numpy as np
import pytest

from oracle import OracleReplay
from pasta_workloads import (Geometry, cfg1_tiny, cfg2_single_request, cfg3_batched, cfg4_long_prefix, cfg5_trace,
                             random_script, run_tensors, step_tensors)

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 1e-2, 1e-3


@pytest.fixture(scope="module")
def lib():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2502_11517_b200 import binding, build
    build()
    return binding


def compare(got, got_lse, want, want_lse, what=""):
    got = got.double().cpu().numpy(); got_lse = got_lse.double().cpu().numpy()
    assert np.all(np.isfinite(got)), what
    err = np.abs(got - want)
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (what, err.max(), err.mean())
    assert np.abs(got_lse - want_lse).max() <= 1e-2, (what, np.abs(got_lse - want_lse).max())
    return err.max(), err.mean()


def run_script(lib, script, flags=0, layers=None, check_steps=None, tail=None, **kw):
    """Replays on both sides; compares bookkeeping after every op and attention at every (chosen) step."""
    from lib_replay import LibReplay, make_pool
    layers = list(range(script.geometry.n_layers)) if layers is None else layers
    pool = make_pool(script, flags=flags, **kw)
    if tail is not None:
        pool.debug_set_tail(*tail)
    rep = LibReplay(script, pool)
    ora = OracleReplay(script, layers=layers)
    worst = (0.0, 0.0)
    for i, op in enumerate(script.ops):
        if op[0] == "step":
            attend = check_steps is None or i in check_steps
            res = rep.apply(i, attend=attend)
            want = ora.apply(i, attend=attend)
            slots = [None if s[0] < 0 else (int(s[0]), int(s[1])) for s in rep.last_slots]
            assert slots == [s for s in _oracle_slots(ora, op)], (i, "slots")
            if attend:
                out, lse = res
                for l in layers:
                    e = compare(out[l], lse[l], want[l][0], want[l][1], f"op {i} layer {l}")
                    worst = (max(worst[0], e[0]), max(worst[1], e[1]))
        else:
            rep.apply(i); ora.apply(i)
    assert pool.dump() == ora.model.dump()
    assert pool.status() == 0
    pool.close()
    return worst


def _oracle_slots(ora, op):
    """Slots of the step's entries as the oracle's model placed them (last token of each appended stream)."""
    out = []
    for req, t, n_new in op[1]:
        if not n_new:
            out.append(None); continue
        r = ora.model.requests[req]
        for k in range(r.stream_len[t] - n_new, r.stream_len[t]):     # one slot per new token
            out.append((r.stream_pages[t][k // 16], k % 16))
    return out


# ------------------------------------------------------------------------------------------------ K1
@pytest.mark.parametrize("geo", [Geometry(2, 4, 2, 64, 16), Geometry(2, 8, 2, 128, 16)])
def test_append_is_a_bit_copy_into_the_right_slots(lib, geo):
    import torch
    from lib_replay import LibReplay, make_pool
    script = random_script(5, n_ops=60, geo=geo)
    pool = make_pool(script)
    rep = LibReplay(script, pool)
    ora = OracleReplay(script, layers=[0, 1])
    for i in range(len(script.ops)):
        rep.apply(i, attend=False); ora.apply(i, attend=False)
    dump = pool.dump()
    assert dump == ora.model.dump()
    checked = 0
    for req, r in dump["requests"].items():
        for sid, s in r["streams"].items():
            if s["len"] == 0:
                continue
            slots = [(s["pages"][k // 16], k % 16) for k in range(s["len"])]
            for layer in (0, 1):
                k, v = pool.kv_read(layer, req, sid, 0, s["len"])
                wk, wv = ora.stores[layer].gather(slots)
                assert np.array_equal(k.float().cpu().numpy().astype(np.float64), wk)
                assert np.array_equal(v.float().cpu().numpy().astype(np.float64), wv)
                checked += 1
    assert checked > 4 and pool.status() == 0
    pool.close()


# ------------------------------------------------------------------------------------------------ attention
@pytest.mark.parametrize("variant", ["base", "cutoffs", "chunk16", "chunk33", "append"])
def test_config1_tiny(lib, variant):
    run_script(lib, cfg1_tiny(variant))


@pytest.mark.parametrize("variant", ["a", "b"])
@pytest.mark.parametrize("tensor", [True, False])
def test_config2_single_request(lib, variant, tensor):
    run_script(lib, cfg2_single_request(variant), flags=0 if tensor else lib.FLAG_NO_TENSOR_PATH)


@pytest.mark.parametrize("tensor", [True, False])
def test_config3_batched_reduced(lib, tensor):
    # 16 requests, 3 layers, two launches of <= 2 layers
    run_script(lib, cfg3_batched(16, 3), flags=0 if tensor else lib.FLAG_NO_TENSOR_PATH, max_layers_per_launch=2)


@pytest.mark.parametrize("tensor", [True, False])
def test_config4_long_prefix_reduced(lib, tensor):
    # 2 requests x 4111-token prefix (ragged: not a multiple of the tile) x 16 forks
    run_script(lib, cfg4_long_prefix(2, 4111, 16), flags=0 if tensor else lib.FLAG_NO_TENSOR_PATH)


def test_config4_appending_step(lib):
    run_script(lib, cfg4_long_prefix(2, 2048, 16, n_new=1))


def test_config5_trace_reduced(lib):
    script = cfg5_trace(8, 96, 2, prompt_range=(32, 300), p_promise=0.08, mean_chunk=20.0)
    steps = [i for i, op in enumerate(script.ops) if op[0] == "step"]
    run_script(lib, script, check_steps=set(steps[::8] + steps[-2:]))


@pytest.mark.parametrize("seed", range(6))
def test_random_scripts(lib, seed):
    geo = Geometry(1, 8, 2, 128, 16) if seed % 2 else Geometry(1, 4, 2, 64, 16)
    run_script(lib, random_script(40 + seed, n_ops=70, geo=geo))


@pytest.mark.parametrize("seed", range(4))
def test_random_scripts_with_several_tokens_per_entry(lib, seed):
    geo = Geometry(1, 8, 2, 128, 16) if seed % 2 else Geometry(1, 4, 2, 64, 16)
    run_script(lib, random_script(60 + seed, n_ops=70, geo=geo, multi_token=True))


def test_prompt_fed_in_chunks(lib):
    """Chunked prefill: a 300-token prompt fed 30 tokens per step (120 stacked rows on the tensor-core path), then two
    forks and the main thread feeding 3, 1 and 5 tokens in one step."""
    from pasta_workloads import Script
    geo = Geometry(2, 32, 8, 128, 16)
    ops = [("begin", 0), ("run", 0, 0, 1)] + [("step", ((0, 0, 30),)) for _ in range(10)]
    ops += [("spawn", 0, 1), ("spawn", 0, 2), ("run", 0, 1, 20), ("step", ((0, 1, 3), (0, 2, 1), (0, 0, 5)))]
    script = Script("chunked_prefill", geo, 64, np.arange(64, dtype=np.int32), 2, 4, 8, 7, ops)
    run_script(lib, script)


def test_page_placement_does_not_change_the_result(lib):
    import torch
    from lib_replay import LibReplay, make_pool
    outs = []
    for order_seed in (0, 1):
        script = cfg2_single_request("b")
        script.free_order = np.random.default_rng(order_seed).permutation(script.n_pages).astype(np.int32)
        pool = make_pool(script); rep = LibReplay(script, pool)
        res = [rep.apply(i) for i in range(len(script.ops))]
        outs.append([r[0].cpu() for r in res if r is not None])
        pool.close()
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_step_device_entry_point_equals_the_three_calls(lib):
    import torch
    from lib_replay import LibReplay, make_pool
    outs = []
    for fused in (False, True):
        script = cfg2_single_request("b")
        pool = make_pool(script)
        rep = LibReplay(script, pool)
        first = next(i for i, op in enumerate(script.ops) if op[0] == "step")
        for i in range(first):
            rep.apply(i)
        op = script.ops[first]
        L = range(script.geometry.n_layers)
        ks, vs, qs = zip(*[step_tensors(script, first, l) for l in L])
        k = torch.stack(ks).cuda(); v = torch.stack(vs).cuda(); q = torch.stack(qs).cuda()
        out = torch.empty(q.shape, dtype=torch.float32, device="cuda")
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
        reqs = [e[0] for e in op[1]]; thr = [e[1] for e in op[1]]; nn = [e[2] for e in op[1]]
        if fused:
            pool.step_device(reqs, thr, nn, k, v, q, out, lse)
        else:
            pool.step_begin(reqs, thr, nn); pool.kv_append(k, v); pool.decode_attn(q, out, lse)
        torch.cuda.synchronize()
        assert pool.status() == 0
        outs.append((out.cpu(), lse.cpu(), pool.dump()))
        pool.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1]) and outs[0][2] == outs[1][2]


def test_bf16_output_option(lib):
    """The same step with fp32 and with bf16 outputs: the bf16 result is the fp32 one rounded once."""
    import torch
    from lib_replay import LibReplay, make_pool
    outs = {}
    for flag in (0, lib.FLAG_OUT_BF16):
        script = cfg2_single_request("b")
        pool = make_pool(script, flags=flag)
        rep = LibReplay(script, pool)
        first = next(i for i, op in enumerate(script.ops) if op[0] == "step")
        for i in range(first):
            rep.apply(i)
        op = script.ops[first]
        L = range(script.geometry.n_layers)
        ks, vs, qs = zip(*[step_tensors(script, first, l) for l in L])
        k = torch.stack(ks).cuda(); v = torch.stack(vs).cuda(); q = torch.stack(qs).cuda()
        out = torch.empty(q.shape, dtype=torch.bfloat16 if flag else torch.float32, device="cuda")
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
        pool.step_device([e[0] for e in op[1]], [e[1] for e in op[1]], [e[2] for e in op[1]], k, v, q, out, lse)
        torch.cuda.synchronize()
        assert pool.status() == 0
        outs[flag] = (out.cpu(), lse.cpu())
        pool.close()
    assert torch.equal(outs[0][0].to(torch.bfloat16), outs[lib.FLAG_OUT_BF16][0])
    assert torch.equal(outs[0][1], outs[lib.FLAG_OUT_BF16][1])


def test_step_host_entry_point(lib):
    """The host-buffer entry point (copies inside the call) gives the same numbers as the device one."""
    import torch
    from lib_replay import LibReplay, make_pool
    script = cfg2_single_request("a")
    pool = make_pool(script); rep = LibReplay(script, pool)
    ora = OracleReplay(script)
    last = len(script.ops) - 1
    for i in range(last):
        rep.apply(i, attend=False); ora.apply(i, attend=False)
    op = script.ops[last]
    k, v, q = step_tensors(script, last, 0)
    want = ora.apply(last)[0]
    out = torch.empty(q.unsqueeze(0).shape, dtype=torch.float32).pin_memory()
    staging = torch.empty(pool.step_host_bytes(len(op[1])), dtype=torch.uint8, device="cuda")
    pool.step_host([e[0] for e in op[1]], [e[1] for e in op[1]], [e[2] for e in op[1]],
                   k.unsqueeze(0).contiguous().pin_memory(), v.unsqueeze(0).contiguous().pin_memory(),
                   q.unsqueeze(0).contiguous().pin_memory(), out, staging)
    err = np.abs(out[0].double().numpy() - want[0])
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS
    assert pool.dump() == ora.model.dump() and pool.status() == 0
    pool.close()


@pytest.mark.parametrize("slots", [1, 2, 3])
def test_step_host_in_two_halves_keeps_two_steps_in_flight(lib, slots):
    """pasta_step_host_begin / _wait: five appending steps, the next ones begun before the previous ones are waited for
    (two in flight; three with a staging area for three steps); every step's output against the oracle, with a staging
    area for one, two and three steps."""
    import torch
    from lib_replay import LibReplay, make_pool
    script = cfg2_single_request("a")
    first = next(i for i, op in enumerate(script.ops) if op[0] == "step")
    entries = tuple((r, t, 1) for r, t, _ in script.ops[first][1])
    script.ops = script.ops[:first] + [("step", entries)] * 5
    pool = make_pool(script); rep = LibReplay(script, pool)
    ora = OracleReplay(script)
    for i in range(first):
        rep.apply(i, attend=False); ora.apply(i, attend=False)
    n = len(entries)
    staging = torch.empty(slots * pool.step_host_bytes(n), dtype=torch.uint8, device="cuda")
    reqs = [e[0] for e in entries]; thr = [e[1] for e in entries]; nn = [e[2] for e in entries]
    bufs = []
    for i in range(first, first + 5):
        k, v, q = step_tensors(script, i, 0)
        bufs.append([t.unsqueeze(0).contiguous().pin_memory() for t in (k, v, q)] +
                    [torch.full((1,) + tuple(q.shape), float("nan"), dtype=torch.float32).pin_memory()])

    def check(j):
        pool.step_host_wait()
        want = ora.apply(first + j)[0]
        err = np.abs(bufs[j][3][0].double().numpy() - want[0])
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (j, err.max())

    depth = max(2, slots)                             # steps that may be in flight
    waited = 0
    for j in range(5):
        pool.step_host_begin(reqs, thr, nn, bufs[j][0], bufs[j][1], bufs[j][2], bufs[j][3], staging)
        if j == depth - 1:                            # all in flight: one begin more is refused, nothing changes
            with pytest.raises(lib.PastaError) as e:
                pool.step_host_begin(reqs, thr, nn, bufs[j + 1][0], bufs[j + 1][1], bufs[j + 1][2], bufs[j + 1][3], staging)
            assert e.value.code == lib.BAD_STATE
        if j >= depth - 1:
            check(waited); waited += 1
    while waited < 5:
        check(waited); waited += 1
    with pytest.raises(lib.PastaError) as e:
        pool.step_host_wait()
    assert e.value.code == lib.BAD_STATE
    assert pool.dump() == ora.model.dump() and pool.status() == 0
    pool.close()


@pytest.mark.parametrize("tail", [(10, 16), (50, 10), (0, 4)])
def test_units_shared_out_at_run_time_long_runs(lib, tail):
    """Enough tiles (64 runs of 38) for the planner to keep whole runs back as units the CTAs take from a counter at
    run time; with half of all tiles shared in units of 10 tiles every CTA goes through several of them."""
    from lib_replay import LibReplay, make_pool
    script = cfg4_long_prefix(8, 4000, 4, n_new=1)
    pool = make_pool(script, host_only=True)
    pool.debug_set_tail(*tail)
    rep = LibReplay(script, pool)
    for i in range(len(script.ops)):
        rep.apply(i)
    assert (pool.plan_words()[23] > 0) == (tail[0] > 0)          # shared units in the plan
    pool.close()
    run_script(lib, script, tail=tail)


def test_units_shared_out_at_run_time_short_runs_three_layers(lib):
    """The batched configuration with three layers in one launch: whole short runs go to the shared pool, and a shared
    unit is a (layer, unit) pair.  Two launches in a row: the counter starts from zero each time."""
    run_script(lib, cfg3_batched(64, 3, n_new=1), tail=(20, 3))
    run_script(lib, cfg3_batched(64, 3), tail=(20, 3), max_layers_per_launch=2)


def _one_step(lib, script, flags=0, overlap=True, want_lse=True):
    """Replays `script` up to its last step and runs that step through pasta_step_device; returns out, lse, plan words."""
    import torch
    from lib_replay import LibReplay, make_pool
    lib.Pool.debug_set_launch_overlap(overlap)
    try:
        pool = make_pool(script, flags=flags)
        rep = LibReplay(script, pool)
        last = max(i for i, op in enumerate(script.ops) if op[0] == "step")
        for i in range(last):
            rep.apply(i, attend=False)
        op = script.ops[last]
        L = range(script.geometry.n_layers)
        ks, vs, qs = zip(*[step_tensors(script, last, l) for l in L])
        k = torch.stack(ks).cuda(); v = torch.stack(vs).cuda(); q = torch.stack(qs).cuda()
        out = torch.full(q.shape, float("nan"), dtype=torch.bfloat16 if flags & lib.FLAG_OUT_BF16 else torch.float32, device="cuda")
        lse = torch.full(q.shape[:3], float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
        before = pool.launch_count()
        pool.step_device([e[0] for e in op[1]], [e[1] for e in op[1]], [e[2] for e in op[1]], k, v, q, out, lse)
        torch.cuda.synchronize()
        assert pool.status() == 0
        words = np.array(pool.plan_words())
        if words[26] == 0 and words[23] == 0:        # nothing to merge: append and attention, no third launch
            assert pool.launch_count() - before <= 2
        pool.close()
        return out.cpu(), None if lse is None else lse.cpu(), words
    finally:
        lib.Pool.debug_set_launch_overlap(True)


def _final_flags(words):
    """The final marks of a plan's assigned and shared units (word 11 of every 12-word record)."""
    t = words[words[13]: words[13] + 12 * words[4]].reshape(-1, 12)[:, 11]
    d = words[words[24]: words[24] + 12 * words[23]].reshape(-1, 12)[:, 11]
    return np.concatenate([t, d])


def test_a_step_with_final_and_merged_rows(lib):
    """The batched configuration cuts some of its runs at CTA boundaries and leaves most whole: whole runs are final
    units, whose rows the tensor-core kernel writes to the output itself, the rest goes through partial rows and the
    merge.  Every output element is written by exactly one of the two (none stays NaN), both equal the oracle's, with
    fp32 and bf16 outputs (bf16 = the fp32 result rounded once), with and without a log-sum-exp output."""
    import torch
    script = cfg3_batched(64, 2, n_new=1)
    out32, lse32, words = _one_step(lib, script)
    fin = _final_flags(words)
    assert 0 < fin.sum() < len(fin), "the step should mix final and merged units"
    ora = OracleReplay(script, layers=[0, 1])
    last = max(i for i, op in enumerate(script.ops) if op[0] == "step")
    for i in range(last):
        ora.apply(i, attend=False)
    want = ora.apply(last)
    for l in (0, 1):
        compare(out32[l], lse32[l], want[l][0], want[l][1], f"layer {l}")
    out16, lse16, _ = _one_step(lib, script, flags=lib.FLAG_OUT_BF16)
    assert torch.equal(out32.to(torch.bfloat16), out16) and torch.equal(lse32, lse16)
    out_nolse, _, _ = _one_step(lib, script, want_lse=False)
    assert torch.equal(out_nolse, out32)


@pytest.mark.parametrize("maker", [lambda: cfg3_batched(64, 3, n_new=1), lambda: cfg4_long_prefix(4, 3000, 6, n_new=1),
                                   lambda: random_script(3, n_ops=80, geo=Geometry(2, 4, 2, 64, 16))])
def test_launch_overlap_does_not_change_results(lib, maker):
    """The kernels of a step launched so that each sets itself up while the one ahead drains, against the same step
    launched strictly in sequence: identical bits (tensor-core path with several layers per launch, long runs with a
    merge, and the warp-shuffle path)."""
    import torch
    script = maker()
    a = _one_step(lib, script, overlap=True)
    b = _one_step(lib, script, overlap=False)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    assert not torch.isnan(a[0]).any() and not torch.isnan(a[1]).any()


def test_a_step_with_nothing_to_merge(lib):
    """Two responses with short contexts: every run is one final unit, the plan counts no unit that leaves partial rows,
    the library launches no merge kernel, and every output element and log-sum-exp still arrives (none stays NaN) and
    equals the oracle's."""
    script = cfg3_batched(2, 2, prefix_range=(20, 40), n_new=1)
    out, lse, words = _one_step(lib, script)
    assert words[26] == 0 and words[23] == 0 and words[4] > 0          # nothing partial, no shared units, tensor path
    ora = OracleReplay(script, layers=[0, 1])
    last = max(i for i, op in enumerate(script.ops) if op[0] == "step")
    for i in range(last):
        ora.apply(i, attend=False)
    want = ora.apply(last)
    for l in (0, 1):
        compare(out[l], lse[l], want[l][0], want[l][1], f"layer {l}")
