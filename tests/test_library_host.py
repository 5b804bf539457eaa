"""CPU-only tests of the CUDA library's host side: exported symbols, bookkeeping parity with the
oracle's pool model (bit-exact, every operation), error codes, and the step plan."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import OracleReplay, PoolError, PoolModel
from paper_2502_11517_b200 import binding, build
from pasta_workloads import (Geometry, cfg1_tiny, cfg2_single_request, cfg3_batched, cfg4_long_prefix, cfg5_trace,
                             random_script)
from lib_replay import LibReplay, make_pool

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "pasta.h")).read()
    declared = set(re.findall(r"\b(pasta_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS), declared ^ set(binding.EXPORTS)
    lib = ctypes.CDLL(build())
    for name in declared:
        assert hasattr(lib, name), name


def _same_state(script, every_op=True):
    pool = make_pool(script, host_only=True)
    lib = LibReplay(script, pool)
    ora = OracleReplay(script, with_kv=False)
    for i, op in enumerate(script.ops):
        if op[0] == "step":
            want = ora.model.reserve(op[1]); ora.next_op += 1
            lib.apply(i)
            got = [None if s[0] < 0 else (int(s[0]), int(s[1])) for s in lib.last_slots]
            assert got == want, (i, op)
        else:
            ora.apply(i); lib.apply(i)
        if every_op or i == len(script.ops) - 1:
            assert pool.dump() == ora.model.dump(), (i, op)
    pool.close()


@pytest.mark.parametrize("seed", range(16))
def test_bookkeeping_matches_oracle_on_random_scripts(seed):
    _same_state(random_script(seed, n_ops=90, geo=Geometry(1, 4, 2, 64, 16), paper_flow=bool(seed % 2)))


@pytest.mark.parametrize("maker", [cfg1_tiny, lambda: cfg1_tiny("cutoffs"), lambda: cfg1_tiny("chunk33"),
                                   lambda: cfg2_single_request("a"), lambda: cfg2_single_request("b"),
                                   lambda: cfg3_batched(12, 2), lambda: cfg4_long_prefix(2, 1024, 5)])
def test_bookkeeping_matches_oracle_on_configs(maker):
    _same_state(maker())


@pytest.mark.parametrize("seed", range(6))
def test_bookkeeping_matches_oracle_with_several_tokens_per_entry(seed):
    _same_state(random_script(100 + seed, n_ops=90, geo=Geometry(1, 4, 2, 64, 16), multi_token=True))


def test_bookkeeping_matches_oracle_on_a_trace():
    _same_state(cfg5_trace(12, 160, 1, prompt_range=(16, 200), p_promise=0.08, mean_chunk=20.0), every_op=False)
    _same_state(cfg5_trace(6, 120, 1, prompt_range=(16, 100), p_promise=0.1, mean_chunk=15.0, overlap=True))


def _codes(fn_lib, fn_ora):
    try:
        fn_lib(); a = 0
    except binding.PastaError as e:
        a = e.code
    try:
        fn_ora(); b = 0
    except PoolError as e:
        b = e.code
    return a, b


def test_error_codes_match_and_leave_state_unchanged():
    pool = binding.Pool(1, 4, 2, 64, 2, 2, 3, 3, flags=binding.FLAG_HOST_ONLY)
    m = PoolModel(2, 16, None, 2, 3, 3)
    for obj in (pool, m):
        r = obj.request_begin()
    pool.kv_append_run(0, 0, 16); m.append_run(0, 0, 16)
    t = pool.thread_spawn(0); assert t == m.thread_spawn(0)
    cases = [
        (lambda: pool.kv_append_run(0, 0, 17), lambda: m.append_run(0, 0, 17)),            # out of pages
        (lambda: pool.step_begin([0, 0], [0, t], [1, 1]), lambda: m.reserve([(0, 0, 1), (0, t, 1)])),
        (lambda: pool.sync_merge(0, [t]), lambda: m.sync_merge(0, [t])),                    # still decoding
        (lambda: pool.step_begin([0, 0], [0, 0]), lambda: m.reserve([(0, 0, 1), (0, 0, 1)])),
        (lambda: pool.step_begin([0], [7]), lambda: m.reserve([(0, 7, 1)])),
        (lambda: pool.step_begin([1], [0]), lambda: m.reserve([(1, 0, 1)])),
        (lambda: pool.step_begin([0], [0], [-1]), lambda: m.reserve([(0, 0, -1)])),
        (lambda: pool.thread_finish(0, 0), lambda: m.thread_finish(0, 0)),
        (lambda: pool.thread_finish(0, 5), lambda: m.thread_finish(0, 5)),
        (lambda: pool.request_end(1), lambda: m.request_end(1)),
        (lambda: pool.sync_merge(0, [t, t]), lambda: m.sync_merge(0, [t, t])),
    ]
    before = pool.dump()
    for fl, fo in cases:
        a, b = _codes(fl, fo)
        assert a == b and a != 0, (a, b)
        assert pool.dump() == before == m.dump()
    pool.thread_finish(0, t); m.thread_finish(0, t)
    for fl, fo in [(lambda: pool.step_begin([0], [t]), lambda: m.reserve([(0, t, 1)])),
                   (lambda: pool.thread_finish(0, t), lambda: m.thread_finish(0, t))]:
        a, b = _codes(fl, fo); assert a == b and a != 0
    pool.sync_merge(0, [t]); m.sync_merge(0, [t])
    a, b = _codes(lambda: pool.sync_merge(0, [t]), lambda: m.sync_merge(0, [t])); assert a == b == 1
    pool.sync_merge(0); m.sync_merge(0)
    assert pool.dump() == m.dump()
    # capacities
    pool.request_begin(); m.request_begin()
    a, b = _codes(pool.request_begin, m.request_begin); assert a == b == 4
    t2 = pool.thread_spawn(0); assert t2 == m.thread_spawn(0)
    a, b = _codes(lambda: pool.thread_spawn(0), lambda: m.thread_spawn(0)); assert a == b == 4
    # a fork spawned at position 0 of an empty request sees nothing yet
    tt = pool.thread_spawn(1); assert tt == m.thread_spawn(1)
    a, b = _codes(lambda: pool.step_begin([1], [tt], [0]), lambda: m.reserve([(1, tt, 0)])); assert a == b == 1
    # compute entry points refuse a host-only pool
    with pytest.raises(binding.PastaError) as e:
        pool.kv_append_run(0, 0, 0, layer_count=1)
    assert e.value.code == binding.BAD_STATE
    pool.close()


def test_bad_configurations_are_rejected():
    for kw in (dict(head_dim=96), dict(n_q_heads=6, n_kv_heads=4), dict(page_size=32), dict(n_pages=0)):
        args = dict(n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=64, n_pages=8, max_requests=1,
                    max_threads_per_request=2, max_segments_per_thread=4, flags=binding.FLAG_HOST_ONLY)
        args.update(kw)
        with pytest.raises(binding.PastaError) as e:
            binding.Pool(**args)
        assert e.value.code == binding.INVALID_ARG
    with pytest.raises(binding.PastaError):
        binding.Pool(1, 4, 2, 64, 4, 1, 2, 4, free_order=[0, 1, 1, 3], flags=binding.FLAG_HOST_ONLY)


@pytest.mark.parametrize("seed", range(20, 28))
def test_position_ids_match_oracle(seed):
    """Promises with length predictions: the library's position ids (per step entry, and the per-thread counters in
    the dump) equal the oracle model's."""
    script = random_script(seed, n_ops=90, geo=Geometry(1, 4, 2, 64, 16), predictions=True)
    pool = make_pool(script, host_only=True)
    lib = LibReplay(script, pool)
    ora = OracleReplay(script, with_kv=False)
    checked = 0
    for i, op in enumerate(script.ops):
        lib.apply(i)
        if op[0] == "step":
            ora.model.reserve(op[1]); ora.next_op += 1
            want = [ora.model.last_position(e[0], e[1]) for e in op[1]]
            assert pool.step_positions().tolist() == want
            checked += 1
        else:
            ora.apply(i)
        assert pool.dump() == ora.model.dump(), (i, op)
    assert checked
    pool.close()


@pytest.mark.parametrize("seed", range(8))
def test_pending_spawn_matches_oracle(seed):
    """Spawning on a decoded, not yet appended promise: same state as the oracle after every call, same refusals."""
    rng = np.random.default_rng(77 + seed)
    pool = binding.Pool(1, 4, 2, 64, 128, 2, 8, 6, flags=binding.FLAG_HOST_ONLY)
    model = PoolModel(128, 16, max_requests=2, max_threads_per_request=8, max_segments_per_thread=6)

    def both(name_lib, name_ora, *args):
        a, b = _codes(lambda: getattr(pool, name_lib)(*args), lambda: getattr(model, name_ora)(*args))
        assert a == b, (name_lib, args, a, b)
        assert pool.dump() == model.dump(), (name_lib, args)
        return a

    req = pool.request_begin(); assert model.request_begin() == req
    both("kv_append_run", "append_run", req, 0, int(rng.integers(0, 40)))
    live = []
    for _ in range(30):
        what = int(rng.integers(0, 6))
        if what == 0:
            code = both("thread_spawn_predicted", "thread_spawn", req, int(rng.integers(0, 4)) * 10, int(rng.integers(0, 2)))
            if code == 0:
                live.append(max(model.requests[req].state))
        elif what == 1:
            entries = [(req, 0, int(rng.integers(1, 4)))] if rng.integers(0, 2) else []
            entries += [(req, t, int(rng.integers(0, 4))) for t in live if rng.integers(0, 2)]
            if not entries:
                continue
            a, b = _codes(lambda: pool.step_begin(*zip(*entries)), lambda: model.reserve(entries))
            assert a == b, (entries, a, b)
            assert pool.dump() == model.dump()
            if a == 0:
                assert pool.step_positions().tolist() == model.step_positions
        elif what == 2 and live:
            both("kv_append_run", "append_run", req, live[int(rng.integers(0, len(live)))], int(rng.integers(0, 20)))
        elif what == 3 and live:
            t = live.pop(int(rng.integers(0, len(live))))
            both("thread_finish", "thread_finish", req, t)
            both("sync_merge", "sync_merge", req, [t])
        elif what == 4:
            both("kv_append_run", "append_run", req, 0, int(rng.integers(0, 3)))
    pool.close()


def test_a_step_that_cannot_be_planned_leaves_the_pool_unchanged():
    """max_partial_rows too small for the step's partial results: pasta_step_begin returns CAPACITY and takes the
    reservation back (lengths, page lists, free order, views, position ids), so the caller can go on with a smaller
    step; the oracle's model, which never saw the failed step, stays equal to the pool."""
    from oracle import PoolModel
    build()
    order = np.random.default_rng(3).permutation(64).astype(np.int32)
    pool = binding.Pool(1, 8, 2, 128, 64, 2, 6, 12, free_order=order, flags=binding.FLAG_HOST_ONLY, max_partial_rows=40,
                        max_step_queries=8)
    model = PoolModel(64, 16, order, 2, 6, 12)
    assert pool.request_begin() == model.request_begin() == 0
    pool.kv_append_run(0, 0, 16); model.append_run(0, 0, 16)        # the next main-thread token opens a page
    for _ in range(4):
        assert pool.thread_spawn_predicted(0, 7) == model.thread_spawn(0, 7)
    pool.kv_append_run(0, 1, 15); model.append_run(0, 1, 15)
    before = pool.dump()
    assert before == model.dump()
    entries = [(0, 0, 1), (0, 1, 2), (0, 2, 1), (0, 3, 1), (0, 4, 1)]      # 6 queries x 4 heads x 2 kv heads = 48 partial rows > 40
    with pytest.raises(binding.PastaError) as e:
        pool.step_begin([x[0] for x in entries], [x[1] for x in entries], [x[2] for x in entries])
    assert e.value.code == binding.CAPACITY
    assert pool.dump() == before
    small = [(0, 1, 2), (0, 0, 1)]                                   # 3 queries, 24 partial rows: fits
    pool.step_begin([x[0] for x in small], [x[1] for x in small], [x[2] for x in small])
    want_slots = model.reserve(small)
    assert [(int(a), int(b)) for a, b in pool.step_slots()] == want_slots
    assert pool.dump() == model.dump()
    assert list(pool.step_positions()) == [model.last_position(0, 1) - 1, model.last_position(0, 1), model.last_position(0, 0)]
    pool.close()


def test_tuning_and_test_hooks_check_their_arguments():
    build()
    pool = binding.Pool(1, 8, 2, 128, 16, 1, 2, 4, flags=binding.FLAG_HOST_ONLY)
    pool.debug_set_tail(0, 2); pool.debug_set_tail(50, 1024); pool.debug_set_tail(10, 16)
    for bad in ((-1, 4), (51, 4), (10, 1), (10, 1025)):
        with pytest.raises(binding.PastaError) as e:
            pool.debug_set_tail(*bad)
        assert e.value.code == binding.INVALID_ARG
    for call in (lambda: pool.debug_set_wait_limit(1000), lambda: pool.debug_hold_roles(1)):
        with pytest.raises(binding.PastaError) as e:       # a host-only pool launches nothing
            call()
        assert e.value.code == binding.BAD_STATE
    pool.close()
