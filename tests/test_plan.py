"""The step plan, executed on the CPU by tests/plan_interpreter.py, must reproduce the oracle."""
import numpy as np
import pytest

from oracle import OracleReplay
from paper_2502_11517_b200 import binding, build
from pasta_workloads import (Geometry, cfg1_tiny, cfg2_single_request, cfg3_batched, cfg4_long_prefix, cfg5_trace,
                             random_script, run_tensors, step_tensors)
from lib_replay import LibReplay, make_pool
from plan_interpreter import run_plan


@pytest.fixture(scope="module", autouse=True)
def _built():
    build()


def _f64(t):
    import torch
    return t.to(torch.float32).numpy().astype(np.float64)


def check_script(script, flags=0, steps=None, tail=None, **kw):
    geo = script.geometry
    pool = make_pool(script, host_only=True, flags=flags, **kw)
    if tail is not None:
        pool.debug_set_tail(*tail)
    lib = LibReplay(script, pool)
    ora = OracleReplay(script)
    K = np.zeros((script.n_pages, 16, geo.n_kv_heads, geo.head_dim)); V = np.zeros_like(K)
    n_checked = 0
    stats = {"tunits": 0, "wunits": 0}
    for i, op in enumerate(script.ops):
        if op[0] == "run":
            before = pool.dump()["requests"][op[1]]["streams"][op[2]]["len"]
            lib.apply(i); ora.apply(i)
            pages = pool.dump()["requests"][op[1]]["streams"][op[2]]["pages"]
            k, v = run_tensors(script, i, 0)
            for j in range(op[3]):
                t = before + j
                K[pages[t // 16], t % 16] = _f64(k[j]); V[pages[t // 16], t % 16] = _f64(v[j])
        elif op[0] == "step":
            lib.apply(i)
            k, v, q = step_tensors(script, i, 0)
            j = 0
            for s in lib.last_slots:                  # one slot per query; (-1, -1) where nothing was appended
                if s[0] >= 0:
                    K[s[0], s[1]] = _f64(k[j]); V[s[0], s[1]] = _f64(v[j]); j += 1
            if steps is not None and i not in steps:
                ora.apply(i, attend=False)
                continue
            want, want_lse = ora.apply(i)[0]
            w = pool.plan_words()
            stats["tunits"] += int(w[4]); stats["wunits"] += int(w[5]); stats["steps"] = stats.get("steps", 0) + 1
            got, got_lse = run_plan(w, K, V, _f64(q), geo.n_kv_heads)
            np.testing.assert_allclose(got, want, rtol=0, atol=1e-11)
            np.testing.assert_allclose(got_lse, want_lse, rtol=0, atol=1e-11)
            n_checked += 1
        else:
            lib.apply(i); ora.apply(i)
    pool.close()
    assert n_checked
    return stats


@pytest.mark.parametrize("seed", range(10))
def test_plan_on_random_scripts_d64(seed):
    check_script(random_script(seed, n_ops=70, geo=Geometry(1, 4, 2, 64, 16)))


@pytest.mark.parametrize("seed", range(10, 18))
@pytest.mark.parametrize("flags", [0, binding.FLAG_NO_TENSOR_PATH])
def test_plan_on_random_scripts_d128(seed, flags):
    check_script(random_script(seed, n_ops=70, geo=Geometry(1, 8, 2, 128, 16)), flags=flags)


@pytest.mark.parametrize("seed", range(20, 28))
def test_plan_with_several_tokens_per_entry(seed):
    geo = Geometry(1, 8, 2, 128, 16) if seed % 2 else Geometry(1, 4, 2, 64, 16)
    check_script(random_script(seed, n_ops=70, geo=geo, multi_token=True))


@pytest.mark.parametrize("maker", [cfg1_tiny, lambda: cfg1_tiny("cutoffs"), lambda: cfg1_tiny("append"),
                                   lambda: cfg2_single_request("a"), lambda: cfg2_single_request("b"),
                                   lambda: cfg3_batched(6, 1, prefix_range=(64, 400)),
                                   lambda: cfg4_long_prefix(2, 1100, 5)])
def test_plan_on_configs(maker):
    check_script(maker())


def test_plan_on_a_trace():
    script = cfg5_trace(5, 60, 1, prompt_range=(16, 120), p_promise=0.1, mean_chunk=12.0)
    steps = [i for i, op in enumerate(script.ops) if op[0] == "step"][::6]
    check_script(script, steps=set(steps))


def test_small_partial_budget_still_plans():
    # few partial rows allowed: the planner must use longer pieces instead of failing
    script = cfg3_batched(4, 1, prefix_range=(300, 600))
    n = len(script.ops[-1][1])
    check_script(script, max_partial_rows=n * 32 * 2 + 160 * 128)


@pytest.mark.parametrize("tail", [None, (25, 10), (50, 16), (25, 2), (0, 4)])
def test_plan_with_shared_units(tail):
    """Enough tiles (64 runs of 38) for the planner to keep whole runs back as units the CTAs share out at run time,
    when runs of 38 tiles count as short (at most four units long): every run must still be tiled exactly once and the
    merged result must equal the oracle's."""
    from plan_interpreter import STATS
    before = STATS.get("dunits", 0)
    check_script(cfg4_long_prefix(8, 4000, 4), tail=tail)
    assert (STATS.get("dunits", 0) > before) == (tail not in ((0, 4), (25, 2)))


def test_plan_with_a_shared_tail_short_runs():
    """Many short runs (the batched configuration, one layer): whole runs go to the shared pool, every so often."""
    from plan_interpreter import STATS
    before = STATS.get("dunits", 0)
    check_script(cfg3_batched(64, 1))
    assert STATS.get("dunits", 0) > before


def test_shared_tail_is_dropped_when_it_does_not_fit():
    """With room for the partial rows of the assigned units only, the step is planned without a shared tail instead of
    being refused."""
    script = cfg4_long_prefix(8, 4000, 4)

    def plan(tail, **kw):
        pool = make_pool(script, host_only=True, **kw)
        if tail:
            pool.debug_set_tail(*tail)
        lib = LibReplay(script, pool)
        for i in range(len(script.ops)):
            lib.apply(i)
        w = pool.plan_words()
        pool.close()
        return int(w[7]), int(w[23])               # partial rows of a layer, shared units

    rows_without, none = plan((0, 4))
    rows_with, some = plan(None)
    assert none == 0 and some > 0 and rows_with > rows_without
    assert plan(None, max_partial_rows=rows_without + 8) == (rows_without, 0)


def test_final_units_are_marked_and_only_those():
    """Short runs fit one unit each: the plan marks such units final (their rows are the result, the merge skips them),
    the interpreter checks that a final row is the only row of its (query, head) pair
    and that every lone row is marked.  With runs cut in several pieces by a small grid's worth of work, cut runs stay
    unmarked."""
    from plan_interpreter import STATS
    before = STATS.get("final_units", 0)
    stats = check_script(cfg3_batched(20, 1, prefix_range=(64, 700)))
    marked = STATS["final_units"] - before
    assert 0 < marked <= stats["tunits"]
    before = STATS["final_units"]
    stats = check_script(cfg4_long_prefix(2, 3000, 3))            # 16 runs of 24 tiles over 148 CTAs: every run is cut
    assert STATS["final_units"] == before and stats["tunits"] > 16


def test_small_steps_are_not_cut():
    """Two responses with contexts of a few dozen tokens (every run has a CTA of its own and is a tile or two long): the
    runs stay whole, every unit is final and the plan says that nothing is left to merge.  Ten-tile runs are cut."""
    from plan_interpreter import STATS
    before = STATS.get("no_merge_plans", 0)
    stats = check_script(cfg3_batched(2, 1, prefix_range=(20, 40)))
    assert STATS["no_merge_plans"] - before == stats["steps"] > 0
    before = STATS["no_merge_plans"]
    check_script(cfg2_single_request("a"))
    assert STATS["no_merge_plans"] == before


def test_zz_all_visible_page_flag_is_exercised():
    """The plans interpreted above marked some pages as visible in full to every thread (checked page by page in
    plan_interpreter.run_plan) and left others unmarked."""
    from plan_interpreter import STATS
    assert 0 < STATS["flagged"] < STATS["pages"], STATS
