"""GPU parity on the edges of the method and of the kernels' limits: empty steps, one-token contexts, ragged page
and tile boundaries, exactly as many stacked rows as the tensor-core tile holds and one thread more, every supported
group size, row counts on both sides of the half-height MMA tile, more streams than the tensor-core path takes, forks
with empty chunks."""
import numpy as np
import pytest

from pasta_workloads import Geometry, Script
from test_gpu_parity import lib, run_script  # noqa: F401  (fixture + helper)

pytestmark = pytest.mark.gpu


def manual(ops, geo, n_pages=256, max_threads=40, max_segments=8, max_requests=2):
    return Script("manual", geo, n_pages, np.random.default_rng(3).permutation(n_pages).astype(np.int32),
                  max_requests, max_threads, max_segments, 31, list(ops))


def test_empty_step(lib):
    import torch
    pool = lib.Pool(1, 8, 2, 128, 8, 1, 2, 2)
    pool.step_begin([], [], [])
    q = torch.empty((1, 0, 8, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((1, 0, 8, 128), dtype=torch.float32, device="cuda")
    pool.kv_append(q[:, :, :2], q[:, :, :2])
    pool.decode_attn(q, out)
    torch.cuda.synchronize()
    assert pool.status() == 0
    pool.close()


@pytest.mark.parametrize("prefix", [1, 15, 16, 17, 127, 128, 129, 255, 257])
def test_ragged_prefix_lengths(lib, prefix):
    geo = Geometry(1, 32, 8, 128, 16)
    ops = [("begin", 0), ("run", 0, 0, prefix), ("spawn", 0, 1), ("spawn", 0, 2), ("run", 0, 2, 17),
           ("step", ((0, 0, 1), (0, 1, 0), (0, 2, 1))),       # fork 1 has an empty chunk and only reads the prefix
           ("step", ((0, 1, 1), (0, 2, 0)))]
    run_script(lib, manual(ops, geo))


@pytest.mark.parametrize("n_forks,tensor_units", [(31, True), (32, False)])
def test_as_many_rows_as_the_tile_holds_and_one_thread_more(lib, n_forks, tensor_units):
    geo = Geometry(1, 32, 8, 128, 16)                          # group 4: 32 threads fill the 128 rows
    ops = [("begin", 0), ("run", 0, 0, 300)]
    for t in range(1, n_forks + 1):
        ops += [("spawn", 0, t), ("run", 0, t, 3 + t % 5)]
    ops.append(("step", tuple((0, t, 1) for t in range(n_forks + 1))))
    script = manual(ops, geo, n_pages=256, max_threads=40)
    from lib_replay import LibReplay, make_pool
    pool = make_pool(script, host_only=True, max_step_queries=64)
    rep = LibReplay(script, pool)
    for i in range(len(script.ops)):
        rep.apply(i)
    w = pool.plan_words()
    assert (w[4] > 0) == tensor_units and (w[5] > 0) == (not tensor_units)     # t-units / w-units of the plan
    pool.close()
    run_script(lib, script, max_step_queries=64)


@pytest.mark.parametrize("n_forks", [0, 3, 4, 7, 8, 11, 15, 16])
def test_row_counts_around_the_half_height_tile(lib, n_forks):
    """Units of at most 64 stacked rows run their MMAs with M = 64 (another row-to-lane layout in tensor memory), larger
    ones with M = 128: 1, 4, 5, 8, 9, 12, 16 and 17 threads of group 4 cover every warp's first and last row on both
    sides of the switch; a second request with 20 threads puts both kinds of unit into one launch."""
    geo = Geometry(1, 32, 8, 128, 16)
    ops = [("begin", 0), ("run", 0, 0, 333), ("begin", 1), ("run", 1, 0, 150)]
    for t in range(1, n_forks + 1):
        ops += [("spawn", 0, t), ("run", 0, t, 1 + (7 * t) % 40)]
    for t in range(1, 20):
        ops += [("spawn", 1, t), ("run", 1, t, 2 + t % 9)]
    ops.append(("step", tuple((0, t, 1) for t in range(n_forks + 1)) + tuple((1, t, 1) for t in range(20))))
    ops.append(("step", tuple((0, t, 1) for t in range(n_forks + 1))))
    run_script(lib, manual(ops, geo, n_pages=400, max_threads=24), max_step_queries=64)


@pytest.mark.parametrize("hq,hkv,d", [(8, 8, 128), (8, 4, 128), (16, 2, 128), (8, 8, 64), (16, 2, 64)])
def test_group_sizes(lib, hq, hkv, d):
    geo = Geometry(2, hq, hkv, d, 16)
    ops = [("begin", 0), ("run", 0, 0, 200), ("spawn", 0, 1), ("run", 0, 0, 40), ("spawn", 0, 2), ("run", 0, 1, 33),
           ("step", ((0, 0, 1), (0, 1, 1), (0, 2, 1))), ("finish", 0, 1), ("finish", 0, 2), ("merge", 0, None),
           ("step", ((0, 0, 1),))]
    run_script(lib, manual(ops, geo))


def test_a_main_thread_that_merged_hundreds_of_chunks_stays_on_the_tensor_path(lib):
    """A long response: 300 chunks merged into the main thread, two forks still decoding.  The request reads 303 streams;
    it must keep its tensor-core units (the prefix staged once for its three threads), not fall back to one warp per
    query and stream."""
    geo = Geometry(1, 8, 2, 128, 16)
    n = 300
    ops = [("begin", 0), ("run", 0, 0, 50)]
    for t in range(1, n + 1):
        ops += [("spawn", 0, t), ("run", 0, t, 1 + t % 3), ("finish", 0, t)]
    ops += [("merge", 0, None), ("run", 0, 0, 200), ("spawn", 0, n + 1), ("spawn", 0, n + 2), ("run", 0, n + 1, 21),
            ("step", ((0, 0, 1), (0, n + 1, 1), (0, n + 2, 1)))]
    script = manual(ops, geo, n_pages=500, max_threads=n + 4, max_segments=2 * n + 8)
    from lib_replay import LibReplay, make_pool
    pool = make_pool(script, host_only=True)
    rep = LibReplay(script, pool)
    for i in range(len(script.ops)):
        rep.apply(i)
    w = pool.plan_words()
    assert w[4] > 0 and w[5] == 0                              # t-units only, no w-units
    pool.close()
    run_script(lib, script)


def test_fork_spawned_before_any_token(lib):
    geo = Geometry(1, 8, 2, 128, 16)
    ops = [("begin", 0), ("spawn", 0, 1), ("run", 0, 1, 5), ("run", 0, 0, 9),
           ("step", ((0, 1, 1), (0, 0, 1))), ("finish", 0, 1), ("merge", 0, (1,)), ("step", ((0, 0, 1),))]
    run_script(lib, manual(ops, geo))


def test_kernel_timing_can_sample_every_kth_step(lib):
    """pasta_profile_enable(k): every k-th attention launch group is bracketed by events, the first one included."""
    import torch
    geo = Geometry(1, 8, 2, 128, 16)
    pool = lib.Pool(geo.n_layers, geo.n_q_heads, geo.n_kv_heads, geo.head_dim, 64, 1, 2, 4)
    r = pool.request_begin()
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    rnd = lambda *shape: torch.randn(shape, generator=g, device="cuda").to(torch.bfloat16)
    pool.kv_append_run(r, 0, 600, rnd(1, 600, 2, 128), rnd(1, 600, 2, 128))    # five tiles per run: cut, so a merge follows
    q, out = rnd(1, 1, 8, 128), torch.empty((1, 1, 8, 128), dtype=torch.float32, device="cuda")
    for stride, steps, want in ((1, 5, 5), (3, 7, 3), (8, 8, 1)):
        pool.profile_enable(stride)
        for _ in range(steps):
            pool.step_begin([r], [0], [1])
            pool.kv_append(rnd(1, 1, 2, 128), rnd(1, 1, 2, 128))
            pool.decode_attn(q, out)
        ms, launches = pool.profile_read()
        assert launches[0] == want and launches[2] == want and launches[1] == 0
        assert ms[0] > 0 and ms[2] > 0
    pool.profile_enable(False)
    with pytest.raises(Exception):
        pool.profile_enable(-1)
    torch.cuda.synchronize()
    assert pool.status() == 0
    pool.close()
