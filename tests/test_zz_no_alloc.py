"""The allocation-free attention entry point against the oracle and against the regular entry point.

pasta_decode_attn_noalloc serves callers that must not allocate once they are running (engine plug-ins,
real-time loops, processes whose GPU memory belongs to a framework arena): its intermediate results live
in a fixed array inside the library, shared by every call on the GPU.  Here it is called through the C ABI
twice in a row for every step, and between the two calls another pool's step runs through the same entry
point, so that the second call finds the array full of foreign data.  Each result must be within the
stated tolerance of the fp64 oracle and bit-identical to pasta_decode_attn (same plan, same kernels, same
summation order: only the address of the intermediate rows differs).
Collected last on purpose, so that a stop-at-first-failure run has already been through everything else."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 1e-2, 1e-3


def _other_pool_step():
    """A pool of another shape with a planned step, and its queries: something else to run through the array."""
    import torch
    from pasta_workloads import cfg4_long_prefix, step_tensors
    from lib_replay import LibReplay, make_pool
    script = cfg4_long_prefix(1, 700, 9)
    pool = make_pool(script)
    rep = LibReplay(script, pool)
    last = len(script.ops) - 1
    for i in range(last + 1):
        rep.apply(i, attend=False)
    q = step_tensors(script, last, 0)[2].cuda()
    return pool, q, torch.empty(q.shape, dtype=torch.float32, device="cuda")


def test_noalloc_entry_point_matches_oracle_and_regular_one_twice():
    import torch
    assert torch.cuda.is_available()
    from oracle import OracleReplay
    from paper_2502_11517_b200 import build
    from pasta_workloads import cfg2_single_request, cfg3_batched, cfg4_long_prefix, step_tensors
    from lib_replay import LibReplay, make_pool
    build()
    other, other_q, other_out = _other_pool_step()
    checked = 0
    # the last script has three layers: the entry point is asked for layers 0 and 2 of it
    for script, layers in ((cfg2_single_request("b"), [0]), (cfg4_long_prefix(1, 1500, 6), [0]),
                           (cfg3_batched(6, 3), [0, 2])):
        pool = make_pool(script)
        rep = LibReplay(script, pool)
        ora = OracleReplay(script, layers=layers)
        for i, op in enumerate(script.ops):
            res = rep.apply(i)
            want = ora.apply(i)
            if res is None:
                continue
            for layer in layers:
                q = step_tensors(script, i, layer)[2].cuda()
                for call in range(2):
                    got = torch.full(q.shape, float("nan"), dtype=torch.float32, device="cuda")
                    lse = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device="cuda")
                    pool.decode_attn_noalloc(q, got, lse, layer=layer)
                    torch.cuda.synchronize()
                    err = np.abs(got.double().cpu().numpy() - want[layer][0])
                    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (script.name, i, layer, call, err.max())
                    assert np.abs(lse.double().cpu().numpy() - want[layer][1]).max() <= 1e-2
                    assert torch.equal(got, res[0][layer]) and torch.equal(lse, res[1][layer]), (script.name, i, layer, call)
                    checked += 1
                    other.decode_attn_noalloc(other_q, other_out)          # foreign rows for the next call to find
                    torch.cuda.synchronize()
        assert pool.status() == 0
        pool.close()
    assert other.status() == 0
    other.close()
    assert checked >= 10


def test_noalloc_accepts_an_empty_step_like_the_regular_entry_point():
    import torch
    from paper_2502_11517_b200 import binding, build
    build()
    pool = binding.Pool(1, 8, 2, 128, 8, 1, 2, 2)
    pool.step_begin([], [], [])
    pool.decode_attn(None, None)
    pool.decode_attn_noalloc(None, None)
    torch.cuda.synchronize()
    assert pool.status() == 0
    pool.close()


def test_noalloc_refuses_steps_beyond_its_fixed_size():
    import torch
    from paper_2502_11517_b200 import binding, build
    from pasta_workloads import cfg4_long_prefix, step_tensors
    from lib_replay import LibReplay, make_pool
    build()
    script = cfg4_long_prefix(6, 3000, 31)                     # 128 stacked rows per unit: more partial rows than the array holds
    pool = make_pool(script, max_step_queries=256)
    rep = LibReplay(script, pool)
    last = len(script.ops) - 1
    for i in range(last + 1):
        rep.apply(i, attend=False)
    assert pool.plan_words()[7] > 16384
    _, _, q = step_tensors(script, last, 0)
    q = q.cuda()
    out = torch.empty(q.shape, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.PastaError) as e:
        pool.decode_attn_noalloc(q, out)
    assert e.value.code == binding.CAPACITY
    pool.close()
