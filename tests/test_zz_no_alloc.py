"""The allocation-free attention entry point against the regular one.

pasta_decode_attn_noalloc serves callers that must not allocate once they are running (engine plug-ins,
real-time loops, processes whose GPU memory belongs to a framework arena): its intermediate results live
in a fixed array inside the library.  Here it is called through the C ABI twice in a row — the second
call finds the array full of the first call's data — and must reproduce pasta_decode_attn each time.
Collected last on purpose, so that a stop-at-first-failure run has already been through everything else."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 1e-2, 1e-3


def test_noalloc_entry_point_matches_regular_one_twice():
    import torch
    assert torch.cuda.is_available()
    from paper_2502_11517_b200 import binding, build
    from pasta_workloads import cfg2_single_request, cfg4_long_prefix, run_tensors, step_tensors
    from lib_replay import LibReplay, make_pool
    build()
    checked = 0
    for script in (cfg2_single_request("b"), cfg4_long_prefix(1, 1500, 6)):
        pool = make_pool(script)
        rep = LibReplay(script, pool)
        for i, op in enumerate(script.ops):
            res = rep.apply(i)
            if res is None:
                continue
            want = res[0][0]                                   # pasta_decode_attn, layer 0
            _, _, q = step_tensors(script, i, 0)
            q = q.cuda()
            for call in range(2):
                got = torch.full(q.shape, float("nan"), dtype=torch.float32, device="cuda")
                lse = torch.empty(q.shape[:2], dtype=torch.float32, device="cuda")
                pool.decode_attn_noalloc(q, got, lse)
                torch.cuda.synchronize()
                err = (got.double() - want.double()).abs()
                assert torch.isfinite(got).all()
                assert err.max().item() <= MAX_ABS and err.mean().item() <= MEAN_ABS, (script.name, i, call)
                assert (lse - res[1][0]).abs().max().item() <= 1e-2
                checked += 1
        assert pool.status() == 0
        pool.close()
    assert checked >= 6


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
