"""A bounded device wait that runs out: reported as PASTA_ERR_TIMEOUT, the kernel returns, the pool stays usable.

Every wait of one kernel role for another carries a cycle limit (the pool's, 3e9 cycles by default).  Nothing in a
correct run ever makes one expire, so the limit is shortened through the test hook and a one-warp kernel waits for a
barrier phase that nobody completes: the permitted way to see the limit, the status word and the recovery at work
without hanging or faulting anything.  The abort paths inside the tensor-core kernel itself (draining the bulk
copies and MMAs in flight, freeing TMEM after a role gave up) are reached by holding one of its roles back."""
import numpy as np
import pytest

from oracle import OracleReplay
from pasta_workloads import cfg2_single_request
from test_gpu_parity import compare, lib  # noqa: F401  (fixture + helper)

pytestmark = pytest.mark.gpu


def _replay_to_parity(pool, script):
    from lib_replay import LibReplay
    rep = LibReplay(script, pool)
    ora = OracleReplay(script)
    steps = 0
    for i, op in enumerate(script.ops):
        res, want = rep.apply(i), ora.apply(i)
        if op[0] == "step":
            compare(res[0][0], res[1][0], want[0][0], want[0][1], f"op {i}")
            steps += 1
    assert steps == 2 and pool.dump() == ora.model.dump()


@pytest.mark.parametrize("tensor", [True, False], ids=["tensor", "warp"])
def test_expired_wait_is_reported_and_cleared_and_the_next_steps_are_right(lib, tensor):
    import time
    import torch
    from lib_replay import make_pool
    script = cfg2_single_request("b")
    pool = make_pool(script, flags=0 if tensor else lib.FLAG_NO_TENSOR_PATH)
    assert pool.status() == lib.OK
    pool.debug_set_wait_limit(200_000)                # about 0.1 ms of SM clock
    t0 = time.perf_counter()
    pool.debug_wait_expiry()
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 0.5             # it gave up after the short limit, not after the default 1.5 s
    assert pool.status() == lib.TIMEOUT               # read ...
    assert pool.status() == lib.OK                    # ... and cleared by the read
    # the attention kernels take the same (still shortened, but ample) limit from the pool: 50 ms of waiting allowed
    pool.debug_set_wait_limit(100_000_000)
    _replay_to_parity(pool, script)
    assert pool.status() == lib.OK
    pool.debug_set_wait_limit(0)                      # back to the default
    pool.close()


def test_two_expiries_in_a_row_and_a_host_only_pool(lib):
    import torch
    from lib_replay import make_pool
    script = cfg2_single_request("a")
    pool = make_pool(script)
    pool.debug_set_wait_limit(50_000)
    pool.debug_wait_expiry(); pool.debug_wait_expiry()
    torch.cuda.synchronize()
    assert pool.status() == lib.TIMEOUT and pool.status() == lib.OK
    pool.close()
    host = make_pool(script, host_only=True)
    with pytest.raises(lib.PastaError) as e:
        host.debug_set_wait_limit(10)
    assert e.value.code == lib.BAD_STATE
    host.close()


@pytest.mark.parametrize("mask", [1, 2, 4, 8, 16], ids=["producer", "mma_issue", "query_builder", "softmax_0", "softmax_1"])
def test_a_role_that_never_starts_makes_the_tensor_kernel_give_up_cleanly(lib, mask):
    """The abort paths of the tensor-core kernel itself: one role is held back (a flag that nothing sets), the roles
    that wait for it run into a short limit, every CTA drains its copies and MMAs in flight, frees its tensor memory
    and returns; the status word says TIMEOUT; the same planned step then runs normally and matches the oracle."""
    import time
    import torch
    from lib_replay import LibReplay, make_pool
    from pasta_workloads import cfg3_batched, step_tensors
    script = cfg3_batched(40, 2)                       # 320 (request, kv head) runs: several units per CTA, two layers
    pool = make_pool(script)
    rep = LibReplay(script, pool)
    ora = OracleReplay(script, layers=[0, 1])
    last = len(script.ops) - 1
    for i in range(last):
        rep.apply(i); ora.apply(i)
    rep.apply(last, attend=False)                      # plans the step and appends; no attention yet
    want = ora.apply(last)
    assert pool.plan_words()[4] > 148                  # t-units
    q = torch.stack([step_tensors(script, last, l)[2] for l in (0, 1)]).cuda()
    out = torch.zeros(q.shape, dtype=torch.float32, device="cuda")
    lse = torch.zeros(q.shape[:3], dtype=torch.float32, device="cuda")
    pool.debug_set_wait_limit(400_000)                 # about 0.2 ms
    pool.debug_hold_roles(mask)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    pool.decode_attn(q, out, lse)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 2.0
    assert pool.status() == lib.TIMEOUT and pool.status() == lib.OK
    pool.debug_hold_roles(0)
    pool.debug_set_wait_limit(0)
    pool.decode_attn(q, out, lse)
    for l in (0, 1):
        compare(out[l], lse[l], want[l][0], want[l][1], f"layer {l} after a timed-out launch")
    assert pool.status() == lib.OK
    pool.close()
