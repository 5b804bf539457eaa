"""A bounded device wait that runs out: reported as PASTA_ERR_TIMEOUT, the kernel returns, the pool stays usable.

Every wait of one kernel role for another carries a cycle limit (the pool's, 3e9 cycles by default).  Nothing in a
correct run ever makes one expire, so the limit is shortened through the test hook and a one-warp kernel waits for a
barrier phase that nobody completes: the permitted way to see the limit, the status word and the recovery at work
without hanging or faulting anything.  The abort paths inside the attention kernels themselves (draining the bulk
copies and MMAs in flight, freeing TMEM after a role gave up) are not reached by this test."""
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
