"""The paper's own layout (one dense pool per response, tokens in decode order, a boolean mask row per thread) run on
the GPU through the C ABI, against the oracle's outputs for the same threaded script.  The oracle gathers each
thread's visible tokens through page tables and segment lists; here the same sets are encoded as mask rows over an
interleaved pool.  Equal results say that the two formulations of visibility agree (Section 3 "Efficiency")."""
import numpy as np
import pytest

from oracle import OracleReplay
from pasta_workloads import Geometry, cfg1_tiny, cfg2_single_request, random_script, run_tensors, step_tensors

pytestmark = pytest.mark.gpu
MAX_ABS, MEAN_ABS = 1e-2, 1e-3


def run_both(script):
    import torch
    from paper_2502_11517_b200.build import build
    from paper_2502_11517_b200.dense_mask import DensePool
    build()
    geo = script.geometry
    total = sum(op[3] for op in script.ops if op[0] == "run") + sum(len(op[1]) for op in script.ops if op[0] == "step")
    dp = DensePool(geo.n_q_heads, geo.n_kv_heads, geo.head_dim, total + 8, script.max_threads_per_request)
    ora = OracleReplay(script)
    finished, merged = set(), set()
    worst, n_cmp = 0.0, 0
    for i, op in enumerate(script.ops):
        kind = op[0]
        want = ora.apply(i)
        if kind == "begin":
            dp.begin(op[1])
        elif kind == "end":
            dp.end(op[1])
            finished = {x for x in finished if x[0] != op[1]}; merged = {x for x in merged if x[0] != op[1]}
        elif kind == "spawn":
            dp.spawn(op[1], op[2])
        elif kind == "finish":
            finished.add((op[1], op[2]))
        elif kind == "merge":
            forks = op[2] if op[2] is not None else sorted(t for (r, t) in finished if r == op[1] and (r, t) not in merged)
            dp.merge(op[1], forks)
            merged.update((op[1], t) for t in forks)
        elif kind == "run":
            if op[3]:
                k, v = run_tensors(script, i, 0)
                dp.run(op[1], op[2], op[3], k.cuda(), v.cuda())
        elif kind == "step":
            k, v, q = step_tensors(script, i, 0)
            q = q.cuda()
            out = torch.full(q.shape, float("nan"), dtype=torch.float32, device="cuda")
            lse = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device="cuda")
            dp.step(op[1], k.cuda(), v.cuda(), q, out, lse)
            torch.cuda.synchronize()
            err = np.abs(out.double().cpu().numpy() - want[0][0])
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (i, err.max())
            assert np.abs(lse.double().cpu().numpy() - want[0][1]).max() <= 1e-2
            worst = max(worst, err.max()); n_cmp += 1
    return worst, n_cmp, dp


@pytest.mark.parametrize("maker", [cfg1_tiny, lambda: cfg1_tiny("cutoffs"), lambda: cfg1_tiny("append"),
                                   lambda: cfg2_single_request("a"), lambda: cfg2_single_request("b")])
def test_configs(maker):
    worst, n, dp = run_both(maker())
    print(f"dense pool + mask: {n} steps compared, worst max-abs {worst:.2e}; last step read {dp.bytes_read_last_step} B")
    assert n > 0


@pytest.mark.parametrize("seed", [1, 4, 6, 9, 12])
def test_random_scripts(seed):
    geo = Geometry(1, 8, 2, 128, 16) if seed % 2 else Geometry(1, 4, 2, 64, 16)
    worst, n, _ = run_both(random_script(seed, n_ops=70, geo=geo, paper_flow=bool(seed % 3)))
    assert n > 0


def test_argument_checks():
    import torch
    from paper_2502_11517_b200 import binding, build
    build()
    k = torch.zeros((64, 2, 128), dtype=torch.bfloat16, device="cuda")
    mask = torch.zeros((2, 64), dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.PastaError) as e:                       # beyond the pool's last slot
        binding.dense_append(k, k, mask, mask.clone(), 60, [0] * 8, k[:8], k[:8])
    assert e.value.code == binding.INVALID_ARG
    q = torch.zeros((1, 4, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((1, 4, 128), dtype=torch.float32, device="cuda")
    rows = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.PastaError) as e:                       # scratch too small
        binding.dense_mask_attn(k, k, mask, rows, q, out, None, torch.empty(256, dtype=torch.uint8, device="cuda"), 64)
    assert e.value.code == binding.INVALID_ARG
