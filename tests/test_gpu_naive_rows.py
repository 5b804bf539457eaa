"""The comparison layout (one dense row per thread, prefix duplicated at spawn, chunks copied at sync) run on the
GPU through the same C ABI, against the oracle's outputs for the ORIGINAL threaded script: both must give every
thread the same attention result, which is the paper's premise for comparing the two layouts by cost alone."""
import numpy as np
import pytest

from oracle import OracleReplay
from pasta_workloads import Geometry, cfg1_tiny, cfg2_single_request, random_script, run_tensors, step_tensors

pytestmark = pytest.mark.gpu
MAX_ABS, MEAN_ABS = 1e-2, 1e-3


def run_both(script):
    import torch
    from paper_2502_11517_b200 import binding
    from paper_2502_11517_b200.build import build
    from paper_2502_11517_b200.naive_rows import NaiveRows
    build()
    geo = script.geometry
    n_rows = sum(op[0] in ("begin", "spawn") for op in script.ops)
    pool = binding.Pool(geo.n_layers, geo.n_q_heads, geo.n_kv_heads, geo.head_dim,
                        script.n_pages * (script.max_threads_per_request + 1) + 4 * n_rows, n_rows, 1, 4,
                        max_step_queries=64)
    nr = NaiveRows(pool)
    ora = OracleReplay(script, layers=list(range(geo.n_layers)))
    finished, merged = set(), set()
    worst, n_cmp = 0.0, 0
    L = range(geo.n_layers)
    for i, op in enumerate(script.ops):
        kind = op[0]
        want = ora.apply(i)
        if kind == "begin":
            nr.begin(op[1])
        elif kind == "end":
            nr.end(op[1])
            finished = {x for x in finished if x[0] != op[1]}; merged = {x for x in merged if x[0] != op[1]}
        elif kind == "spawn":
            nr.spawn(op[1], op[2])
        elif kind == "finish":
            finished.add((op[1], op[2]))
        elif kind == "merge":
            forks = op[2] if op[2] is not None else sorted(t for (r, t) in finished if r == op[1] and (r, t) not in merged)
            nr.merge(op[1], forks)
            merged.update((op[1], t) for t in forks)
        elif kind == "run":
            if op[3]:
                ks, vs = zip(*[run_tensors(script, i, l) for l in L])
                nr.run(op[1], op[2], op[3], torch.stack(ks).cuda(), torch.stack(vs).cuda())
        elif kind == "step":
            ks, vs, qs = zip(*[step_tensors(script, i, l) for l in L])
            k = torch.stack(ks).cuda(); v = torch.stack(vs).cuda(); q = torch.stack(qs).cuda()
            out = torch.empty(q.shape, dtype=torch.float32, device="cuda")
            lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
            nr.step(op[1], k, v, q, out, lse)
            torch.cuda.synchronize()
            assert pool.status() == 0
            for l in L:
                err = np.abs(out[l].double().cpu().numpy() - want[l][0])
                assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (i, l, err.max())
                assert np.abs(lse[l].double().cpu().numpy() - want[l][1]).max() <= 1e-2
                worst = max(worst, err.max()); n_cmp += 1
    stats = (nr.bytes_copied_at_spawn, nr.bytes_copied_at_sync)
    pool.close()
    return worst, n_cmp, stats


@pytest.mark.parametrize("maker", [cfg1_tiny, lambda: cfg1_tiny("cutoffs"), lambda: cfg2_single_request("a"),
                                   lambda: cfg2_single_request("b")])
def test_configs(maker):
    worst, n, (spawn_b, sync_b) = run_both(maker())
    print(f"naive rows: {n} steps x layers compared, worst max-abs {worst:.2e}; copied {spawn_b} B at spawn, {sync_b} B at sync")
    assert n > 0 and spawn_b > 0


@pytest.mark.parametrize("seed", [1, 4, 6, 9])
def test_random_scripts(seed):
    script = random_script(seed, n_ops=70, geo=Geometry(1, 32, 8, 128, 16), paper_flow=bool(seed % 2))
    worst, n, _ = run_both(script)
    assert n > 0
