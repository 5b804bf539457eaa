"""GPU parity of the position-id / rotary-embedding step in front of the pool: positions bit-exact, the keys the
library stores equal to the float64 oracle's rotated keys rounded to bf16 (at most one bf16 ulp apart, and
almost always identical), attention over them within the usual tolerance."""
import numpy as np
import pytest

from oracle import KVStore, PoolModel, decode_attention, rope_bf16
from pasta_workloads import Geometry, random_script, run_tensors, step_tensors

pytestmark = pytest.mark.gpu
THETA = 10000.0


def _ulp_distance(a, b):
    """Distance in bf16 units in the last place between two bf16 tensors (same shape)."""
    import torch
    ia = a.view(torch.int16).to(torch.int32); ib = b.view(torch.int16).to(torch.int32)
    key = lambda x: torch.where(x < 0, -(x & 0x7FFF), x)       # sign-magnitude -> ordered integers
    return (key(ia) - key(ib)).abs()


@pytest.mark.parametrize("geo", [Geometry(2, 8, 2, 128, 16), Geometry(1, 4, 2, 64, 16)])
def test_rope_append_and_attention_match_oracle(geo):
    import torch
    from paper_2502_11517_b200 import binding, build
    from lib_replay import LibReplay, make_pool
    build()
    script = random_script(77, n_ops=80, geo=geo, predictions=True)
    pool = make_pool(script)
    rep = LibReplay(script, pool, rope_theta=THETA)
    model = PoolModel(script.n_pages, geo.page_size, script.free_order)
    layers = list(range(geo.n_layers))
    stores = {l: KVStore(script.n_pages, geo.page_size, geo.n_kv_heads, geo.head_dim) for l in layers}
    n_steps = 0
    for i, op in enumerate(script.ops):
        kind = op[0]
        got = rep.apply(i)
        if kind == "begin":
            model.request_begin()
        elif kind == "end":
            model.request_end(op[1])
        elif kind == "spawn":
            model.thread_spawn(op[1], op[3])
        elif kind == "finish":
            model.thread_finish(op[1], op[2])
        elif kind == "merge":
            model.sync_merge(op[1], None if op[2] is None else list(op[2]))
        elif kind == "run":
            pos0 = model.requests[op[1]].pos_next[op[2]]
            slots = model.append_run(op[1], op[2], op[3])
            for l in layers:
                k, v = run_tensors(script, i, l)
                stores[l].write(slots, rope_bf16(k, np.arange(pos0, pos0 + op[3]), THETA), v)
        elif kind == "step":
            slots = [s for s in model.reserve(op[1]) if s is not None]
            pos_q = [model.last_position(e[0], e[1]) for e in op[1]]
            assert pool.step_positions().tolist() == pos_q
            pos_app = [p for p, e in zip(pos_q, op[1]) if e[2]]
            out, lse = got
            for l in layers:
                k, v, q = step_tensors(script, i, l)
                stores[l].write(slots, rope_bf16(k, pos_app, THETA), v)
                want, want_lse = decode_attention(model, stores[l], [(e[0], e[1]) for e in op[1]], rope_bf16(q, pos_q, THETA))
                err = np.abs(out[l].double().cpu().numpy() - want)
                assert err.max() <= 1e-2 and err.mean() <= 1e-3, (i, l, err.max(), err.mean())
            n_steps += 1
    assert n_steps and pool.dump() == model.dump()
    # the stored keys themselves
    worst, total, differ = 0, 0, 0
    for req, r in pool.dump()["requests"].items():
        for sid, st in r["streams"].items():
            if st["len"] == 0:
                continue
            slots = [(st["pages"][t // 16], t % 16) for t in range(st["len"])]
            for l in layers:
                k, v = pool.kv_read(l, req, sid, 0, st["len"])
                wk, wv = stores[l].gather(slots)
                d = _ulp_distance(k.cpu(), torch.from_numpy(wk).to(torch.bfloat16))
                worst = max(worst, int(d.max())); total += d.numel(); differ += int((d > 0).sum())
                assert np.array_equal(v.float().cpu().numpy().astype(np.float64), wv)       # V is a bit copy
    assert worst <= 1 and differ <= total * 1e-3, (worst, differ, total)
    assert pool.status() == 0
    print(f"rope keys: {differ} of {total} elements differ by one bf16 ulp, none by more")
    pool.close()
