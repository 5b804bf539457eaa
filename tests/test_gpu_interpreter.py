"""GPU parity through the interpreter: the library decodes a multi-thread response step by step (scripted tokens,
seeded K/V/Q per token), the oracle follows the paper's timeline on its own; attention outputs of every thread at
every step must agree within the stated tolerance, bookkeeping exactly."""
import numpy as np
import pytest

from oracle import KVStore, PoolModel, decode_attention, paper_timeline
from pasta_workloads import Geometry, token_tensors
from test_interpreter import Scripted, random_threads
from test_interpreter_model import CLOSE, OPEN, PROMISE, SYNC, TAGS, fig2_scripts

pytestmark = pytest.mark.gpu
MAX_ABS, MEAN_ABS = 1e-2, 1e-3
SEED = 4242


def oracle_side(geo, prompt, emissions, n_pages):
    model = PoolModel(n_pages, geo.page_size)
    stores = [KVStore(n_pages, geo.page_size, geo.n_kv_heads, geo.head_dim) for _ in range(geo.n_layers)]
    fed_count = {}
    results = {}

    def slot_of_newest(t):
        r = model.requests[0]
        k = r.stream_len[t] - 1
        return (r.stream_pages[t][k // geo.page_size], k % geo.page_size)

    def write(t, layer_tensors):
        for l in range(geo.n_layers):
            k, v, _q = layer_tensors[l]
            stores[l].write([slot_of_newest(t)], k[None], v[None])

    def on_T(T, entered):
        if T == 1:      # the prompt went in as a run before T=1: write its KV now (slots are known from the pages)
            r = model.requests[0]
            for i in range(len(prompt)):
                for l in range(geo.n_layers):
                    k, v, _ = token_tensors(SEED, geo, 0, i, l)
                    stores[l].write([(r.stream_pages[0][i // geo.page_size], i % geo.page_size)], k[None], v[None])
            fed_count[0] = len(prompt)
        qs = []
        for t, _tok in entered:
            i = fed_count.get(t, 0); fed_count[t] = i + 1
            tens = [token_tensors(SEED, geo, t, i, l) for l in range(geo.n_layers)]
            write(t, tens)
            qs.append(tens)
        for l in range(geo.n_layers):
            import torch
            q = torch.stack([tens[l][2] for tens in qs])
            out, lse = decode_attention(model, stores[l], [(0, t) for t, _ in entered], q)
            for row, (t, _tok) in enumerate(entered):
                results[(T, t, l)] = (out[row], lse[row])

    paper_timeline(model, prompt, emissions, predicted_length=lambda k: 10, on_timestamp=on_T, **TAGS)
    return results, model


def library_side(geo, prompt, emissions, n_pages, n_steps, flags=0):
    import torch
    from paper_2502_11517_b200 import binding
    from paper_2502_11517_b200.build import build
    from paper_2502_11517_b200.interpreter import Interpreter, Tags
    build()
    pool = binding.Pool(geo.n_layers, geo.n_q_heads, geo.n_kv_heads, geo.head_dim, n_pages, 2, 16, 64, flags=flags)
    it = Interpreter(pool, Tags(PROMISE, OPEN, CLOSE, SYNC), predicted_length=lambda req, k: 10)
    L, n0 = geo.n_layers, len(prompt) - 1
    pre = [[token_tensors(SEED, geo, 0, i, l) for i in range(n0)] for l in range(L)]
    k0 = torch.stack([torch.stack([x[0] for x in pre[l]]) for l in range(L)]).cuda()
    v0 = torch.stack([torch.stack([x[1] for x in pre[l]]) for l in range(L)]).cuda()
    req = it.add_request(prompt, k0, v0)
    fake = Scripted(emissions)
    fed_count = {0: n0}
    results = {}
    for step in range(1, n_steps + 1):
        entries = it.begin_step()
        tens = []
        for _r, t, _tok in entries:
            i = fed_count.get(t, 0); fed_count[t] = i + 1
            tens.append([token_tensors(SEED, geo, t, i, l) for l in range(L)])
        k = torch.stack([torch.stack([x[l][0] for x in tens]) for l in range(L)]).cuda()
        v = torch.stack([torch.stack([x[l][1] for x in tens]) for l in range(L)]).cuda()
        q = torch.stack([torch.stack([x[l][2] for x in tens]) for l in range(L)]).cuda()
        out = torch.empty((L, len(entries), geo.n_q_heads, geo.head_dim), dtype=torch.float32, device="cuda")
        lse = torch.empty((L, len(entries), geo.n_q_heads), dtype=torch.float32, device="cuda")
        pool.kv_append(k, v)
        pool.decode_attn(q, out, lse)
        torch.cuda.synchronize()
        assert pool.status() == 0
        for row, (_r, t, _tok) in enumerate(entries):
            for l in range(L):
                results[(step - 1, t, l)] = (out[l, row].double().cpu().numpy(), lse[l, row].double().cpu().numpy())
        it.end_step(fake(entries))
    launches = pool.launch_count() if hasattr(pool, "launch_count") else None
    dump = pool.dump()
    pool.close()
    return results, dump, launches


def compare(geo, prompt, emissions, flags=0):
    want, model = oracle_side(geo, prompt, emissions, 256)
    T_max = max(T for T, _t, _l in want)
    got, dump, _ = library_side(geo, prompt, emissions, 256, T_max + 1, flags)
    worst = 0.0
    n = 0
    for key, (o, l) in want.items():
        g_o, g_l = got[key]
        err = np.abs(g_o - o)
        assert np.all(np.isfinite(g_o)), key
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (key, err.max(), err.mean())
        assert np.abs(g_l - l).max() <= 1e-2, key
        worst = max(worst, err.max()); n += 1
    print(f"interpreter parity: {n} (timestamp, thread, layer) rows, worst max-abs {worst:.2e}")
    want_dump = model.dump()
    for d in (dump, want_dump):
        for r in d["requests"].values():
            for th in r["threads"].values():
                th.pop("state")
    assert dump == want_dump


def test_fig2_through_interpreter_tensor_path():
    ids, prompt, emissions = fig2_scripts()
    prompt = list(range(1000, 1000 + 700)) + prompt          # a prefix long enough for several tiles
    compare(Geometry(2, 32, 8, 128, 16), prompt, emissions)


def test_fig2_through_interpreter_warp_path():
    from paper_2502_11517_b200 import binding
    ids, prompt, emissions = fig2_scripts()
    compare(Geometry(2, 8, 2, 64, 16), prompt, emissions)
    compare(Geometry(1, 32, 8, 128, 16), list(range(1000, 1300)) + prompt, emissions, flags=binding.FLAG_NO_TENSOR_PATH)


@pytest.mark.parametrize("seed", [3, 8, 11])
def test_random_threads_through_interpreter(seed):
    prompt, emissions = random_threads(seed)
    compare(Geometry(2, 32, 8, 128, 16), list(range(1000, 1400)) + prompt, emissions)
