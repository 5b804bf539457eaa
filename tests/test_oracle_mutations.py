"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's source (on the CPU) and
checks that at least one pin then fails.  The unmodified copy must pass all of them."""
import importlib
import os
import shutil
import sys
import tempfile

import numpy as np
import pytest

from pasta_workloads import Geometry, Script, random_script, run_tensors, step_tensors
from formulations import TokenGraph

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

MUTATIONS = [
    ("attention.py", "g = h // group", "g = h % k.shape[1]"),                       # query head -> kv head map
    ("attention.py", "scale = 1.0 / np.sqrt(d)", "scale = 1.0 / d"),                  # softmax scale
    ("attention.py", "w = e / z", "w = e / e.max()"),                                 # normalisation
    ("attention.py", "o[h] = w @ v[:, g, :]", "o[h] = w @ k[:, g, :]"),               # values
    ("attention.py", "lse[h] = m + np.log(z)", "lse[h] = np.log(z)"),                 # log-sum-exp
    ("pool_model.py", "r.view[t] = [list(e) for e in r.view[0]]", "r.view[t] = []"),  # fork forgets the prefix
    ("pool_model.py", "r.cutoff[t] = r.stream_len[0]", "r.cutoff[t] = max(r.stream_len[0] - 1, 0)"),   # cut-off off by one
    ("pool_model.py", "if k % self.page_size == 0:", "if (k + 1) % self.page_size == 0 or not r.stream_pages[stream]:"),  # paging
    ("pool_model.py", "(anchor == p and s > t)", "(anchor == p and s < t)"),          # tie order of merged chunks
    ("pool_model.py", "for k in range(a, end))", "for k in range(a, end - 1))"),      # last token of a piece dropped
    ("pool_model.py", "self.free.insert(0, page)", "self.free.append(page)"),         # where freed pages go
    ("pool_model.py", "if s == 0 and a < p < a + ln:", "if s == 0 and a < p <= a + ln:"),   # split at a piece's end
    ("pool_model.py", "own_end = r.stream_len[thread] - hide", "own_end = r.stream_len[thread]"),   # later tokens of the step seen
    ("pool_model.py", "max(1, n_new) - 1 - j)", "j)"),                                 # hide counts from the wrong end
]


def _load(mutation):
    tmp = tempfile.mkdtemp(prefix="oracle_mut_")
    name = "oracle_copy_%d" % (abs(hash((mutation, tmp))) % 10**9)
    dst = os.path.join(tmp, name)
    shutil.copytree(os.path.join(ROOT, "oracle"), dst, ignore=shutil.ignore_patterns("__pycache__"))
    if mutation is not None:
        fname, old, new = mutation
        path = os.path.join(dst, fname)
        src = open(path).read()
        assert src.count(old) == 1, (fname, old, src.count(old))
        open(path, "w").write(src.replace(old, new))
    sys.path.insert(0, tmp)
    try:
        return importlib.import_module(name)
    finally:
        sys.path.remove(tmp)


def _manual(ops, geo=None, n_pages=64):
    geo = geo or Geometry(1, 4, 2, 8, 4)
    return Script("manual", geo, n_pages, np.arange(n_pages, dtype=np.int32), 8, 16, 64, 7, list(ops))


def _pins(O):
    """A compact copy of the pins of test_oracle_pins.py / test_pool_model.py, run against module O."""
    # token-graph formulation on random scripts
    for seed in (0, 1, 5):
        script = random_script(seed, paper_flow=bool(seed % 2))
        ours = {i: r[0] for i, r in O.OracleReplay(script).run_all().items()}
        theirs = TokenGraph(script).run_all()
        for i in ours:
            np.testing.assert_allclose(ours[i][0], theirs[i][0], rtol=0, atol=1e-12)
            np.testing.assert_allclose(ours[i][1], theirs[i][1], rtol=0, atol=1e-12)
    # closed forms: scale and head map
    d = 16
    k = np.zeros((2, 1, d)); k[0, 0, 0] = 1.0
    v = np.zeros((2, 1, d)); v[0, 0, 0] = 1.0; v[1, 0, 1] = 1.0
    q = np.zeros((1, d)); q[0, 0] = np.log(3.0) * np.sqrt(d)
    o, lse, w = O.attend(q, k, v)
    np.testing.assert_allclose(w[0], [0.75, 0.25], atol=1e-14)
    np.testing.assert_allclose(o[0, :2], [0.75, 0.25], atol=1e-14)
    assert abs(lse[0] - np.log(4.0)) < 1e-13
    rng = np.random.default_rng(5)
    n, hkv, hq = 9, 2, 6
    k3 = np.zeros((n, hkv, 8)); k3[4, 1, 0] = 200.0
    v3 = rng.standard_normal((n, hkv, 8))
    qq = np.zeros((hq, 8)); qq[:, 0] = 1.0
    o3, _, _ = O.attend(qq, k3, v3)
    for h in range(hq):
        np.testing.assert_allclose(o3[h], v3[4, 1] if h >= 3 else v3[:, 0].mean(0), atol=1e-12)
    # integer rules
    m = O.PoolModel(8, 16, [5, 2, 7, 0, 1, 3, 4, 6])
    r = m.request_begin()
    slots = m.append_run(r, 0, 32)
    assert slots[0] == (5, 0) and slots[16] == (2, 0) and m.free == [7, 0, 1, 3, 4, 6]
    m = O.PoolModel(8, 4, list(range(8)))
    r = m.request_begin(); m.append_run(r, 0, 6); t = m.thread_spawn(r); m.append_run(r, t, 9); m.request_end(r)
    assert m.free == [4, 3, 2, 1, 0, 5, 6, 7]
    m = O.PoolModel(64, 4)
    r = m.request_begin(); m.append_run(r, 0, 10)
    a = m.thread_spawn(r); m.append_run(r, 0, 5)
    b = m.thread_spawn(r); c = m.thread_spawn(r); m.append_run(r, 0, 2)
    for t, cnt in ((a, 3), (b, 4), (c, 2)):
        m.append_run(r, t, cnt); m.thread_finish(r, t)
    m.sync_merge(r, [c]); m.sync_merge(r, [b]); m.sync_merge(r, [a])
    assert m.view(r, 0) == [(0, 0, 10), (a, 0, 3), (0, 10, 5), (b, 0, 4), (c, 0, 2), (0, 15, 2)]
    assert len(m.visible_slots(r, 0)) == 26
    # a fork spawned exactly at the end of a main piece, merged: the chunk goes after that piece, nothing is split
    m = O.PoolModel(64, 4)
    r = m.request_begin(); m.append_run(r, 0, 4); f1 = m.thread_spawn(r); m.append_run(r, f1, 1); m.thread_finish(r, f1)
    m.sync_merge(r, [f1])
    assert m.view(r, 0) == [(0, 0, 4), (f1, 0, 1)]
    # several tokens of a thread in one step = the same tokens one step at a time
    rng = np.random.default_rng(11)
    ms = [O.PoolModel(64, 4), O.PoolModel(64, 4)]
    st = [O.KVStore(64, 4, 1, 4), O.KVStore(64, 4, 1, 4)]
    k0, v0 = rng.standard_normal((5, 1, 4)), rng.standard_normal((5, 1, 4))
    for mm, ss in zip(ms, st):
        r = mm.request_begin(); ss.write(mm.append_run(r, 0, 5), k0, v0)
    k, v, q = rng.standard_normal((3, 1, 4)), rng.standard_normal((3, 1, 4)), rng.standard_normal((3, 2, 4))
    st[0].write(ms[0].reserve([(0, 0, 3)]), k, v)
    out, _ = O.decode_attention(ms[0], st[0], O.PoolModel.queries_of([(0, 0, 3)]), q)
    for j in range(3):
        st[1].write(ms[1].reserve([(0, 0, 1)]), k[j:j + 1], v[j:j + 1])
        o1, _ = O.decode_attention(ms[1], st[1], [(0, 0)], q[j:j + 1])
        np.testing.assert_allclose(out[j], o1[0], rtol=0, atol=1e-12)


def test_unmodified_copy_passes_every_pin():
    _pins(_load(None))


@pytest.mark.parametrize("mutation", MUTATIONS, ids=[m[2][:40] for m in MUTATIONS])
def test_planted_mistake_is_caught(mutation):
    O = _load(mutation)
    with pytest.raises((AssertionError, IndexError, KeyError, ValueError, ZeroDivisionError, FloatingPointError)):
        with np.errstate(all="ignore"):
            _pins(O)
