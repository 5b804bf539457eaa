"""Pins for the oracle's position ids (Section 6 "Positional Embedding": exact prediction -> consecutive ids,
too few -> ids not monotone after sync, too many -> a gap) and for its rotary embedding (complex-number form,
the cos/sin + rotate-half form, relative-position property, norm preservation)."""
import numpy as np
import pytest
import torch

from oracle import PoolModel, rope, rope_bf16


def _logical_positions(m, req, pos_of):
    """Position ids of the main thread's visible tokens in logical (annotation) order."""
    out = []
    for s, a, n in m.view(req, 0):
        out.extend(pos_of[(s, k)] for k in range(a, a + n))
    return out


def _append(m, req, t, n, pos_of):
    for _ in range(n):
        m.append_run(req, t, 1)
        k = m.requests[req].stream_len[t] - 1
        pos_of[(t, k)] = m.last_position(req, t)


def _scenario(pred_a, pred_b, len_a=7, len_b=12):
    m = PoolModel(256, 16)
    req = m.request_begin()
    pos_of = {}
    _append(m, req, 0, 20, pos_of)                      # prompt ... <promise/> #a is the 20th token
    a = m.thread_spawn(req, pred_a)
    _append(m, req, 0, 5, pos_of)                       # main continues ... <promise/> #b
    b = m.thread_spawn(req, pred_b)
    _append(m, req, 0, 3, pos_of)
    _append(m, req, a, len_a, pos_of); _append(m, req, b, len_b, pos_of)
    m.thread_finish(req, a); m.thread_finish(req, b); m.sync_merge(req)
    _append(m, req, 0, 4, pos_of)                       # <sync/> and what follows
    return _logical_positions(m, req, pos_of)


def test_no_forks_positions_are_consecutive():
    m = PoolModel(64, 16); r = m.request_begin(); pos_of = {}
    _append(m, r, 0, 40, pos_of)
    assert _logical_positions(m, r, pos_of) == list(range(40))


def test_exact_prediction_gives_consecutive_positions_after_sync():
    pos = _scenario(7, 12)
    assert pos == list(range(len(pos)))


def test_predicting_too_many_leaves_a_gap():
    pos = _scenario(10, 20)              # Pred-10X style: 7 -> 10, 12 -> 20
    d = np.diff(pos)
    assert np.all(d >= 1)                # still increasing ...
    assert sorted(d[d > 1].tolist()) == [4, 9]      # ... with gaps of 10 - 7 + 1 and 20 - 12 + 1


def test_predicting_too_few_is_not_monotone():
    pos = _scenario(3, 12)               # the first chunk is 4 tokens longer than predicted
    d = np.diff(pos)
    assert (d < 1).sum() == 1 and d.min() == -(7 - 3) + 1


def test_fork_starts_right_after_its_promise_and_main_skips_the_prediction():
    m = PoolModel(64, 16); r = m.request_begin()
    m.append_run(r, 0, 10)                               # positions 0..9, the promise is token 9
    t = m.thread_spawn(r, 30)
    m.append_run(r, t, 1); m.append_run(r, 0, 1)
    assert m.last_position(r, t) == 10 and m.last_position(r, 0) == 40


# ------------------------------------------------------------------ rotary embedding
def _complex_form(x, pos, theta):
    n, H, d = x.shape
    z = x[..., : d // 2] + 1j * x[..., d // 2:]
    w = np.exp(1j * np.asarray(pos)[:, None] * theta ** (-2.0 * np.arange(d // 2) / d))
    y = z * w[:, None, :]
    return np.concatenate([y.real, y.imag], axis=-1)


def _rotate_half_form(x, pos, theta):
    x = torch.from_numpy(x)
    d = x.shape[-1]
    inv = 1.0 / (theta ** (torch.arange(0, d, 2, dtype=torch.float64) / d))
    ang = torch.as_tensor(pos, dtype=torch.float64)[:, None] * inv[None, :]
    emb = torch.cat([ang, ang], dim=-1)[:, None, :]
    rot = torch.cat([-x[..., d // 2:], x[..., : d // 2]], dim=-1)
    return (x * emb.cos() + rot * emb.sin()).numpy()


@pytest.mark.parametrize("theta", [10000.0, 500000.0])
def test_rope_matches_two_other_formulations(theta):
    rng = np.random.default_rng(3)
    x = rng.standard_normal((9, 3, 16)); pos = np.array([0, 1, 2, 7, 40, 41, 1000, 32767, 131071])
    y = rope(x, pos, theta)
    np.testing.assert_allclose(y, _complex_form(x, pos, theta), atol=1e-9)
    np.testing.assert_allclose(y, _rotate_half_form(x, pos, theta), atol=1e-9)


def test_rope_properties():
    rng = np.random.default_rng(4)
    q = rng.standard_normal((1, 2, 32)); k = rng.standard_normal((1, 2, 32))
    assert np.array_equal(rope(q, [0]), q)                                   # position 0 is the identity
    np.testing.assert_allclose(np.linalg.norm(rope(q, [123]), axis=-1), np.linalg.norm(q, axis=-1), rtol=1e-12)
    base = (rope(q, [5]) * rope(k, [2])).sum(-1)
    for shift in (1, 17, 4000):                                             # scores depend on the distance only
        np.testing.assert_allclose((rope(q, [5 + shift]) * rope(k, [2 + shift])).sum(-1), base, atol=1e-9)
    assert abs((rope(q, [6]) * rope(k, [2])).sum() - base.sum()) > 1e-3     # ... and do depend on it


def test_rope_bf16_rounds_the_float64_result():
    x = torch.randn(4, 2, 64, generator=torch.Generator().manual_seed(0)).to(torch.bfloat16)
    y = rope_bf16(x, [3, 4, 5, 6])
    want = torch.from_numpy(rope(x.double().numpy(), [3, 4, 5, 6])).to(torch.bfloat16)
    assert y.dtype == torch.bfloat16 and torch.equal(y, want)
