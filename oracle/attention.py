"""Oracle, part 2: KV storage and decode attention in fp64.  TEST INFRASTRUCTURE — not a product path.

For every query (request, thread) and query head h, with kv head g = h // (Hq / Hkv):

    visible = the thread's visible tokens, gathered one by one through the oracle's own page
              tables and concatenated into dense arrays K, V            (the paper fixes this set:
              Section 3 "Efficiency", the visibility rule illustrated in Fig. 2b)
    s = K q / sqrt(d)            w = exp(s - max s) / sum exp(s - max s)          o = w V
    lse = max s + log sum exp(s - max s)

The attention formula itself is ordinary scaled-dot-product attention (the paper prints none);
inputs are bf16 values widened exactly, all arithmetic is float64.  No blocking, no sharing of
the prefix between threads, no split or merge: the visible K/V of every thread is materialised.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np

from .pool_model import PoolModel


def _to_f32(x) -> np.ndarray:
    """Accept a torch tensor (any float dtype, bf16 included) or an array; bf16 -> fp32 is exact."""
    if hasattr(x, "detach"):
        import torch
        return x.detach().to("cpu", torch.float32).numpy()
    return np.asarray(x, dtype=np.float32)


class KVStore:
    """K and V of one layer: [n_pages, page_size, Hkv, d], kept as fp32 (exact for bf16 inputs)."""

    def __init__(self, n_pages: int, page_size: int, n_kv_heads: int, head_dim: int):
        self.k = np.zeros((n_pages, page_size, n_kv_heads, head_dim), dtype=np.float32)
        self.v = np.zeros((n_pages, page_size, n_kv_heads, head_dim), dtype=np.float32)

    def write(self, slots: Sequence[Tuple[int, int]], k_new, v_new) -> None:
        """Store token i of k_new / v_new ([m, Hkv, d]) at slots[i] = (page, offset)."""
        k_new, v_new = _to_f32(k_new), _to_f32(v_new)
        assert len(slots) == k_new.shape[0] == v_new.shape[0]
        if not slots:
            return
        idx = np.asarray(slots, dtype=np.int64)
        self.k[idx[:, 0], idx[:, 1]] = k_new
        self.v[idx[:, 0], idx[:, 1]] = v_new

    def gather(self, slots: Sequence[Tuple[int, int]]):
        """Dense fp64 K, V ([n_visible, Hkv, d]) of the listed slots, in the order given."""
        idx = np.asarray(slots, dtype=np.int64).reshape(-1, 2)
        return (self.k[idx[:, 0], idx[:, 1]].astype(np.float64),
                self.v[idx[:, 0], idx[:, 1]].astype(np.float64))


def attend(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: Optional[float] = None):
    """One query over a dense visible set.  q: [Hq, d]; k, v: [n, Hkv, d] (fp64).

    Returns (o [Hq, d], lse [Hq], w [Hq, n]) — w are the softmax weights."""
    n_q_heads, d = q.shape
    group = n_q_heads // k.shape[1]
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    o = np.empty((n_q_heads, d), dtype=np.float64)
    lse = np.empty(n_q_heads, dtype=np.float64)
    w_all = np.empty((n_q_heads, k.shape[0]), dtype=np.float64)
    for h in range(n_q_heads):
        g = h // group
        s = (k[:, g, :] @ q[h]) * scale
        m = s.max()
        e = np.exp(s - m)
        z = e.sum()
        w = e / z
        o[h] = w @ v[:, g, :]
        lse[h] = m + np.log(z)
        w_all[h] = w
    return o, lse, w_all


def decode_attention(model: PoolModel, store: KVStore, queries: Sequence[Tuple[int, int]], q,
                     scale: Optional[float] = None, return_weights: bool = False):
    """Attention of one decode step for one layer.

    queries: (request, thread) or (request, thread, hide) per row of q ([n, Hq, d]); hide = newest tokens of the
    thread the query does not see (PoolModel.queries_of).  Returns out [n, Hq, d] fp64 and
    lse [n, Hq] fp64 (and the list of weight arrays when asked)."""
    q = _to_f32(q).astype(np.float64)
    out = np.empty(q.shape, dtype=np.float64)
    lse = np.empty(q.shape[:2], dtype=np.float64)
    weights: List[np.ndarray] = []
    for i, qr in enumerate(queries):
        k, v = store.gather(model.visible_slots(*qr))
        out[i], lse[i], w = attend(q[i], k, v, scale)
        if return_weights:
            weights.append(w)
    return (out, lse, weights) if return_weights else (out, lse)
