"""Comparison layout: the paper's own (Section 3 "Efficiency", Fig. 2b/2c).

One dense, token-granular KV pool per response.  Tokens enter it in the order they are decoded, so the tokens of
concurrently decoding threads interleave; nothing is ever moved.  What a thread may attend to is a boolean mask row
over the pool's slots: a fork starts from a copy of the main thread's row (the main-thread tokens that existed when
it was spawned), every thread adds the slots it decodes itself, and <sync/> adds the merged forks' own slots to the
main thread's row.  Attention is masked attention over the whole pool for every query
(pasta_dense_mask_attn): each thread reads every slot, the mask decides what counts.

This object only holds the tensors and mirrors a workload script's operations; the kernels are the library's.
Single-layer use is enough for the comparison it exists for (`bench.py --layout dense_mask`, tests).
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

from . import binding


class DensePool:
    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, max_slots: int, max_threads: int, device="cuda"):
        import torch
        self.torch = torch
        self.n_q_heads, self.n_kv_heads, self.head_dim = n_q_heads, n_kv_heads, head_dim
        self.max_slots, self.max_threads, self.device = max_slots, max_threads, device
        self.req: Dict[int, dict] = {}
        self.scratch = None
        self._rows: Dict[tuple, object] = {}
        self.bytes_read_last_step = 0

    # ---- the operations of a workload script
    def begin(self, req: int) -> None:
        t = self.torch
        self.req[req] = {
            "k": t.zeros((self.max_slots, self.n_kv_heads, self.head_dim), dtype=t.bfloat16, device=self.device),
            "v": t.zeros((self.max_slots, self.n_kv_heads, self.head_dim), dtype=t.bfloat16, device=self.device),
            "mask": t.zeros((self.max_threads, self.max_slots), dtype=t.uint8, device=self.device),
            "own": t.zeros((self.max_threads, self.max_slots), dtype=t.uint8, device=self.device),
            "n": 0,
        }

    def _append(self, r: dict, rows: Sequence[int], k, v) -> None:
        done = 0
        while done < len(rows):                        # the append call takes 64 tokens at a time
            cnt = min(64, len(rows) - done)
            if r["n"] + cnt > self.max_slots:
                raise RuntimeError("dense pool is full")
            binding.dense_append(r["k"], r["v"], r["mask"], r["own"], r["n"], rows[done:done + cnt],
                                 k[done:done + cnt].contiguous(), v[done:done + cnt].contiguous())
            r["n"] += cnt
            done += cnt

    def run(self, req: int, thread: int, m: int, k, v) -> None:
        """m tokens of one thread (k, v: [m, Hkv, d], one layer) enter the pool at the next m slots."""
        if m:
            self._append(self.req[req], [thread] * m, k, v)

    def spawn(self, req: int, thread: int) -> None:
        r = self.req[req]
        r["mask"][thread].copy_(r["mask"][0])          # the main thread's view at this moment; nothing else is copied
        r["own"][thread].zero_()

    def merge(self, req: int, forks: Sequence[int]) -> None:
        r = self.req[req]
        for t in forks:
            r["mask"][0] |= r["own"][t]                # <sync/>: a mask change, no KV moves

    def step(self, entries: Sequence[Tuple[int, int, int]], k_new, v_new, q, out, lse=None) -> None:
        """One decode step.  entries: (request, thread, n_new in {0, 1}); k_new, v_new: [appended tokens, Hkv, d];
        q, out: [len(entries), Hq, d] (out fp32); lse: [len(entries), Hq] or None.  Tokens enter their request's pool
        in entry order (interleaved across threads), then every query attends over its request's whole pool."""
        t = self.torch
        by_req: Dict[int, List[int]] = {}
        for i, (req, _th, _n) in enumerate(entries):
            by_req.setdefault(req, []).append(i)
        app_index = {}
        a = 0
        for i, (_r, _th, n) in enumerate(entries):
            assert n in (0, 1), "one token per entry in this layout object"
            if n:
                app_index[i] = a
                a += 1
        self.bytes_read_last_step = 0
        for req, idx in by_req.items():
            r = self.req[req]
            new = [i for i in idx if i in app_index]
            if new:
                ai = [app_index[i] for i in new]
                if ai == list(range(ai[0], ai[0] + len(ai))):
                    kn, vn = k_new[ai[0]:ai[0] + len(ai)], v_new[ai[0]:ai[0] + len(ai)]
                else:
                    sel = t.tensor(ai, device=self.device)
                    kn, vn = k_new[sel], v_new[sel]
                self._append(r, [entries[i][1] for i in new], kn, vn)
            key = (req, tuple(entries[i][1] for i in idx))
            rows = self._rows.get(key)
            if rows is None:                           # the same threads step again and again: upload their rows once
                rows = self._rows[key] = t.tensor(key[1], dtype=t.int32, device=self.device)
            contiguous = idx == list(range(idx[0], idx[0] + len(idx)))
            qr = q[idx[0]:idx[0] + len(idx)] if contiguous else q[t.tensor(idx, device=self.device)].contiguous()
            orr = out[idx[0]:idx[0] + len(idx)] if contiguous else t.empty_like(qr, dtype=t.float32)
            lr = None
            if lse is not None:
                lr = lse[idx[0]:idx[0] + len(idx)] if contiguous else t.empty(qr.shape[:2], dtype=t.float32, device=self.device)
            need = binding.dense_mask_scratch_bytes(len(idx), r["n"], self.n_q_heads, self.n_kv_heads, self.head_dim)
            if self.scratch is None or self.scratch.numel() < need:
                self.scratch = t.empty(need * 2, dtype=t.uint8, device=self.device)
            binding.dense_mask_attn(r["k"], r["v"], r["mask"], rows, qr, orr, lr, self.scratch, r["n"])
            if not contiguous:
                sel = t.tensor(idx, device=self.device)
                out[sel] = orr
                if lse is not None:
                    lse[sel] = lr
            # every query walks every slot of its request's pool: K and V rows plus a mask byte per slot
            self.bytes_read_last_step += len(idx) * r["n"] * (2 * self.n_kv_heads * self.head_dim * 2 + 1)

    def end(self, req: int) -> None:
        self.req.pop(req, None)
