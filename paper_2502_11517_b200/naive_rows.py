"""Comparison layout: every thread a dense row of its own (paper, Appendix B, the second design it describes and
sets aside; Section 3 "Efficiency" names its costs).

Each thread of a response is stored as a separate sequence: when a fork is spawned, the main thread's row is
DUPLICATED into the fork's row; at <sync/> each finished chunk is COPIED into the main thread's row.  Attention is
then plain causal decode attention over one row per thread.  Here the rows are ordinary fork-less requests of the
same pool, served by the same kernels, so that what is measured is the layout alone: the bytes a step reads
(the prefix once per thread instead of once per request) and the bytes spawn and sync move.

The copied chunk is appended at the end of the main row, not inserted behind its <promise/>: softmax attention does
not depend on the order of the keys, and position information is already inside K when rotary embedding is used, so
the result is the same while no tail has to be shifted (an insertion would move even more bytes).
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple


class NaiveRows:
    COPY_CHUNK = 4096        # tokens per device-to-device copy call (bounds the transient buffers)

    def __init__(self, pool):
        self.pool = pool
        self.row: Dict[Tuple[int, int], int] = {}        # (request, thread) -> the pool request that holds its row
        self.length: Dict[int, int] = {}                 # row -> tokens
        self.own_start: Dict[Tuple[int, int], int] = {}  # (request, fork) -> where its own chunk starts in its row
        self.bytes_copied_at_spawn = 0
        self.bytes_copied_at_sync = 0

    def _token_bytes(self) -> int:
        p = self.pool
        return 2 * p.n_kv_heads * p.head_dim * 2 * p.n_layers

    def _copy(self, src_row: int, start: int, m: int, dst_row: int) -> None:
        """Appends tokens [start, start + m) of src_row to dst_row, every layer, through the pool's own read and append."""
        import torch
        p = self.pool
        done = 0
        while done < m:
            cnt = min(self.COPY_CHUNK, m - done)
            ks, vs = zip(*[p.kv_read(l, src_row, 0, start + done, cnt) for l in range(p.n_layers)])
            p.kv_append_run(dst_row, 0, cnt, torch.stack(ks), torch.stack(vs))
            done += cnt
        self.length[dst_row] += m

    # ---- the operations of a workload script
    def begin(self, req: int) -> None:
        r = self.pool.request_begin()
        self.row[(req, 0)] = r
        self.length[r] = 0

    def spawn(self, req: int, thread: int) -> None:
        main = self.row[(req, 0)]
        r = self.pool.request_begin()
        self.row[(req, thread)] = r
        self.length[r] = 0
        self._copy(main, 0, self.length[main], r)                 # the duplicated prefix
        self.own_start[(req, thread)] = self.length[r]
        self.bytes_copied_at_spawn += self.length[r] * self._token_bytes()

    def run(self, req: int, thread: int, m: int, k, v) -> None:
        r = self.row[(req, thread)]
        if m:
            self.pool.kv_append_run(r, 0, m, k, v)
        self.length[r] += m

    def step(self, entries: Sequence[Tuple[int, int, int]], k_new, v_new, q, out, lse=None) -> None:
        rows = [self.row[(req, t)] for req, t, _n in entries]
        n_new = [n for _r, _t, n in entries]
        self.pool.step_begin(rows, [0] * len(rows), n_new)
        self.pool.kv_append(k_new, v_new)
        self.pool.decode_attn(q, out, lse)
        for r, n in zip(rows, n_new):
            self.length[r] += n

    def merge(self, req: int, forks: Sequence[int]) -> None:
        main = self.row[(req, 0)]
        for t in sorted(forks):
            r = self.row[(req, t)]
            m = self.length[r] - self.own_start[(req, t)]
            self._copy(r, self.own_start[(req, t)], m, main)
            self.bytes_copied_at_sync += m * self._token_bytes()

    def end(self, req: int) -> None:
        for key in [k for k in self.row if k[0] == req]:
            r = self.row.pop(key)
            self.pool.request_end(r)
            del self.length[r]
            self.own_start.pop(key, None)
