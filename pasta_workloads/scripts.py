"""Scripts: seeded sequences of pool operations plus the tensors they carry.

A script is a list of operations that a replayer applies, in order, to a KV
pool (the oracle's model or the CUDA library):

    ("begin",  req)                      a request starts; `req` is the id the replayer must hand out
    ("run",    req, thread, m)           m tokens are appended to one thread's stream (prefill / catch-up)
    ("spawn",  req, thread[, predicted[, pending]])
                                         the main thread emitted <promise/>; `thread` is the new fork's id; the optional
                                         fourth field is the block length predicted in the promise (position ids); a
                                         fifth field of 1 says that the promise is the main thread's next token, decoded
                                         but not appended yet
    ("step",   ((req, thread, n_new), …)) one decode step: every listed thread appends n_new >= 0 tokens and issues
                                         one attention query per new token (each blind to the later ones), or
                                         one query over what it sees already when n_new == 0
    ("finish", req, thread)              a fork emitted </async>
    ("merge",  req, threads | None)      <sync/>: merge the named finished forks (None = all finished ones)
    ("end",    req)                      the request is over, its pages return to the pool

Ids follow the convention both replayers implement on their own: a request gets
the lowest unused id, forks of a request are numbered 1, 2, 3, … in spawn order
and the main thread is 0.  Only lengths and ids are tracked here (bookkeeping to
emit valid scripts and to size the pool); what a thread may attend to is never
computed in this module.

Tensors are drawn from N(0, 1) in bf16 with a torch generator seeded from
(script seed, operation index, layer), so every (operation, layer) can be
regenerated independently and identically by whoever needs it.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

SEED = 25021151


@dataclass(frozen=True)
class Geometry:
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int = 16

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def kv_bytes_per_token(self) -> int:
        """bf16 K and V of one token in one layer."""
        return 2 * self.n_kv_heads * self.head_dim * 2


@dataclass
class Script:
    name: str
    geometry: Geometry
    n_pages: int
    free_order: np.ndarray
    max_requests: int
    max_threads_per_request: int
    max_segments_per_thread: int
    seed: int
    ops: List[tuple] = field(default_factory=list)
    notes: dict = field(default_factory=dict)


# --------------------------------------------------------------------------- tensors
def _gen(seed: int, op_index: int, layer: int, device: str = "cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + op_index * 7919 + layer * 104729) % (2**62))
    return g


def _randn_bf16(shape, g: torch.Generator, device: str) -> torch.Tensor:
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)


def token_tensors(seed: int, geo: "Geometry", thread: int, index: int, layer: int):
    """(k, v, q) of the index-th token a thread feeds to the model, for one layer: k, v [Hkv, d], q [Hq, d] bf16.
    For drivers that produce tokens one by one (no script): the tensors depend on who feeds the token and on
    its rank in that thread, on nothing else."""
    g = _gen(seed, thread * 1000003 + index, layer)
    return (_randn_bf16((geo.n_kv_heads, geo.head_dim), g, "cpu"), _randn_bf16((geo.n_kv_heads, geo.head_dim), g, "cpu"),
            _randn_bf16((geo.n_q_heads, geo.head_dim), g, "cpu"))


def run_tensors(script: Script, op_index: int, layer: int, device: str = "cpu"):
    """K and V ([m, Hkv, d] bf16 each) carried by the "run" operation `op_index` for one layer."""
    op = script.ops[op_index]
    assert op[0] == "run"
    geo = script.geometry
    g = _gen(script.seed, op_index, layer, device)
    shape = (op[3], geo.n_kv_heads, geo.head_dim)
    return _randn_bf16(shape, g, device), _randn_bf16(shape, g, device)


def step_tensors(script: Script, op_index: int, layer: int, device: str = "cpu"):
    """(k_new, v_new, q) of the "step" operation `op_index` for one layer.

    k_new, v_new: [number of appended tokens, Hkv, d]; q: [number of queries, Hq, d], where an entry
    with n_new tokens contributes max(1, n_new) queries (one per new token, or one over the existing view).
    """
    op = script.ops[op_index]
    assert op[0] == "step"
    geo = script.geometry
    g = _gen(script.seed, op_index, layer, device)
    n = sum(max(1, e[2]) for e in op[1])
    n_app = sum(e[2] for e in op[1])
    k = _randn_bf16((n_app, geo.n_kv_heads, geo.head_dim), g, device)
    v = _randn_bf16((n_app, geo.n_kv_heads, geo.head_dim), g, device)
    q = _randn_bf16((n, geo.n_q_heads, geo.head_dim), g, device)
    return k, v, q


# --------------------------------------------------------------------------- bookkeeping
class _Book:
    """Ids and stream lengths only — enough to emit valid scripts and count pages."""

    def __init__(self, page_size: int):
        self.page = page_size
        self.live = {}          # req -> {"len": {thread: tokens}, "next": next fork id, "active": set, "finished": set}
        self.pages_now = 0
        self.pages_peak = 0

    def begin(self) -> int:
        req = 0
        while req in self.live:
            req += 1
        self.live[req] = {"len": {0: 0}, "next": 1, "active": set(), "finished": set()}
        return req

    def add(self, req: int, thread: int, m: int) -> None:
        lens = self.live[req]["len"]
        before = -(-lens[thread] // self.page)
        lens[thread] += m
        self.pages_now += -(-lens[thread] // self.page) - before
        self.pages_peak = max(self.pages_peak, self.pages_now)

    def spawn(self, req: int) -> int:
        r = self.live[req]
        t = r["next"]
        r["next"] += 1
        r["len"][t] = 0
        r["active"].add(t)
        return t

    def finish(self, req: int, t: int) -> None:
        r = self.live[req]
        r["active"].remove(t)
        r["finished"].add(t)

    def merge(self, req: int, threads: Optional[Sequence[int]]) -> None:
        r = self.live[req]
        for t in (list(r["finished"]) if threads is None else threads):
            r["finished"].remove(t)

    def end(self, req: int) -> None:
        r = self.live.pop(req)
        self.pages_now -= sum(-(-n // self.page) for n in r["len"].values())


def _finalise(name, geo, ops, book, rng, seed, slack_pages=8, max_requests=None,
              max_threads=None, max_segments=None, notes=None) -> Script:
    n_pages = book.pages_peak + slack_pages
    free_order = rng.permutation(n_pages).astype(np.int32)
    n_req = 1 + max((op[1] for op in ops if op[0] == "begin"), default=0)
    n_thr = 1 + max((op[2] for op in ops if op[0] == "spawn"), default=0)
    return Script(
        name=name, geometry=geo, n_pages=int(n_pages), free_order=free_order,
        max_requests=max_requests or n_req,
        max_threads_per_request=max_threads or n_thr,
        max_segments_per_thread=max_segments or (2 * n_thr + 2),
        seed=seed, ops=ops, notes=notes or {},
    )


# --------------------------------------------------------------------------- the five configurations
def cfg1_tiny(variant: str = "base") -> Script:
    """Tiny single-layer step: 4 q heads / 2 kv heads, d 64, one request, 128-token prefix, 3 forks.

    variants: "base" (chunks 0/17/32 seen by attention, all cut-offs 128),
              "cutoffs" (forks spawned at 96/112/128), "chunk16", "chunk33",
              "append" (same lengths, but reached by a step that appends one token per thread).
    """
    geo = Geometry(1, 4, 2, 64, 16)
    seed = SEED + 1
    rng = np.random.default_rng(seed)
    book = _Book(geo.page_size)
    ops: List[tuple] = []
    req = book.begin()
    ops.append(("begin", req))
    chunks = {"base": (0, 17, 32), "cutoffs": (0, 17, 32), "chunk16": (0, 16, 32),
              "chunk33": (0, 33, 32), "append": (1, 17, 32)}[variant]
    append = variant == "append"
    forks = []
    if variant == "cutoffs":
        done = 0
        for cut in (96, 112, 128):
            ops.append(("run", req, 0, cut - done)); book.add(req, 0, cut - done); done = cut
            t = book.spawn(req); ops.append(("spawn", req, t)); forks.append(t)
    else:
        m = 127 if append else 128
        ops.append(("run", req, 0, m)); book.add(req, 0, m)
        for _ in range(3):
            t = book.spawn(req); ops.append(("spawn", req, t)); forks.append(t)
    for t, c in zip(forks, chunks):
        pre = c - 1 if append else c
        if pre > 0:
            ops.append(("run", req, t, pre)); book.add(req, t, pre)
    n_new = 1 if append else 0
    entries = tuple((req, t, n_new) for t in forks) + ((req, 0, n_new),)
    for e in entries:
        book.add(e[0], e[1], e[2])
    ops.append(("step", entries))
    return _finalise(f"cfg1_{variant}", geo, ops, book, rng, seed, slack_pages=64 - book.pages_peak)


def cfg2_single_request(variant: str = "a") -> Script:
    """One request, 32q/8kv heads, d 128: prefix 512 + 256, 4 forks with chunks U[20, 200].

    Step A: the 4 forks append one token each and attend, the main thread attends over its 768
    tokens.  Then every fork finishes, <sync/> merges them, the main thread appends the <sync/>
    token and attends over 769 + all chunks (step B).
    variant "a": every fork is spawned at 768; "b": cut-offs 512 + sorted U[1, 256].
    """
    geo = Geometry(1, 32, 8, 128, 16)
    seed = SEED + 2
    rng = np.random.default_rng(seed)
    book = _Book(geo.page_size)
    ops: List[tuple] = []
    req = book.begin(); ops.append(("begin", req))
    chunk_len = [int(x) for x in rng.integers(20, 201, 4)]
    cuts = [768] * 4 if variant == "a" else [512 + int(x) for x in np.sort(rng.integers(1, 257, 4))]
    forks, done = [], 0
    for cut in cuts:
        if cut > done:
            ops.append(("run", req, 0, cut - done)); book.add(req, 0, cut - done); done = cut
        t = book.spawn(req); ops.append(("spawn", req, t)); forks.append(t)
    if done < 768:
        ops.append(("run", req, 0, 768 - done)); book.add(req, 0, 768 - done)
    for t, c in zip(forks, chunk_len):
        ops.append(("run", req, t, c - 1)); book.add(req, t, c - 1)
    entries = tuple((req, t, 1) for t in forks) + ((req, 0, 0),)
    for e in entries:
        book.add(e[0], e[1], e[2])
    ops.append(("step", entries))
    for t in forks:
        ops.append(("finish", req, t)); book.finish(req, t)
    ops.append(("merge", req, None)); book.merge(req, None)
    book.add(req, 0, 1)
    ops.append(("step", ((req, 0, 1),)))
    return _finalise(f"cfg2{variant}", geo, ops, book, rng, seed, slack_pages=128 - book.pages_peak,
                     notes={"chunks": chunk_len, "cutoffs": cuts})


def _batched(name, geo, seed, n_requests, prefix_lo, prefix_hi, fork_draw, chunk_lo, chunk_hi,
             n_new) -> Script:
    rng = np.random.default_rng(seed)
    book = _Book(geo.page_size)
    ops: List[tuple] = []
    entries = []
    stats = {"prefix": [], "forks": [], "chunks": []}
    for _ in range(n_requests):
        req = book.begin(); ops.append(("begin", req))
        prefix = int(rng.integers(prefix_lo, prefix_hi + 1))
        n_forks = int(fork_draw(rng))
        chunk_len = [int(x) for x in rng.integers(chunk_lo, chunk_hi + 1, n_forks)]
        stats["prefix"].append(prefix); stats["forks"].append(n_forks); stats["chunks"].append(chunk_len)
        ops.append(("run", req, 0, prefix - n_new)); book.add(req, 0, prefix - n_new)
        forks = []
        # the forks are spawned one token before the main thread's current end when the step appends,
        # so that after the step every fork's cut-off trails the main stream by that one token
        for _c in chunk_len:
            t = book.spawn(req); ops.append(("spawn", req, t)); forks.append(t)
        for t, c in zip(forks, chunk_len):
            if c - n_new > 0:
                ops.append(("run", req, t, c - n_new)); book.add(req, t, c - n_new)
        for t in forks:
            entries.append((req, t, n_new))
        entries.append((req, 0, n_new))
    for e in entries:
        book.add(e[0], e[1], e[2])
    ops.append(("step", tuple(entries)))
    return _finalise(name, geo, ops, book, rng, seed, slack_pages=64, notes=stats)


def cfg3_batched(n_requests: int = 64, n_layers: int = 32, n_new: int = 0,
                 prefix_range=(256, 2048)) -> Script:
    """Batched serving step: prefix U[256, 2048], forks min(geometric(0.35) - 1, 8), chunks U[10, 300]."""
    geo = Geometry(n_layers, 32, 8, 128, 16)
    return _batched(f"cfg3_r{n_requests}_l{n_layers}", geo, SEED + 3, n_requests,
                    prefix_range[0], prefix_range[1],
                    lambda rng: min(int(rng.geometric(0.35)) - 1, 8), 10, 300, n_new)


def cfg4_long_prefix(n_requests: int = 8, prefix: int = 32768, n_forks: int = 16,
                     n_layers: int = 1, n_new: int = 0) -> Script:
    """Long shared prefix: `prefix` tokens shared by `n_forks` forks with chunks U[50, 400]."""
    geo = Geometry(n_layers, 32, 8, 128, 16)
    return _batched(f"cfg4_r{n_requests}_p{prefix}_f{n_forks}", geo, SEED + 4, n_requests,
                    prefix, prefix, lambda rng: n_forks, 50, 400, n_new)


def cfg5_trace(n_requests: int = 256, n_steps: int = 512, n_layers: int = 32,
               prompt_range=(64, 1024), p_promise: float = 0.02, mean_chunk: float = 80.0,
               overlap: bool = False) -> Script:
    """Synthetic interpreter trace.

    Every step, every request decodes one token on its main thread and on each unfinished fork.
    After the step: each active fork ends with probability 1/mean_chunk; the main thread draws a
    promise with probability p_promise and, if accepted, spawns U[2, 6] forks; a promise group whose
    forks have all ended is merged.  With overlap=False at most one group is outstanding per request
    (draws made meanwhile are taken from the generator and dropped, so the random stream is the same).
    """
    geo = Geometry(n_layers, 32, 8, 128, 16)
    seed = SEED + 5
    rng = np.random.default_rng(seed)
    book = _Book(geo.page_size)
    ops: List[tuple] = []
    groups = {}
    for _ in range(n_requests):
        req = book.begin(); ops.append(("begin", req))
        prompt = int(rng.integers(prompt_range[0], prompt_range[1] + 1))
        ops.append(("run", req, 0, prompt)); book.add(req, 0, prompt)
        groups[req] = []          # list of lists of fork ids, outstanding
    max_active = 1
    n_thread_tokens = 0
    for _step in range(n_steps):
        entries = []
        for req in range(n_requests):
            for t in sorted(book.live[req]["active"]):
                entries.append((req, t, 1))
            entries.append((req, 0, 1))
        for e in entries:
            book.add(e[0], e[1], 1)
        n_thread_tokens += len(entries)
        ops.append(("step", tuple(entries)))
        for req in range(n_requests):
            r = book.live[req]
            for t in sorted(r["active"]):
                if rng.random() < 1.0 / mean_chunk:
                    ops.append(("finish", req, t)); book.finish(req, t)
            promise = rng.random() < p_promise
            k = int(rng.integers(2, 7))
            if promise and (overlap or not groups[req]) and len(r["active"]) + k <= 16:
                grp = []
                for _ in range(k):
                    t = book.spawn(req); ops.append(("spawn", req, t)); grp.append(t)
                groups[req].append(grp)
            still = []
            for grp in groups[req]:
                if all(t in r["finished"] for t in grp):
                    ops.append(("merge", req, tuple(grp))); book.merge(req, grp)
                else:
                    still.append(grp)
            groups[req] = still
            max_active = max(max_active, 1 + len(r["active"]))
    return _finalise(f"cfg5_r{n_requests}_s{n_steps}_l{n_layers}", geo, ops, book, rng, seed,
                     slack_pages=64, notes={"thread_tokens": n_thread_tokens, "max_active": max_active})


# --------------------------------------------------------------------------- random small scripts (property tests)
def random_script(seed: int, geo: Optional[Geometry] = None, n_ops: int = 60, max_requests: int = 3,
                  max_forks: int = 5, paper_flow: bool = False, predictions: bool = False,
                  multi_token: bool = False) -> Script:
    """A random but valid operation sequence on a small pool.

    Exercises partial merges, merges of empty chunks, forks spawned after a merge, request reuse and
    steps mixing appending and attention-only entries.  With paper_flow=True the main thread always
    appends a token right after a merge before anything else happens to that request (the paper's
    <sync/> token), which is the situation the token-graph formulation of visibility describes.
    With multi_token=True about a third of the appending entries feed 2 to 5 tokens in their step.
    """
    geo = geo or Geometry(1, 4, 2, 8, 4)
    rng = np.random.default_rng(seed)
    book = _Book(geo.page_size)
    ops: List[tuple] = []
    need_sync_token = set()

    def do_step(reqs):
        entries = []
        for req in reqs:
            r = book.live[req]
            threads = sorted(r["active"]) + [0]
            picked = [t for t in threads if rng.random() < 0.8] or [0]
            for t in picked:
                n_new = 1 if (rng.random() < 0.8 or r["len"][t] == 0) else 0
                if t == 0 and req in need_sync_token:
                    n_new = 1
                if multi_token and n_new == 1 and rng.random() < 0.35:
                    n_new = int(rng.integers(2, 6))
                entries.append((req, t, n_new))
        order = rng.permutation(len(entries))
        entries = [entries[i] for i in order]
        for e in entries:
            book.add(e[0], e[1], e[2])
            if e[1] == 0 and e[2] >= 1:
                need_sync_token.discard(e[0])
        ops.append(("step", tuple(entries)))

    while len(ops) < n_ops:
        live = sorted(book.live)
        choice = rng.random()
        if not live or (choice < 0.08 and len(live) < max_requests):
            req = book.begin(); ops.append(("begin", req))
            m = int(rng.integers(1, 4 * geo.page_size))
            ops.append(("run", req, 0, m)); book.add(req, 0, m)
            continue
        req = int(rng.choice(live))
        r = book.live[req]
        blocked = paper_flow and req in need_sync_token
        if blocked:
            do_step([req])
        elif choice < 0.25 and r["next"] <= max_forks:
            t = book.spawn(req)
            ops.append(("spawn", req, t, 10 * int(rng.integers(0, 6))) if predictions else ("spawn", req, t))
            if rng.random() < 0.5:
                m = int(rng.integers(1, 3 * geo.page_size))
                ops.append(("run", req, t, m)); book.add(req, t, m)
        elif choice < 0.35 and r["active"]:
            t = int(rng.choice(sorted(r["active"])))
            ops.append(("finish", req, t)); book.finish(req, t)
        elif choice < 0.47 and r["finished"]:
            fin = sorted(r["finished"])
            if rng.random() < 0.5:
                ops.append(("merge", req, None)); book.merge(req, None)
            else:
                pick = tuple(int(t) for t in fin if rng.random() < 0.6) or (fin[0],)
                ops.append(("merge", req, pick)); book.merge(req, pick)
            need_sync_token.add(req)
        elif choice < 0.50 and len(live) > 1:
            ops.append(("end", req)); book.end(req); need_sync_token.discard(req)
        elif choice < 0.56:
            m = int(rng.integers(1, 2 * geo.page_size))
            ops.append(("run", req, 0, m)); book.add(req, 0, m); need_sync_token.discard(req)
        else:
            do_step([q for q in live if rng.random() < 0.7] or [req])
    if not any(op[0] == "step" for op in ops[-3:]):
        do_step(sorted(book.live))
    return _finalise(f"random_{seed}", geo, ops, book, rng, seed, slack_pages=4,
                     max_requests=max_requests, max_threads=max_forks + 1)
