"""Host-side PASTA-LANG interpreter: drives a pool from the token streams of the decoding threads.

What it does (paper, Section 3 "Interpreter" and "Efficiency"; Fig. 2a):
  * decode sequentially until the main thread emits <promise/>; then start a fork whose prefix is everything
    the main thread has produced so far (the promise included) and whose first token is an <async> tag that
    the interpreter inserts; promise and <async> are fed to the model in the same step, so the fork decodes
    its first own token one step after the promise was decoded; the main thread keeps decoding without the
    fork's content;
  * a fork runs until it emits </async>;
  * when the main thread emits <sync/>, that token is held back — it does not enter the KV pool — and the main
    thread pauses until every fork has finished; then the chunks are merged into the main thread's view (no KV
    moves), the held <sync/> enters the pool and the main thread resumes, now conditioned on all chunks.

Tokens enter the pool when they are fed to the model: a step feeds every runnable thread's pending token, the
caller runs the model (pasta_kv_append + pasta_decode_attn inside it) and hands back one next token per fed token.
A prompt can be fed through the same steps, several tokens at a time (`add_request(..., chunk=m)`): the request's
entry then carries up to m tokens, each with its own query, and only what the model says after the prompt's last
token is used.
The interpreter is token-id agnostic: the four tag ids and a function that reads the predicted length out of a
promise are given by the caller.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Tuple


@dataclass(frozen=True)
class Tags:
    promise: int
    async_open: int
    async_close: int
    sync: int


@dataclass
class _Thread:
    pending: Optional[int]           # token to feed at the next step (None: nothing to feed)
    done: bool = False               # a fork that emitted </async>
    tokens: List[int] = field(default_factory=list)   # tokens fed so far (for inspection)
    backlog: List[int] = field(default_factory=list)  # prompt tokens still to feed before `pending` (chunked prefill)
    chunk: int = 1                   # how many backlog tokens one step may feed


@dataclass
class _Request:
    threads: Dict[int, _Thread]
    unmerged: List[int] = field(default_factory=list)  # forks spawned since the last sync
    held_sync: Optional[int] = None  # the <sync/> token while the main thread waits
    finished: bool = False


class Interpreter:
    def __init__(self, pool, tags: Tags, predicted_length: Callable[[int, int], int] = lambda req, promise_index: 0,
                 close_enters_pool: bool = True):
        """pool: a binding.Pool (host-only pools work: the caller then skips the device calls).
        predicted_length(req, k): tokens predicted for the k-th promise of the request (position ids)."""
        self.pool, self.tags = pool, tags
        self.predicted_length = predicted_length
        self.close_enters_pool = close_enters_pool
        self.requests: Dict[int, _Request] = {}
        self._promises: Dict[int, int] = {}
        self._entries: List[Tuple[int, int]] = []

    # ------------------------------------------------------------------ requests
    def add_request(self, prompt: Sequence[int], k=None, v=None, stream=None, chunk: int = 0) -> int:
        """chunk == 0: the prompt's tokens except the last are appended now, with their KV (k, v: device tensors
        [layers, len(prompt) - 1, Hkv, d], or None on a host-only pool); the last prompt token is the first
        pending input.  chunk > 0: nothing is appended now; the prompt is fed through the following steps, up to
        `chunk` tokens per step, like any other token (the model computes their KV and attention)."""
        req = self.pool.request_begin()
        if chunk > 0:
            main = _Thread(pending=prompt[-1], backlog=list(prompt[:-1]), chunk=chunk)
            self.requests[req] = _Request(threads={0: main})
            self._promises[req] = 0
            return req
        if len(prompt) > 1:
            self.pool.kv_append_run(req, 0, len(prompt) - 1, k, v, stream=stream)
        main = _Thread(pending=prompt[-1], tokens=list(prompt[:-1]))
        self.requests[req] = _Request(threads={0: main})
        self._promises[req] = 0
        return req

    def end_request(self, req: int) -> None:
        self.pool.request_end(req)
        del self.requests[req]

    # ------------------------------------------------------------------ one decode step
    def begin_step(self, stream=None) -> List[Tuple[int, int, int]]:
        """Feeds every runnable thread's pending token (or its next chunk of prompt tokens): reserves the slots and
        plans the step.  Returns one (request, thread, token) per fed token, in the order of the step's queries;
        the caller runs the model on them."""
        entries = []
        step_reqs, step_threads, step_new = [], [], []
        for req, r in self.requests.items():
            if r.finished:
                continue
            # order inside a request: forks that have been fed before, the main thread, the fork spawned on the
            # promise the main thread feeds now (its prefix needs that promise appended first)
            runnable = [t for t, th in r.threads.items() if th.pending is not None and not th.done]
            order = sorted(runnable, key=lambda t: (1 if t == 0 else 2 if not r.threads[t].tokens else 0, t))
            for t in order:
                th = r.threads[t]
                if th.backlog:                  # a chunk of the prompt; the pending token joins it when it fits
                    feed = th.backlog[:th.chunk]
                    del th.backlog[:len(feed)]
                    if not th.backlog and len(feed) < th.chunk:
                        feed.append(th.pending); th.pending = None
                else:
                    feed = [th.pending]; th.pending = None
                entries.extend((req, t, tok) for tok in feed)
                th.tokens.extend(feed)
                step_reqs.append(req); step_threads.append(t); step_new.append(len(feed))
        self._entries = [(e[0], e[1]) for e in entries]
        if entries:
            self.pool.step_begin(step_reqs, step_threads, step_new, stream=stream)
        return entries

    def end_step(self, next_tokens: Sequence[int], end_of_text: Optional[int] = None) -> None:
        """next_tokens[i] is what the model produced for entry i of begin_step."""
        assert len(next_tokens) == len(self._entries)
        last_of = {}
        for i, key in enumerate(self._entries):
            last_of[key] = i                      # only what follows a thread's newest token counts
        for i, ((req, t), tok) in enumerate(zip(self._entries, next_tokens)):
            r = self.requests[req]
            th = r.threads[t]
            if last_of[(req, t)] != i or th.backlog or th.pending is not None:
                continue                          # inside a prompt chunk: the model's continuation is not used
            fed = th.tokens[-1]
            if t == 0:
                if end_of_text is not None and tok == end_of_text:
                    r.finished = True
                elif tok == self.tags.sync:
                    r.held_sync = tok            # decoded, but kept out of the pool until the forks are done
                else:
                    th.pending = tok
                    if tok == self.tags.promise:
                        # decoded, not appended yet: the fork's prefix counts it in, and the next step feeds the
                        # promise and the fork's <async> together
                        k = self._promises[req]; self._promises[req] += 1
                        fork = self.pool.thread_spawn_predicted(req, int(self.predicted_length(req, k)), 1)
                        r.threads[fork] = _Thread(pending=self.tags.async_open)
                        r.unmerged.append(fork)
            else:
                if tok == self.tags.async_close:
                    if self.close_enters_pool:
                        th.pending = tok         # the closing tag is fed once more, then the fork is done
                    else:
                        self._finish(req, t)
                elif fed == self.tags.async_close:
                    self._finish(req, t)
                else:
                    th.pending = tok
        for req, r in self.requests.items():
            # a fork whose closing tag has just been fed has nothing pending: finish it
            for t, th in r.threads.items():
                if t != 0 and not th.done and th.pending is None and th.tokens and th.tokens[-1] == self.tags.async_close:
                    self._finish(req, t)
            if r.held_sync is not None and all(r.threads[t].done for t in r.unmerged):
                self.pool.sync_merge(req, r.unmerged)      # zero-copy: only the main thread's segment list changes
                r.unmerged = []
                r.threads[0].pending = r.held_sync         # now the <sync/> token enters the pool
                r.held_sync = None

    def _finish(self, req: int, t: int) -> None:
        th = self.requests[req].threads[t]
        if not th.done:
            self.pool.thread_finish(req, t)
            th.done = True
            th.pending = None

    # ------------------------------------------------------------------ inspection
    def waiting_at_sync(self, req: int) -> bool:
        return self.requests[req].held_sync is not None

    def active_threads(self, req: int) -> List[int]:
        r = self.requests[req]
        return [t for t, th in r.threads.items() if th.pending is not None and not th.done]
