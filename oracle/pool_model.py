"""Oracle, part 1: the KV pool's bookkeeping (integers only).  TEST INFRASTRUCTURE — not a product path.

Only the test-suite, the smoke check and the CPU-baseline leg of the benchmark may import this
package.  It shares no code with the CUDA library; the two are written independently from the
same rules, and their states are compared with `==`.

What the paper fixes (Section 3, "Efficiency"; Fig. 2b/2c; Appendix B):
  * all threads of a response append their KV into one pool while they decode in the same step;
  * a token of an asynchronous thread may attend to the tokens of its own thread and to the
    main-thread tokens that existed before the thread was spawned; threads never see each other
    before synchronisation; the main thread does not condition on asynchronous content until
    <sync/>;
  * after <sync/> the main thread conditions on every chunk, each placed (logically) right
    after its own <promise/>; nothing is copied.

What the paper leaves open, and the reading taken here:
  * storage is paged (page_size tokens per page); a stream (the main thread's tokens, or one
    fork's chunk) receives a new page exactly when it appends token index k with
    k % page_size == 0; pages are handed out from the front of a free sequence that starts as
    `free_order`; ending a request returns its pages stream by stream (ascending stream id),
    page by page, each to the FRONT of the free sequence;
  * a fork's view is a snapshot of the main thread's view taken when it is spawned (so it
    includes chunks merged by earlier syncs, never chunks merged later) followed by its own chunk;
  * a view is a list of (stream, start, length) with empty entries dropped and touching entries
    of one stream coalesced; a merged chunk with cut-off p goes immediately after the
    main-stream piece ending at p (splitting a piece if p is inside one), after chunks already
    placed at the same p with a smaller thread id and before those with a larger one;
  * only the main thread spawns; merging an unfinished fork is an error (the interpreter waits);
  * a thread may feed several tokens in one step (a chunk of the prompt; Section 3 "Efficiency" has the promise and
    the <async> tag enter at one timestamp): every new token then issues its own query, which sees the thread's
    view up to and including that token and none of the later ones, exactly as if the tokens had been fed in
    successive steps.

Position ids (Section 4, "Training a PASTA-SFT model", and Section 6 "Positional Embedding"): the main thread
cannot know how long an asynchronous block will be, so it skips ahead by the length PREDICTED in the promise:
a fork's first token takes the position right after its <promise/>, the main thread's next token takes that
position plus the predicted length.  Positions are never revised: if a chunk turns out longer than predicted,
its ids run into the ids the main thread used after the promise (not monotone after sync); if shorter, a gap
stays.  How the prediction is made (fixed 40, exact, multiples of ten, ground truth) is the caller's business.

Spawning on a decoded promise (Section 3 "Efficiency", the walk through Fig. 2b: the <async> tag joins the pool at
the timestamp of its <promise/>, and the fork decodes its first own token at the next one): a fork may be spawned
while the promise is decoded but its KV is not in the pool yet (`pending=1`).  The fork's view then counts the
main thread's NEXT token in; the result is the same as appending that token first and spawning afterwards, and
the fork may take part in a step only if the main thread's token is in the pool by the end of that step's appends.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

OK, INVALID_ARG, OUT_OF_PAGES, BAD_STATE, CAPACITY = 0, 1, 2, 3, 4
ACTIVE, FINISHED, MERGED = 0, 1, 2


class PoolError(Exception):
    def __init__(self, code: int, what: str = ""):
        super().__init__(f"pool error {code}: {what}")
        self.code = code


class _Request:
    def __init__(self):
        self.stream_len: Dict[int, int] = {0: 0}          # stream id -> tokens
        self.stream_pages: Dict[int, List[int]] = {0: []}  # stream id -> page ids
        self.state: Dict[int, int] = {0: ACTIVE}           # thread id -> ACTIVE / FINISHED / MERGED
        self.cutoff: Dict[int, int] = {0: 0}               # thread id -> main-stream length at spawn
        # a view is a list of [stream, start, length, anchor]; anchor = cut-off of a merged chunk, -1 for main pieces
        self.view: Dict[int, List[List[int]]] = {0: []}
        self.next_thread = 1
        self.pos_next: Dict[int, int] = {0: 0}             # thread id -> position id of the thread's next token
        self.pos_skip = 0                                  # positions the main thread skips after its next token
        self.pos_last: Dict[int, int] = {0: -1}            # thread id -> position id of the thread's newest own token


class PoolModel:
    def __init__(self, n_pages: int, page_size: int, free_order: Optional[Sequence[int]] = None,
                 max_requests: int = 1 << 30, max_threads_per_request: int = 1 << 30,
                 max_segments_per_thread: int = 1 << 30):
        self.page_size = page_size
        self.free: List[int] = list(range(n_pages)) if free_order is None else [int(p) for p in free_order]
        assert sorted(self.free) == list(range(n_pages)), "free_order must be a permutation"
        self.requests: Dict[int, _Request] = {}
        self.max_requests = max_requests
        self.max_threads = max_threads_per_request
        self.max_segments = max_segments_per_thread

    # ------------------------------------------------------------------ lifecycle
    def request_begin(self) -> int:
        req = 0
        while req in self.requests:
            req += 1
        if req >= self.max_requests:
            raise PoolError(CAPACITY, "too many requests")
        self.requests[req] = _Request()
        return req

    def request_end(self, req: int) -> None:
        r = self._req(req)
        for stream in sorted(r.stream_pages):
            for page in r.stream_pages[stream]:
                self.free.insert(0, page)
        del self.requests[req]

    def thread_spawn(self, req: int, predicted_tokens: int = 0, pending: int = 0) -> int:
        """<promise/>: the new fork sees what the main thread sees right now, and nothing later.  Its first token
        takes the position after the promise; the main thread skips `predicted_tokens` positions.
        pending=1: the promise is the main thread's next token, not appended yet; it counts as seen."""
        r = self._req(req)
        if predicted_tokens < 0 or pending not in (0, 1):
            raise PoolError(INVALID_ARG, "negative predicted length")
        t = r.next_thread
        if t >= self.max_threads:
            raise PoolError(CAPACITY, "too many threads")
        if pending:
            if not self._can_grow(r, 0):
                raise PoolError(CAPACITY, "too many segments")
            k = r.stream_len[0]
            snapshot = [list(e) for e in r.view[0]]
            if snapshot and snapshot[-1][0] == 0 and snapshot[-1][1] + snapshot[-1][2] == k:
                snapshot[-1][2] += 1
            else:
                snapshot.append([0, k, 1, -1])
            r.next_thread += 1
            r.stream_len[t] = 0
            r.stream_pages[t] = []
            r.state[t] = ACTIVE
            r.cutoff[t] = k + 1
            r.view[t] = snapshot
            r.pos_last[t] = -1
            r.pos_next[t] = r.pos_next[0] + 1       # right after the promise, which takes pos_next[0]
            r.pos_skip += predicted_tokens          # the main thread jumps once the promise is in
            return t
        r.next_thread += 1
        r.stream_len[t] = 0
        r.stream_pages[t] = []
        r.state[t] = ACTIVE
        r.cutoff[t] = r.stream_len[0]
        r.view[t] = [list(e) for e in r.view[0]]
        r.pos_last[t] = -1
        r.pos_next[t] = r.pos_next[0]
        r.pos_next[0] += predicted_tokens
        return t

    def thread_finish(self, req: int, thread: int) -> None:
        r = self._req(req)
        if thread == 0 or thread not in r.state:
            raise PoolError(INVALID_ARG, "no such fork")
        if r.state[thread] != ACTIVE:
            raise PoolError(BAD_STATE, "fork is not active")
        r.state[thread] = FINISHED

    # ------------------------------------------------------------------ appending
    def reserve(self, entries: Sequence[Tuple[int, int, int]]) -> List[Optional[Tuple[int, int]]]:
        """One step: entries (req, thread, n_new) in order; returns one element per QUERY: the (page, offset) slot
        of each appended token, or None for the single query of an attention-only entry.  All-or-nothing."""
        seen = set()
        need = 0
        for req, thread, n_new in entries:
            r = self._req(req)
            if thread not in r.state or (req, thread) in seen or n_new < 0:
                raise PoolError(INVALID_ARG, "bad step entry")
            if r.state[thread] != ACTIVE:
                raise PoolError(INVALID_ARG, "thread is not active")
            seen.add((req, thread))
            n = r.stream_len[thread]
            need += -(-(n + n_new) // self.page_size) - -(-n // self.page_size)
            if not n_new and not r.view[thread]:
                raise PoolError(INVALID_ARG, "query with nothing visible")
            if n_new and not self._can_grow(r, thread):
                raise PoolError(CAPACITY, "too many segments")
        main_grows = {req: n_new for req, thread, n_new in entries if thread == 0 and n_new}
        for req, thread, n_new in entries:
            r = self.requests[req]
            main_len = r.stream_len[0] + main_grows.get(req, 0)
            if thread != 0 and r.cutoff[thread] > main_len:
                raise PoolError(BAD_STATE, "the fork's promise is not in the pool")
        if need > len(self.free):
            raise PoolError(OUT_OF_PAGES, "pool exhausted")
        out: List[Optional[Tuple[int, int]]] = []
        self.step_positions: List[int] = []          # position id of each query's token
        for req, thread, n_new in entries:
            if n_new == 0:
                out.append(None)
                self.step_positions.append(self.last_position(req, thread))
            for _ in range(n_new):
                out.append(self._append_one(req, thread))
                self.step_positions.append(self.last_position(req, thread))
        return out

    @staticmethod
    def queries_of(entries: Sequence[Tuple[int, int, int]]) -> List[Tuple[int, int, int]]:
        """(req, thread, hide) per query of a step: `hide` = how many of the thread's newest tokens the query does
        not see (the tokens of the same step that come after its own)."""
        out = []
        for req, thread, n_new in entries:
            out.extend((req, thread, max(1, n_new) - 1 - j) for j in range(max(1, n_new)))
        return out

    def append_run(self, req: int, thread: int, m: int) -> List[Tuple[int, int]]:
        r = self._req(req)
        if thread not in r.state or m < 0:
            raise PoolError(INVALID_ARG, "bad run")
        if r.state[thread] != ACTIVE:
            raise PoolError(INVALID_ARG, "thread is not active")
        if thread != 0 and r.cutoff[thread] > r.stream_len[0]:
            raise PoolError(BAD_STATE, "the fork's promise is not in the pool")
        n = r.stream_len[thread]
        need = -(-(n + m) // self.page_size) - -(-n // self.page_size)
        if need > len(self.free):
            raise PoolError(OUT_OF_PAGES, "pool exhausted")
        if m and not self._can_grow(r, thread):
            raise PoolError(CAPACITY, "too many segments")
        return [self._append_one(req, thread) for _ in range(m)]

    def _can_grow(self, r: _Request, thread: int) -> bool:
        view = r.view[thread]
        stream = thread
        extends = bool(view) and view[-1][0] == stream and view[-1][1] + view[-1][2] == r.stream_len[stream]
        return extends or len(view) < self.max_segments

    def _append_one(self, req: int, thread: int) -> Tuple[int, int]:
        r = self.requests[req]
        stream = thread
        k = r.stream_len[stream]
        if k % self.page_size == 0:
            r.stream_pages[stream].append(self.free.pop(0))
        slot = (r.stream_pages[stream][k // self.page_size], k % self.page_size)
        r.stream_len[stream] = k + 1
        r.pos_last[thread] = r.pos_next[thread]
        r.pos_next[thread] += 1
        if thread == 0:
            r.pos_next[0] += r.pos_skip
            r.pos_skip = 0
        view = r.view[thread]
        if view and view[-1][0] == stream and view[-1][1] + view[-1][2] == k:
            view[-1][2] += 1
        else:
            view.append([stream, k, 1, -1])
        return slot

    # ------------------------------------------------------------------ <sync/>
    def sync_merge(self, req: int, threads: Optional[Sequence[int]] = None) -> None:
        r = self._req(req)
        if threads is None:
            threads = [t for t in sorted(r.state) if t != 0 and r.state[t] == FINISHED]
        threads = list(threads)
        if len(set(threads)) != len(threads):
            raise PoolError(INVALID_ARG, "thread named twice")
        for t in threads:
            if t == 0 or t not in r.state or r.state[t] == MERGED:
                raise PoolError(INVALID_ARG, "no such unmerged fork")
        for t in threads:
            if r.state[t] != FINISHED:
                raise PoolError(BAD_STATE, "fork still decoding")
        for t in threads:
            if r.cutoff[t] > r.stream_len[0]:
                raise PoolError(BAD_STATE, "the fork's promise is not in the pool")
        view = [list(e) for e in r.view[0]]
        for t in sorted(threads):
            n = r.stream_len[t]
            if n == 0:
                continue
            p = r.cutoff[t]
            # split the main-stream piece that contains position p strictly inside
            for i, (s, a, ln, _) in enumerate(view):
                if s == 0 and a < p < a + ln:
                    view[i:i + 1] = [[0, a, p - a, -1], [0, p, a + ln - p, -1]]
                    break
            # first entry that must stay behind the new chunk
            at = len(view)
            for i, (s, a, ln, anchor) in enumerate(view):
                if (s == 0 and a >= p) or (s != 0 and (anchor > p or (anchor == p and s > t))):
                    at = i
                    break
            view.insert(at, [t, 0, n, p])
        if len(view) > self.max_segments:
            raise PoolError(CAPACITY, "too many segments")
        r.view[0] = view
        for t in threads:
            r.state[t] = MERGED

    # ------------------------------------------------------------------ queries
    def view(self, req: int, thread: int) -> List[Tuple[int, int, int]]:
        """The thread's visible tokens as (stream, start, length) pieces in logical order."""
        r = self._req(req)
        return [(s, a, n) for s, a, n, _ in r.view[thread]]

    def visible_slots(self, req: int, thread: int, hide: int = 0) -> List[Tuple[int, int]]:
        """(page, offset) of every visible token, in logical order; `hide` newest tokens of the thread's own stream
        left out (a query for an earlier one of several tokens fed in one step)."""
        r = self._req(req)
        own_end = r.stream_len[thread] - hide
        out = []
        for s, a, n, _ in r.view[thread]:
            pages = r.stream_pages[s]
            end = min(a + n, own_end) if s == thread else a + n
            out.extend((pages[k // self.page_size], k % self.page_size) for k in range(a, end))
        return out

    def last_position(self, req: int, thread: int) -> int:
        """Position id of the thread's newest token (the one a decode step's query belongs to)."""
        r = self._req(req)
        if r.pos_last[thread] >= 0:
            return r.pos_last[thread]
        return r.pos_next[thread] - 1       # a fork without own tokens: the promise (or the token before it)

    def dump(self) -> dict:
        """Whole bookkeeping state in a canonical form."""
        reqs = {}
        for req in sorted(self.requests):
            r = self.requests[req]
            reqs[req] = {
                "streams": {s: {"len": r.stream_len[s], "pages": list(r.stream_pages[s])} for s in sorted(r.stream_len)},
                "threads": {t: {"state": r.state[t], "cutoff": r.cutoff[t], "pos_next": r.pos_next[t],
                                "view": [(s, a, n) for s, a, n, _ in r.view[t]]} for t in sorted(r.state)},
            }
        return {"requests": reqs, "free": list(self.free)}

    def _req(self, req: int) -> _Request:
        if req not in self.requests:
            raise PoolError(INVALID_ARG, "no such request")
        return self.requests[req]
