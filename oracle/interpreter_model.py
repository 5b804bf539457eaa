"""Oracle, part 5: the interpreter's timeline.  TEST INFRASTRUCTURE — not a product path.

Restates, one decoding timestamp at a time, what the paper's interpreter does with the tokens the threads
decode (Section 3, "Interpreter" and "Efficiency"; the walk through Fig. 2b / 2c), in the paper's own
accounting: a token takes its place in the KV pool at the timestamp T at which it is decoded.

  * every thread that is running decodes one token per timestamp;
  * when the main thread decodes <promise/>, a fork is created at once and receives an <async> token at the
    same timestamp; the fork decodes its first own token at the next timestamp; it sees the main thread's
    tokens up to and including that promise, and its own;
  * a fork stops when it decodes </async> (which is part of its chunk);
  * when the main thread decodes <sync/> while some fork is still running, or has stopped at this very
    timestamp, the token is withheld: it takes no place in the pool and the main thread decodes nothing
    further; at the first timestamp after every fork has stopped, the chunks are merged, the <sync/> takes
    its place, and the main thread decodes again from the timestamp after that.

Reading taken where the text is silent: a <sync/> decoded when every fork stopped at an earlier timestamp is
not withheld at all; the timestamp at which the withheld <sync/> enters is the one right after the last
</async> (the closing tag has to be in the pool for the main thread to condition on the whole chunk).

What each thread decodes is given (a script per thread), since no model runs here.
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional, Sequence, Tuple

from .pool_model import PoolModel


def paper_timeline(model: PoolModel, prompt: Sequence[int], emissions: Dict[int, Sequence[int]],
                   promise: int, async_open: int, async_close: int, sync: int,
                   predicted_length: Callable[[int], int] = lambda k: 0,
                   on_timestamp: Optional[Callable[[int, List[Tuple[int, int]]], None]] = None):
    """Runs one request to the end of the main thread's script on `model`.

    emissions[0] = what the main thread decodes, in order; emissions[k] = what the fork of the k-th promise
    decodes (ending with async_close).  Returns (req, log, withheld): log = [(T, thread, token, i)] for every
    token that entered the pool, i = its index in one token-granular pool filled in order of entry (the
    prompt takes 0..len-1 at T=0); withheld = [(T_decoded, T_entered)] for every <sync/> that had to wait.
    `on_timestamp(T, entered)` is called after the tokens [(thread, token)] of timestamp T are in the pool.
    """
    req = model.request_begin()
    model.append_run(req, 0, len(prompt))
    log = [(0, 0, tok, i) for i, tok in enumerate(prompt)]
    nxt = {0: 0}                       # thread -> index of its next scripted token
    stopped_at: Dict[int, int] = {}    # fork -> timestamp of its </async>
    unmerged: List[int] = []
    held: Optional[int] = None         # timestamp at which the waiting <sync/> was decoded
    withheld = []
    promises = 0
    T = 0
    main_script = emissions[0]
    while nxt[0] < len(main_script) or held is not None:
        T += 1
        entered: List[Tuple[int, int]] = []
        running = [t for t in sorted(nxt) if t != 0 and t not in stopped_at]
        for t in running:                                  # forks created before this timestamp
            tok = emissions[t][nxt[t]]; nxt[t] += 1
            model.reserve([(req, t, 1)])
            entered.append((t, tok))
            if tok == async_close:
                stopped_at[t] = T
                model.thread_finish(req, t)
        if held is not None:
            if all(stopped_at.get(t, T) < T for t in unmerged):
                model.sync_merge(req, unmerged)
                unmerged = []
                model.reserve([(req, 0, 1)])
                entered.append((0, sync))
                withheld.append((held, T))
                held = None
        else:
            tok = main_script[nxt[0]]; nxt[0] += 1
            if tok == sync and any(stopped_at.get(t, T) >= T for t in unmerged):
                held = T
            else:
                if tok == sync:
                    model.sync_merge(req, unmerged)
                    unmerged = []
                model.reserve([(req, 0, 1)])
                entered.append((0, tok))
                if tok == promise:
                    promises += 1
                    fork = model.thread_spawn(req, predicted_length(promises - 1))
                    assert fork == promises
                    nxt[fork] = 0
                    unmerged.append(fork)
                    model.reserve([(req, fork, 1)])
                    entered.append((fork, async_open))
        for t, tok in entered:
            log.append((T, t, tok, len(log)))
        if on_timestamp is not None:
            on_timestamp(T, entered)
    return req, log, withheld
