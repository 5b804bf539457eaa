"""Theoretical speedup and parallelism of an annotated response (paper, Section 4 "Training a PASTA-SFT model", the
scoring of sampled responses, and Section 5, the list of evaluation metrics).

Both divide by the length of the longest sequence that must be decoded sequentially: the number of decoding
timestamps the interpreter needs for the response when every running thread decodes one token per timestamp.
    theoretical speedup     = tokens of the baseline's (sequential) response / that length
    theoretical parallelism = non-control tokens of the response            / that length
The length follows from the threads' token streams alone, by a recurrence over the main thread's tokens:
  * the main thread decodes one token per timestamp;
  * a fork created by a <promise/> decoded at timestamp t decodes its j-th own token at t + j (the <async> tag is
    inserted by the interpreter at t and costs no timestamp) and stops with its </async>;
  * a <sync/> decoded at timestamp t goes on at once if every fork stopped before t; otherwise it enters the pool at
    the timestamp after the last </async> and the main thread decodes again one timestamp later.
"""
from __future__ import annotations

from typing import Dict, Sequence, Tuple

from .interpreter import Tags


def sequential_length(main: Sequence[int], forks: Dict[int, Sequence[int]], tags: Tags) -> int:
    """main: the tokens the main thread decodes, in order (tags included); forks[k]: the tokens the fork of the
    k-th promise decodes (k = 1, 2, …; its </async> included, the inserted <async> not).  Returns the number of
    decoding timestamps until every thread has decoded its last token."""
    t = 0                     # timestamp of the main thread's latest token
    promises = 0
    open_forks_end = []       # stop timestamps of the forks spawned since the last <sync/>
    last = 0
    for tok in main:
        t += 1
        if tok == tags.promise:
            promises += 1
            end = t + len(forks[promises])
            open_forks_end.append(end)
            last = max(last, end)
        elif tok == tags.sync:
            latest = max(open_forks_end, default=0)
            if latest >= t:
                t = latest + 1            # the withheld <sync/> enters here; the next token comes one timestamp later
            open_forks_end = []
        last = max(last, t)
    return last


def count_non_control(main: Sequence[int], forks: Dict[int, Sequence[int]], tags: Tags) -> int:
    control = {tags.promise, tags.async_open, tags.async_close, tags.sync}
    return sum(tok not in control for tok in main) + sum(tok not in control for f in forks.values() for tok in f)


def theoretical_speedup(baseline_tokens: int, main: Sequence[int], forks: Dict[int, Sequence[int]], tags: Tags) -> float:
    return baseline_tokens / sequential_length(main, forks, tags)


def theoretical_parallelism(main: Sequence[int], forks: Dict[int, Sequence[int]], tags: Tags) -> float:
    return count_non_control(main, forks, tags) / sequential_length(main, forks, tags)


def trace_metrics(responses: Sequence[Tuple[int, Sequence[int], Dict[int, Sequence[int]]]], tags: Tags) -> dict:
    """responses: (baseline_tokens, main, forks) per prompt.  Returns the means the paper reports, plus the geometric
    mean of the speedups (a ratio metric)."""
    import math
    sp = [theoretical_speedup(b, m, f, tags) for b, m, f in responses]
    pa = [theoretical_parallelism(m, f, tags) for _b, m, f in responses]
    n = max(1, len(sp))
    return {"theoretical_speedup_mean": sum(sp) / n,
            "theoretical_speedup_geomean": math.exp(sum(math.log(x) for x in sp) / n) if sp else 0.0,
            "theoretical_parallelism_mean": sum(pa) / n, "responses": len(sp)}
