"""Theoretical speedup / parallelism: the closed recurrence of the library against the oracle's timestamp-by-timestamp
timeline, and hand-checked cases."""
import pytest

from oracle import PoolModel, paper_timeline
from paper_2502_11517_b200.interpreter import Tags
from paper_2502_11517_b200.metrics import (count_non_control, sequential_length, theoretical_parallelism,
                                            theoretical_speedup, trace_metrics)
from test_interpreter import random_threads
from test_interpreter_model import CLOSE, OPEN, PROMISE, SYNC, TAGS, fig2_scripts

T = Tags(PROMISE, OPEN, CLOSE, SYNC)


def timeline_length(prompt, emissions):
    """Timestamps until every thread has decoded its last token, read off the oracle's log."""
    _req, log, _ = paper_timeline(PoolModel(256, 16), prompt, emissions, **TAGS)
    return max(Tm for Tm, _t, _tok, _i in log)


def test_plain_text_has_no_parallelism():
    main = [10, 11, 12, 13]
    assert sequential_length(main, {}, T) == 4
    assert theoretical_parallelism(main, {}, T) == 1.0
    assert theoretical_speedup(8, main, {}, T) == 2.0


def test_hand_checked_two_forks():
    # T=1 promise (fork 1 stops at 1 + 4 = 5), T=2 promise (fork 2 stops at 2 + 5 = 7), T=3 sync decoded and withheld,
    # enters at 8, main decodes at 9 and 10 -> 10 timestamps
    ids, prompt, emissions = fig2_scripts()
    forks = {k: v for k, v in emissions.items() if k != 0}
    assert sequential_length(emissions[0], forks, T) == 10 == timeline_length(prompt, emissions)
    # non-control tokens: main 2 (401, 402), fork 1 three, fork 2 four
    assert count_non_control(emissions[0], forks, T) == 9
    assert theoretical_parallelism(emissions[0], forks, T) == pytest.approx(0.9)


def test_long_forks_overlap():
    # one promise, then three forks' worth of text in parallel with 2 main tokens: the forks dominate
    main = [PROMISE, PROMISE, PROMISE, 50, 51, SYNC, 52]
    forks = {1: [60] * 20 + [CLOSE], 2: [60] * 30 + [CLOSE], 3: [60] * 10 + [CLOSE]}
    # fork 2 stops at 2 + 31 = 33; sync enters at 34; token 52 at 35
    assert sequential_length(main, forks, T) == 35
    assert theoretical_parallelism(main, forks, T) == pytest.approx((3 + 60) / 35)


@pytest.mark.parametrize("seed", range(25))
def test_recurrence_equals_timeline(seed):
    prompt, emissions = random_threads(seed)
    forks = {k: v for k, v in emissions.items() if k != 0}
    assert sequential_length(emissions[0], forks, T) == timeline_length(prompt, emissions)


def test_response_that_ends_before_its_forks():
    main = [PROMISE, 7]
    forks = {1: [61, 62, 63, 64, CLOSE]}
    assert sequential_length(main, forks, T) == 6          # the fork's </async> at 1 + 5


def test_trace_metrics_means():
    r = [(40, [10, 11, 12, 13], {}), (35, [PROMISE, PROMISE, PROMISE, 50, 51, SYNC, 52],
                                      {1: [60] * 20 + [CLOSE], 2: [60] * 30 + [CLOSE], 3: [60] * 10 + [CLOSE]})]
    m = trace_metrics(r, T)
    assert m["theoretical_speedup_mean"] == pytest.approx((10.0 + 1.0) / 2)
    assert m["theoretical_speedup_geomean"] == pytest.approx(10.0 ** 0.5)
    assert m["responses"] == 2
