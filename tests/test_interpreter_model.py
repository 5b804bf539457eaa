"""Pins of the oracle's interpreter timeline: the worked example of the paper's Section 3 "Efficiency" (Fig. 2b/2c),
timestamp by timestamp and index by index, the visibility facts of the same passage, and what follows the <sync/>."""
import os

import pytest

from oracle import PoolModel
from oracle.interpreter_model import paper_timeline

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
PROMISE, OPEN, CLOSE, SYNC = 1, 2, 3, 4
TAGS = dict(promise=PROMISE, async_open=OPEN, async_close=CLOSE, sync=SYNC)


def read_fig2():
    tokens, withheld, facts = [], [], []
    with open(os.path.join(GOLDEN, "fig2_worked_example.txt")) as f:
        for line in f:
            w = line.split("#")[0].split()
            if not w:
                continue
            if w[0] == "token":
                tokens.append((w[1], w[2], int(w[3]), int(w[4])))
            elif w[0] == "withheld":
                withheld.append((w[1], w[2], int(w[3])))
            else:
                facts.append((w[0], w[1], w[2]))
    return tokens, withheld, facts


def fig2_scripts():
    """Token ids for the labels of the figure, and what each thread decodes (the figure stops at T=3; the
    rest of the chunks and of the main thread is made up so that the <sync/> has something to wait for)."""
    ids = {"query19": 119, "segment?": 120, "promise1": PROMISE, "promise2": PROMISE, "async1": OPEN, "async2": OPEN,
           "To": 201, "find": 202, "fork2tok": 301, "sync": SYNC}
    prompt = list(range(100, 121))
    emissions = {0: [PROMISE, PROMISE, SYNC, 401, 402],
                 1: [201, 202, 203, CLOSE],                  # stops at T=5
                 2: [301, 302, 303, 304, CLOSE]}             # first own token at T=3, stops at T=7
    return ids, prompt, emissions


def test_fig2_timeline_indices_and_withheld_sync():
    tokens, withheld_golden, facts = read_fig2()
    ids, prompt, emissions = fig2_scripts()
    thread_id = {"main": 0, "fork1": 1, "fork2": 2}
    model = PoolModel(64, 4)
    seen_at = {}

    def snapshot(T, entered):
        seen_at[T] = {t: set(model.visible_slots(0, t)) for t in model.requests[0].state}

    req, log, withheld = paper_timeline(model, prompt, emissions, predicted_length=lambda k: 10, on_timestamp=snapshot,
                                        **TAGS)
    by_index = {i: (T, t, tok) for T, t, tok, i in log}
    for label, thread, T, i in tokens:
        assert by_index[i] == (T, thread_id[thread], ids[label]), (label, by_index[i])
    # the <sync/> is decoded at T=3, takes no index then (the figure's next free index stays 28) ...
    assert [x for x in log if x[0] <= 3][-1][3] == 27
    (label, thread, T), = withheld_golden
    assert withheld == [(T, 8)]                      # ... and enters right after the last </async> (T=7)
    assert [(T_, t) for T_, t, tok, _ in log if tok == SYNC] == [(8, 0)]
    # the main thread decodes nothing between T=3 and the <sync/>
    assert [T_ for T_, t, tok, _ in log if t == 0 and T_ > 0] == [1, 2, 8, 9, 10]

    # visibility facts of the text, at T=3
    P = model.page_size
    where = {}                                       # label -> (page, offset)
    count = {0: 19, 1: 0, 2: 0}
    for label, thread, T, i in tokens:
        t = thread_id[thread]
        pages = model.requests[0].stream_pages[t]
        where[label] = (pages[count[t] // P], count[t] % P); count[t] += 1
    owner = {label: thread_id[thread] for label, thread, _T, _i in tokens}
    for verdict, who, what in facts:
        if what == "sync":
            assert verdict == "cannot"
            continue
        assert (where[what] in seen_at[3][owner[who]]) == (verdict == "can"), (verdict, who, what)


def test_after_sync_the_main_thread_reads_each_chunk_behind_its_promise():
    ids, prompt, emissions = fig2_scripts()
    model = PoolModel(64, 4)
    req, log, _ = paper_timeline(model, prompt, emissions, **TAGS)
    tok_at = {}
    count = {}
    for T, t, tok, i in log:
        k = count.get(t, 0); count[t] = k + 1
        pages = model.requests[req].stream_pages[t]
        tok_at[(pages[k // 4], k % 4)] = tok
    order = [tok_at[s] for s in model.visible_slots(req, 0)]
    assert order == (prompt + [PROMISE] + [OPEN, 201, 202, 203, CLOSE] + [PROMISE] + [OPEN, 301, 302, 303, 304, CLOSE]
                     + [SYNC, 401, 402])
    # nothing moved: every token is where it was first written (one slot per log entry, all distinct)
    assert len(tok_at) == len(log)


def test_sync_is_not_withheld_when_every_fork_stopped_earlier():
    model = PoolModel(64, 4)
    emissions = {0: [PROMISE, 11, 12, 13, 14, SYNC, 15], 1: [21, CLOSE]}
    req, log, withheld = paper_timeline(model, [7, 8, 9], emissions, **TAGS)
    assert withheld == []
    assert [(T, tok) for T, t, tok, _ in log if t == 0 and T > 0] == [(1, PROMISE), (2, 11), (3, 12), (4, 13), (5, 14),
                                                                      (6, SYNC), (7, 15)]
    # a fork that stops at the very timestamp of the <sync/> delays it by one
    model = PoolModel(64, 4)
    emissions = {0: [PROMISE, 11, SYNC, 15], 1: [21, CLOSE]}      # </async> at T=3, <sync/> decoded at T=3
    req, log, withheld = paper_timeline(model, [7, 8, 9], emissions, **TAGS)
    assert withheld == [(3, 4)]


def test_sequential_text_is_plain_decoding():
    model = PoolModel(64, 4)
    req, log, withheld = paper_timeline(model, [5, 6], {0: [10, 11, 12]}, **TAGS)
    assert [(T, t, tok) for T, t, tok, _ in log] == [(0, 0, 5), (0, 0, 6), (1, 0, 10), (2, 0, 11), (3, 0, 12)]
    assert model.view(req, 0) == [(0, 0, 5)]


def test_position_ids_skip_the_predicted_block():
    # Section 6 "Positional Embedding": the fork's tokens continue after the promise, the main thread jumps ahead
    model = PoolModel(64, 4)
    pos = {}

    def record(T, entered):
        for t, tok in entered:
            pos[(t, tok)] = model.last_position(0, t)

    paper_timeline(model, [7, 8, 9], {0: [PROMISE, 11, 12, SYNC, 13], 1: [21, 22, CLOSE]},
                   predicted_length=lambda k: 20, on_timestamp=record, **TAGS)
    assert pos[(0, PROMISE)] == 3
    assert (pos[(1, OPEN)], pos[(1, 21)], pos[(1, 22)], pos[(1, CLOSE)]) == (4, 5, 6, 7)
    assert (pos[(0, 11)], pos[(0, 12)], pos[(0, SYNC)], pos[(0, 13)]) == (24, 25, 26, 27)
