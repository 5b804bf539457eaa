"""The library-side interpreter against the oracle's timeline: same tokens fed per step, same pool state after
every step (pages, views, cut-offs, position ids), on the worked example of Fig. 2 and on random thread scripts.
Step s+1 of the interpreter feeds what the paper's accounting enters at timestamp s."""
import copy

import numpy as np
import pytest

from oracle import PoolModel, paper_timeline
from paper_2502_11517_b200 import binding
from paper_2502_11517_b200.build import build
from paper_2502_11517_b200.interpreter import Interpreter, Tags
from test_interpreter_model import CLOSE, OPEN, PROMISE, SYNC, TAGS, fig2_scripts


@pytest.fixture(scope="module", autouse=True)
def _built():
    build()


class Scripted:
    """A stand-in for the model: thread t's k-th decoded token is emissions[t][k]."""

    def __init__(self, emissions):
        self.emissions, self.count = emissions, {}

    def __call__(self, entries):
        out = []
        for req, t, _tok in entries:
            k = self.count.get((req, t), 0); self.count[(req, t)] = k + 1
            out.append(self.emissions[t][k] if k < len(self.emissions[t]) else -1)
        return out


def oracle_run(prompt, emissions, n_pages, predicted):
    model = PoolModel(n_pages, 16)
    states, fed = {0: None}, {}

    def snap(T, entered):
        states[T] = copy.deepcopy(model.dump()); fed[T] = list(entered)

    req, log, withheld = paper_timeline(model, prompt, emissions, predicted_length=predicted, on_timestamp=snap, **TAGS)
    return states, fed, withheld


def library_run(prompt, emissions, n_pages, predicted, n_steps):
    pool = binding.Pool(1, 4, 2, 64, n_pages, 2, 16, 64, flags=binding.FLAG_HOST_ONLY)
    it = Interpreter(pool, Tags(PROMISE, OPEN, CLOSE, SYNC), predicted_length=lambda req, k: predicted(k))
    req = it.add_request(prompt)
    fake = Scripted(emissions)
    states, fed = {}, {}
    for step in range(1, n_steps + 1):
        entries = it.begin_step()
        fed[step] = [(t, tok) for _r, t, tok in entries]
        states[step] = pool.dump()
        it.end_step(fake(entries))
    pool.close()
    return states, fed


def random_threads(seed):
    rng = np.random.default_rng(seed)
    main, forks = [], {}
    for _ in range(int(rng.integers(1, 4))):                  # promise groups, each closed by a <sync/>
        main += [int(x) for x in rng.integers(100, 200, int(rng.integers(0, 4)))]
        for _p in range(int(rng.integers(1, 4))):
            main.append(PROMISE)
            forks[len(forks) + 1] = [int(x) for x in rng.integers(200, 300, int(rng.integers(0, 9)))] + [CLOSE]
            main += [int(x) for x in rng.integers(100, 200, int(rng.integers(0, 3)))]
        main += [int(x) for x in rng.integers(100, 200, int(rng.integers(0, 12)))] + [SYNC]
    main += [int(x) for x in rng.integers(100, 200, int(rng.integers(1, 4)))]
    prompt = [int(x) for x in rng.integers(300, 400, int(rng.integers(1, 40)))]
    return prompt, {0: main, **forks}


def check(prompt, emissions, predicted):
    o_states, o_fed, withheld = oracle_run(prompt, emissions, 64, predicted)
    T_max = max(o_fed)
    l_states, l_fed = library_run(prompt, emissions, 64, predicted, T_max + 1)
    assert l_fed[1] == [(0, prompt[-1])]
    for T in range(1, T_max + 1):
        assert l_fed[T + 1] == o_fed[T], (T, l_fed[T + 1], o_fed[T])
        want = o_states[T]
        got = l_states[T + 1]
        # thread states differ in one respect only: the library marks a fork finished after its </async> was fed,
        # and merged right away once the waiting <sync/> may go on; the oracle's accounting does both when the
        # tokens enter.  Compare everything else exactly.
        for d in (want, got):
            for r in d["requests"].values():
                for th in r["threads"].values():
                    th.pop("state")
        assert got == want, T
    return withheld


def test_fig2_replay_through_the_library():
    ids, prompt, emissions = fig2_scripts()
    withheld = check(prompt, emissions, lambda k: 10)
    assert withheld == [(3, 8)]


@pytest.mark.parametrize("seed", range(20))
def test_random_thread_scripts(seed):
    prompt, emissions = random_threads(seed)
    check(prompt, emissions, (lambda k: 0) if seed % 2 else (lambda k: 10 * (k % 4)))


def test_sync_waits_and_merge_moves_nothing():
    ids, prompt, emissions = fig2_scripts()
    pool = binding.Pool(1, 4, 2, 64, 64, 2, 16, 64, flags=binding.FLAG_HOST_ONLY)
    it = Interpreter(pool, Tags(PROMISE, OPEN, CLOSE, SYNC))
    req = it.add_request(prompt)
    fake = Scripted(emissions)
    waited = []
    pages_before = None
    for step in range(1, 12):
        entries = it.begin_step()
        if it.waiting_at_sync(req):
            assert all(t != 0 for _r, t, _tok in entries)      # the main thread is not fed while it waits
            pages_before = {s: v["pages"] for s, v in pool.dump()["requests"][req]["streams"].items()}
        it.end_step(fake(entries))
        waited.append(it.waiting_at_sync(req))
    assert waited == [False, False, True, True, True, True, True, False, False, False, False]
    streams = pool.dump()["requests"][req]["streams"]
    for s, pages in pages_before.items():
        assert streams[s]["pages"][:len(pages)] == pages        # chunks stay where they were written
    view = pool.dump()["requests"][req]["threads"][0]["view"]
    assert [seg[0] for seg in view] == [0, 1, 0, 2, 0]          # each chunk right behind its promise
    pool.close()


def test_prompt_fed_in_chunks_ends_in_the_same_state():
    """Feeding the prompt through the steps, 7 tokens at a time, only delays the response: 20 + 1 prompt tokens take
    three steps instead of one, after which every step feeds the same tokens and leaves the same pool state."""
    ids, prompt, emissions = fig2_scripts()

    def run(chunk, n_steps):
        pool = binding.Pool(1, 4, 2, 64, 64, 2, 16, 64, flags=binding.FLAG_HOST_ONLY)
        it = Interpreter(pool, Tags(PROMISE, OPEN, CLOSE, SYNC), predicted_length=lambda req, k: 10)
        it.add_request(prompt, chunk=chunk)
        fake = Scripted(emissions)
        fed, states = [], []
        for _ in range(n_steps):
            entries = it.begin_step()
            fed.append([(t, tok) for _r, t, tok in entries])
            states.append(pool.dump())
            # the scripted stand-in answers per fed token; inside a prompt chunk its answers must be ignored, so it
            # is asked only for the thread's newest token and the other slots get a token that would derail the run
            newest = {}
            for i, (r, t, _tok) in enumerate(entries):
                newest[(r, t)] = i
            in_prompt = bool(it.requests[0].threads[0].backlog or it.requests[0].threads[0].pending is not None)
            answers = [PROMISE] * len(entries)
            real = [e for i, e in enumerate(entries) if newest[(e[0], e[1])] == i and not (e[1] == 0 and in_prompt)]
            for e, tok in zip(real, fake(real)):
                answers[newest[(e[0], e[1])]] = tok
            it.end_step(answers)
        pool.close()
        return fed, states

    fed1, st1 = run(0, 11)
    fed7, st7 = run(7, 13)
    assert [len(f) for f in fed7[:3]] == [7, 7, 7] and [tok for _t, tok in sum(fed7[:3], [])] == prompt
    assert fed7[3:] == fed1[1:]
    assert st7[2:] == st1[:]          # the same states, two steps later (the state after the whole prompt included)


def test_several_responses_decode_side_by_side():
    """Three responses in one pool, stepped together: every response follows its own timeline (same tokens fed at
    the same step, same views, cut-offs and position ids as when it runs alone); only page numbers differ, since
    the responses draw from one free list."""
    scripts = [random_threads(s) for s in (2, 5, 9)]

    def strip(dump_req):
        return {"streams": {s: v["len"] for s, v in dump_req["streams"].items()},
                "threads": {t: {k: v for k, v in th.items() if k != "state"} for t, th in dump_req["threads"].items()}}

    alone = []
    for prompt, emissions in scripts:
        pool = binding.Pool(1, 4, 2, 64, 256, 1, 16, 64, flags=binding.FLAG_HOST_ONLY)
        it = Interpreter(pool, Tags(PROMISE, OPEN, CLOSE, SYNC))
        it.add_request(prompt)
        fake = Scripted(emissions)
        log = []
        for _ in range(60):
            entries = it.begin_step()
            log.append(([(t, tok) for _r, t, tok in entries], strip(pool.dump()["requests"][0])))
            it.end_step(fake(entries))
        alone.append(log)
        pool.close()

    pool = binding.Pool(1, 4, 2, 64, 256, 3, 16, 64, flags=binding.FLAG_HOST_ONLY, max_step_queries=64)
    it = Interpreter(pool, Tags(PROMISE, OPEN, CLOSE, SYNC))
    fakes = {}
    for prompt, emissions in scripts:
        fakes[it.add_request(prompt)] = Scripted(emissions)
    for step in range(60):
        entries = it.begin_step()
        dump = pool.dump()["requests"]
        answers = [None] * len(entries)
        for req in fakes:
            mine = [(i, e) for i, e in enumerate(entries) if e[0] == req]
            assert ([(t, tok) for _i, (_r, t, tok) in mine], strip(dump[req])) == alone[req][step], (req, step)
            for (i, _e), tok in zip(mine, fakes[req]([(0, e[1], e[2]) for _i, e in mine])):
                answers[i] = tok
        it.end_step(answers)
    pool.close()
