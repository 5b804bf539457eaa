"""Integer rules of the oracle's pool model: paging, free-list order, canonical views, errors.

Expected values here are written out by hand from the stated rules (a page on every append whose
index is a multiple of the page size; pages taken from the front of the free sequence; a merged
chunk right after the main-stream piece that ends at its cut-off, ties by thread id)."""
import numpy as np
import pytest

from oracle import (BAD_STATE, CAPACITY, INVALID_ARG, OUT_OF_PAGES, PoolError, PoolModel)


def test_page_is_taken_exactly_when_needed():
    m = PoolModel(8, 16, [5, 2, 7, 0, 1, 3, 4, 6])
    r = m.request_begin()
    slots = m.append_run(r, 0, 32)
    assert slots[0] == (5, 0) and slots[15] == (5, 15) and slots[16] == (2, 0) and slots[31] == (2, 15)
    assert m.free == [7, 0, 1, 3, 4, 6]                     # 32 tokens = exactly two pages, no third yet
    assert m.reserve([(r, 0, 1)]) == [(7, 0)]               # token 33 takes the third
    t = m.thread_spawn(r)
    assert m.free == [0, 1, 3, 4, 6]                        # spawning takes nothing
    assert m.reserve([(r, t, 1), (r, 0, 1)]) == [(0, 0), (7, 1)]


def test_step_serves_threads_in_list_order():
    m = PoolModel(6, 4, [3, 1, 4, 0, 5, 2])
    r = m.request_begin()
    m.append_run(r, 0, 4)                                   # page 3 full
    a, b = m.thread_spawn(r), m.thread_spawn(r)
    assert m.reserve([(r, b, 1), (r, 0, 1), (r, a, 1)]) == [(1, 0), (4, 0), (0, 0)]


def test_request_end_returns_pages_to_the_front():
    m = PoolModel(8, 4, list(range(8)))
    r = m.request_begin()
    m.append_run(r, 0, 6)            # pages 0, 1
    t = m.thread_spawn(r)
    m.append_run(r, t, 9)            # pages 2, 3, 4
    m.request_end(r)
    # stream 0 first (0 then 1 pushed to the front), then stream 1 (2, 3, 4)
    assert m.free == [4, 3, 2, 1, 0, 5, 6, 7]
    assert m.request_begin() == 0    # lowest unused id again


def test_canonical_view_after_merges():
    m = PoolModel(64, 4)
    r = m.request_begin()
    m.append_run(r, 0, 10)
    a = m.thread_spawn(r)            # cut-off 10
    m.append_run(r, 0, 5)
    b = m.thread_spawn(r)            # cut-off 15
    c = m.thread_spawn(r)            # cut-off 15 as well
    m.append_run(r, 0, 2)            # main stream 17
    for t, n in ((a, 3), (b, 4), (c, 0)):
        m.append_run(r, t, n); m.thread_finish(r, t)
    m.sync_merge(r, [c, b])          # partial merge; c is empty and leaves no entry
    assert m.view(r, 0) == [(0, 0, 15), (b, 0, 4), (0, 15, 2)]
    d = m.thread_spawn(r)            # cut-off 17, sees chunk b
    m.append_run(r, d, 1)
    assert m.view(r, d) == [(0, 0, 15), (b, 0, 4), (0, 15, 2), (d, 0, 1)]
    m.sync_merge(r)                  # merges a: splits the first piece at 10
    assert m.view(r, 0) == [(0, 0, 10), (a, 0, 3), (0, 10, 5), (b, 0, 4), (0, 15, 2)]
    assert m.view(r, d) == [(0, 0, 15), (b, 0, 4), (0, 15, 2), (d, 0, 1)]     # a frozen snapshot
    m.append_run(r, 0, 1)
    assert m.view(r, 0)[-1] == (0, 15, 3)
    m.thread_finish(r, d); m.sync_merge(r, [d])
    assert m.view(r, 0) == [(0, 0, 10), (a, 0, 3), (0, 10, 5), (b, 0, 4), (0, 15, 2), (d, 0, 1), (0, 17, 1)]


def test_same_cutoff_orders_by_thread_id_whatever_the_merge_order():
    m = PoolModel(64, 4)
    r = m.request_begin(); m.append_run(r, 0, 3)
    forks = [m.thread_spawn(r) for _ in range(3)]
    for t in forks:
        m.append_run(r, t, 2); m.thread_finish(r, t)
    m.sync_merge(r, [forks[2]]); m.sync_merge(r, [forks[0]]); m.sync_merge(r, [forks[1]])
    assert m.view(r, 0) == [(0, 0, 3), (1, 0, 2), (2, 0, 2), (3, 0, 2)]
    m.append_run(r, 0, 1)
    assert m.view(r, 0)[-1] == (0, 3, 1)


def test_spawn_at_position_zero():
    m = PoolModel(16, 4)
    r = m.request_begin()
    t = m.thread_spawn(r)
    with pytest.raises(PoolError) as e:
        m.reserve([(r, t, 0)])                   # nothing visible
    assert e.value.code == INVALID_ARG
    m.append_run(r, t, 2); m.append_run(r, 0, 3); m.thread_finish(r, t); m.sync_merge(r)
    assert m.view(r, 0) == [(t, 0, 2), (0, 0, 3)]


def test_errors_leave_the_pool_unchanged():
    m = PoolModel(2, 4)
    r = m.request_begin()
    m.append_run(r, 0, 4)
    t = m.thread_spawn(r)
    before = m.dump()
    with pytest.raises(PoolError) as e:
        m.append_run(r, 0, 5)                    # needs two pages, one left
    assert e.value.code == OUT_OF_PAGES and m.dump() == before
    with pytest.raises(PoolError) as e:
        m.reserve([(r, 0, 1), (r, t, 1)])        # two pages needed in one step
    assert e.value.code == OUT_OF_PAGES and m.dump() == before
    with pytest.raises(PoolError) as e:
        m.sync_merge(r, [t])                     # still decoding: the interpreter has to wait
    assert e.value.code == BAD_STATE and m.dump() == before
    for bad in ([(r, 0, 1), (r, 0, 1)], [(r, 9, 1)], [(7, 0, 1)], [(r, 0, -1)]):
        with pytest.raises(PoolError) as e:
            m.reserve(bad)
        assert e.value.code == INVALID_ARG and m.dump() == before
    m.thread_finish(r, t)
    with pytest.raises(PoolError) as e:
        m.reserve([(r, t, 1)])                   # a finished fork decodes no more
    assert e.value.code == INVALID_ARG
    with pytest.raises(PoolError) as e:
        m.thread_finish(r, t)
    assert e.value.code == BAD_STATE
    m.sync_merge(r, [t]); m.sync_merge(r)        # second one has nothing to do
    with pytest.raises(PoolError) as e:
        m.sync_merge(r, [t])
    assert e.value.code == INVALID_ARG
    with pytest.raises(PoolError) as e:
        m.thread_finish(r, 0)
    assert e.value.code == INVALID_ARG


def test_capacities():
    m = PoolModel(64, 4, max_requests=2, max_threads_per_request=3, max_segments_per_thread=3)
    a, b = m.request_begin(), m.request_begin()
    with pytest.raises(PoolError) as e:
        m.request_begin()
    assert e.value.code == CAPACITY
    m.append_run(a, 0, 2)
    t1, t2 = m.thread_spawn(a), m.thread_spawn(a)
    with pytest.raises(PoolError) as e:
        m.thread_spawn(a)
    assert e.value.code == CAPACITY
    m.append_run(a, 0, 2)
    for t in (t1, t2):
        m.append_run(a, t, 1); m.thread_finish(a, t)
    before = m.dump()
    with pytest.raises(PoolError) as e:
        m.sync_merge(a)                          # would need [main 2][t1][t2][main 2] = 4 entries
    assert e.value.code == CAPACITY and m.dump() == before
    m.sync_merge(a, [t1])                        # [main 2][t1][main 2] fits
    assert len(m.view(a, 0)) == 3


# ------------------------------------------------------------------ spawning on a decoded, not yet appended promise
def _random_state(seed):
    """A pool in some state reached by random valid operations, built twice."""
    import copy
    rng = np.random.default_rng(1000 + seed)
    m = PoolModel(256, 4, max_segments_per_thread=64)
    for _ in range(int(rng.integers(1, 4))):
        req = m.request_begin()
        m.append_run(req, 0, int(rng.integers(0, 11)))
        for _round in range(int(rng.integers(0, 3))):
            forks = [m.thread_spawn(req, int(rng.integers(0, 5)) * 10) for _k in range(int(rng.integers(1, 4)))]
            m.append_run(req, 0, int(rng.integers(0, 6)))
            for t in forks:
                m.append_run(req, t, int(rng.integers(0, 7)))
                m.thread_finish(req, t)
            m.sync_merge(req, forks[:int(rng.integers(0, len(forks) + 1))])
    return m, copy.deepcopy(m), rng


@pytest.mark.parametrize("seed", range(12))
def test_spawn_on_a_pending_promise_equals_append_then_spawn(seed):
    a, b, rng = _random_state(seed)
    for req in sorted(a.requests):
        predicted = int(rng.integers(0, 6)) * 10
        as_step = bool(rng.integers(0, 2))
        # a: the promise enters the pool, then the fork is spawned and takes its first token
        if as_step:
            a.reserve([(req, 0, 1)])
        else:
            a.append_run(req, 0, 1)
        ta = a.thread_spawn(req, predicted)
        # b: the fork is spawned first; promise and the fork's first token enter in one step
        tb = b.thread_spawn(req, predicted, pending=1)
        assert ta == tb
        with pytest.raises(PoolError) as e:
            b.reserve([(req, tb, 1)])                 # the promise is not in the pool yet
        assert e.value.code == BAD_STATE
        with pytest.raises(PoolError) as e:
            b.append_run(req, tb, 1)
        assert e.value.code == BAD_STATE
        if as_step:
            sa = a.reserve([(req, ta, 1)])
            sb = b.reserve([(req, 0, 1), (req, tb, 1)])
            assert sb[1] == sa[0]
        else:
            b.append_run(req, 0, 1)
        assert a.dump() == b.dump()
        # and the two stay the same through the rest of the fork's life
        for m in (a, b):
            m.append_run(req, 0, 3)
            m.append_run(req, ta, 5)
            m.thread_finish(req, ta)
            m.sync_merge(req, [ta])
            m.append_run(req, 0, 1)
        assert a.dump() == b.dump()
        assert a.visible_slots(req, 0) == b.visible_slots(req, 0)


def test_pending_spawn_position_ids_follow_the_closed_form():
    # prompt of n tokens at positions 0..n-1; the promise takes n; the fork starts at n+1; with a predicted block
    # of L tokens the main thread's token after the promise takes n+1+L (Section 6, "Positional Embedding")
    n, L = 7, 30
    m = PoolModel(64, 4)
    req = m.request_begin()
    m.append_run(req, 0, n)
    t = m.thread_spawn(req, L, pending=1)
    assert m.requests[req].pos_next[t] == n + 1
    assert m.requests[req].pos_next[0] == n                 # the promise itself is not displaced
    m.reserve([(req, 0, 1), (req, t, 1)])
    assert m.last_position(req, 0) == n and m.last_position(req, t) == n + 1
    m.reserve([(req, 0, 1), (req, t, 1)])
    assert m.last_position(req, 0) == n + 1 + L and m.last_position(req, t) == n + 2


def test_merging_a_fork_whose_promise_never_arrived_is_refused():
    m = PoolModel(64, 4)
    req = m.request_begin()
    m.append_run(req, 0, 5)
    t = m.thread_spawn(req, 0, pending=1)
    m.thread_finish(req, t)
    before = m.dump()
    with pytest.raises(PoolError) as e:
        m.sync_merge(req, [t])
    assert e.value.code == BAD_STATE and m.dump() == before


# ------------------------------------------------------------------ several tokens of one thread in one step
@pytest.mark.parametrize("seed", range(8))
def test_multi_token_entry_equals_single_token_steps(seed):
    a, b, rng = _random_state(seed)
    for req in sorted(a.requests):
        threads = [0] + [t for t, st in a.requests[req].state.items() if t != 0 and st == 0]
        entries = [(req, t, int(rng.integers(0, 6))) for t in threads if a.requests[req].view[t] or t == 0]
        entries = [(r, t, max(n, 1) if not a.requests[r].view[t] else n) for r, t, n in entries]
        got = a.reserve(entries)
        want, want_pos = [], []
        for r, t, n in entries:                       # the same tokens, one step each, in the same order
            if n == 0:
                want += b.reserve([(r, t, 0)]); want_pos += b.step_positions
            for _ in range(n):
                want += b.reserve([(r, t, 1)]); want_pos += b.step_positions
        assert got == want and a.step_positions == want_pos
        assert a.dump() == b.dump()
        # query j of an entry sees what the thread saw right after its j-th token went in: everything but the later ones
        for (r, t, hide) in PoolModel.queries_of(entries):
            full = a.visible_slots(r, t)
            assert a.visible_slots(r, t, hide) == [s for s in full if s not in set(full[len(full) - hide:])] if hide else full


def test_multi_token_page_count_and_refusal():
    m = PoolModel(3, 4)
    r = m.request_begin()
    m.append_run(r, 0, 3)
    before = m.dump()
    with pytest.raises(PoolError) as e:
        m.reserve([(r, 0, 10)])                        # tokens 3..12 need pages 1, 2 and 3: only two are left
    assert e.value.code == OUT_OF_PAGES and m.dump() == before
    slots = m.reserve([(r, 0, 9)])                     # tokens 3..11: pages 1 and 2
    assert len(slots) == 9 and len(m.free) == 0
    assert PoolModel.queries_of([(r, 0, 3), (r, 1, 0), (r, 2, 1)]) == [(r, 0, 2), (r, 0, 1), (r, 0, 0), (r, 1, 0), (r, 2, 0)]
