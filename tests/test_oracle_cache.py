"""Pins of the expert-buffer model (oracle/cache_sim.py) against things that are not itself:
hand-worked scores of the eviction formula (Section 3.3), a textbook LRU, closed-form special
cases, and brute force over tiny traces."""
import itertools
import random
from collections import OrderedDict

import numpy as np
import pytest

from oracle.cache_sim import ExpertBufferModel, build_profile2, rank_experts, rank_experts2


def _fill(m, ids, layer_fn, acquires):
    for e in ids:
        m.register(e, layer_fn(e), 100)
    for e, n in acquires:
        for _ in range(n):
            s, _, _ = m.acquire(e, 0)
            assert s is not None
            m.release(e)


def test_hand_worked_scores_forward_reading():
    # S = 12 layers, current layer I = 3.  Experts: id = 10*layer + j.
    # f = activations + 1.
    # e41 (layer 4, 2 activations): D = 1,  L = -3        e21 (layer 2, 2): D = 11, L = -3/11
    # e91 (layer 9, 6 activations): D = 6,  L = -7/6      e31 (layer 3, 0): D = 0, protected
    # highest L leaves first: e21 (-0.27), then e91 (-1.17), then e41 (-3), last the protected e31
    m = ExpertBufferModel(4, 12, "forward")
    _fill(m, [41, 21, 91, 31], lambda e: e // 10, [(41, 2), (21, 2), (91, 6)])
    m.prefetch(31, 0)
    order = [m.slot_content[s] for s in m.eviction_order(3)]
    assert order == [21, 91, 41, 31]


def test_hand_worked_scores_printed_reading():
    # same buffer, printed distance (S - i + I) mod S at I = 3:
    # e41: D = 11, L = -3/11   e21: D = 1, L = -3   e91: D = 6, L = -7/6   e31: D = 0 protected
    m = ExpertBufferModel(4, 12, "printed")
    _fill(m, [41, 21, 91, 31], lambda e: e // 10, [(41, 2), (21, 2), (91, 6)])
    m.prefetch(31, 0)
    order = [m.slot_content[s] for s in m.eviction_order(3)]
    assert order == [41, 91, 21, 31]


def test_unused_preloads_rank_by_distance_and_ties_go_to_the_lowest_slot():
    m = ExpertBufferModel(3, 8, "forward")
    for e, layer in ((1, 5), (2, 6), (3, 7)):
        m.register(e, layer)
        m.prefetch(e, 0)                   # never activated: L = -1/5, -1/6, -1/7: the farthest layer leaves first
    assert m.eviction_order(0) == [2, 1, 0]
    m.register(4, 1)
    s, ev = m.prefetch(4, 0)
    assert (s, ev) == (2, 3)
    t = ExpertBufferModel(3, 8, "forward")
    for e in (1, 2, 3):
        t.register(e, 5)
        t.prefetch(e, 0)                   # same layer, same count: a three-way tie
    assert t.eviction_order(0) == [0, 1, 2]


def test_lru_rule_is_textbook_lru():
    rng = random.Random(5)
    m = ExpertBufferModel(4, 6, "lru")
    for e in range(12):
        m.register(e, e % 6)
    book = OrderedDict()
    for step in range(400):
        e = rng.randrange(12)
        s, loaded, ev = m.acquire(e, step % 6)
        m.release(e)
        if e in book:
            assert not loaded and ev is None
            book.move_to_end(e)
        else:
            assert loaded
            if len(book) == 4:
                oldest, _ = book.popitem(last=False)
                assert ev == oldest
            else:
                assert ev is None
            book[e] = True
    assert set(m.where) == set(book)
    assert m.counters["hits"] + m.counters["misses"] == 400


def test_fifo_and_lfu_orders_worked_by_hand():
    """Three slots, experts A B C D of one layer.  Loads: A, B, C (in that order); uses afterwards:
    C twice, A once, B never again.  Every expert was activated once when it was loaded, so the
    counts are A 2, B 1, C 3.
      FIFO: the one loaded first leaves: A, then B, then C, whatever their use.
      LFU: fewest activations first: B (1), then A (2), then C (3).
      LRU for contrast: the touches in order are A, B, C, C, C, A, so the least recently touched
      is B, then C, then A."""
    def filled(rule):
        m = ExpertBufferModel(3, 1, rule)
        for e in "ABCD":
            m.register(e, 0)
        for e in "ABC":
            m.acquire(e, 0)
            m.release(e)
        for e in "CCA":
            assert m.acquire(e, 0)[1] is False
            m.release(e)
        return m
    name = lambda m, order: [m.slot_content[s] for s in order]
    assert name(filled("fifo"), filled("fifo").eviction_order(0)) == ["A", "B", "C"]
    assert name(filled("lfu"), filled("lfu").eviction_order(0)) == ["B", "A", "C"]
    assert name(filled("lru"), filled("lru").eviction_order(0)) == ["B", "C", "A"]
    # and the eviction really takes the head of the order
    m = filled("fifo")
    assert m.acquire("D", 0) == (0, True, "A")
    m = filled("lfu")
    assert m.acquire("D", 0) == (1, True, "B")
    # LFU ties (equal counts) go to the expert loaded earliest
    t = ExpertBufferModel(2, 1, "lfu")
    for e in "XYZ":
        t.register(e, 0)
    for e in "YX":
        t.acquire(e, 0)
        t.release(e)
    assert t.acquire("Z", 0) == (0, True, "Y")


def test_fifo_rule_is_a_textbook_queue():
    rng = random.Random(9)
    m = ExpertBufferModel(4, 6, "fifo")
    for e in range(12):
        m.register(e, e % 6)
    queue = []
    for step in range(400):
        e = rng.randrange(12)
        s, loaded, ev = m.acquire(e, step % 6)
        m.release(e)
        if e in queue:
            assert not loaded and ev is None
        else:
            assert loaded
            if len(queue) == 4:
                assert ev == queue.pop(0)
            else:
                assert ev is None
            queue.append(e)
    assert set(m.where) == set(queue)


@pytest.mark.parametrize("rule", ["forward", "printed", "lru", "lfu", "fifo"])
def test_no_eviction_when_everything_fits_and_counters_add_up(rule):
    rng = random.Random(7)
    m = ExpertBufferModel(16, 4, rule)
    for e in range(16):
        m.register(e, e % 4, 10 + e)
    for step in range(200):
        e = rng.randrange(16)
        if rng.random() < 0.3:
            m.prefetch(e, step % 4)
        else:
            assert m.acquire(e, step % 4)[0] is not None
            m.release(e)
    c = m.counters
    assert c["evictions"] == 0
    assert c["misses"] + c["prefetched"] == len(m.where)             # every expert was loaded exactly once
    assert c["bytes_copied"] == sum(10 + e for e in m.where)
    assert c["prefetch_hits"] <= c["prefetched"]


def test_experts_in_use_are_never_evicted_and_a_full_buffer_refuses():
    m = ExpertBufferModel(2, 4, "forward")
    for e in range(4):
        m.register(e, e)
    assert m.acquire(0, 0)[0] == 0 and m.acquire(1, 0)[0] == 1      # both slots in use
    assert m.prefetch(2, 0) == (None, None) and m.counters["prefetch_refused"] == 1
    assert m.acquire(3, 0) == (None, False, None)
    m.release(1)
    s, loaded, ev = m.acquire(3, 0)
    assert (s, loaded, ev) == (1, True, 1)


def test_victim_maximises_the_score_brute_force():
    """For every small configuration: the evicted expert has the highest L = -f/D among the
    candidates with D > 0 (computed here directly from the formula with floats)."""
    for layers, freqs, current in itertools.product(itertools.permutations(range(1, 5), 3), [(0, 1, 5), (3, 3, 1), (2, 7, 4)], range(5)):
        m = ExpertBufferModel(3, 5, "forward")
        for j, (layer, f) in enumerate(zip(layers, freqs)):
            m.register(j, layer)
            m.prefetch(j, 0)
            for _ in range(f):
                m.acquire(j, 0)
                m.release(j)
        m.register(99, 0)
        s, ev = m.prefetch(99, current)
        scores = {}
        for j, (layer, f) in enumerate(zip(layers, freqs)):
            D = (layer - current) % 5
            if D:
                scores[j] = -(f + 1) / D
        if scores:
            best = max(scores.values())
            assert scores[ev] == pytest.approx(best)
            assert ev == min(j for j, v in scores.items() if v == pytest.approx(best))


def test_rank_experts():
    prior = [[0.7, 0.2, 0.1], [0.1, 0.1, 0.8], [0.3, 0.3, 0.4]]
    assert rank_experts(prior, [0]) == [0, 1, 2]
    assert rank_experts(prior, [1]) == [2, 0, 1]            # tie between 0 and 1: lower index first
    assert rank_experts(prior, [0, 1]) == [2, 0, 1]         # sums 0.8, 0.3, 0.9


def test_profile_keyed_on_two_previous_layers_hand_worked():
    """Four tokens through three layers of three experts, top-1 (picks per layer):
    (0,1,2) (0,1,2) (0,1,0) (1,1,2).  Key (0,1) was seen three times: expert 2 followed twice,
    expert 0 once; key (1,1) once, followed by expert 2; every other key was never seen."""
    trace = [[[0], [1], [2]], [[0], [1], [2]], [[0], [1], [0]], [[1], [1], [2]]]
    t = build_profile2(trace, 3)
    assert t[0] == [[[0.0] * 3] * 3] * 3 and t[1] == [[[0.0] * 3] * 3] * 3
    assert t[2][0][1] == [1 / 3, 0.0, 2 / 3]
    assert t[2][1][1] == [0.0, 0.0, 1.0]
    assert t[2][2][0] == [1 / 3] * 3
    assert rank_experts2(t[2], [0], [1]) == [2, 0, 1]
    assert rank_experts2(t[2], [1], [1]) == [2, 0, 1]          # 0 and 1 tie at zero: lower index first
    assert rank_experts2(t[2], [0, 1], [1]) == [2, 0, 1]       # sums 1/3, 0, 5/3


def test_profile2_rows_are_distributions_and_reduce_to_first_order_when_layer_n_minus_2_is_constant():
    """Closed forms: with Top-K = k every seen key's row sums to k; if layer n-2 always activates
    the same expert, the table is the first-order conditional P(e | b) counted directly."""
    rng = np.random.default_rng(2)
    E, k, L = 5, 2, 4
    trace = [[sorted(rng.choice(E, size=k, replace=False).tolist()) for _ in range(L)] for _ in range(300)]
    t = build_profile2(trace, E)
    for n in range(2, L):
        for a in range(E):
            for b in range(E):
                assert abs(sum(t[n][a][b]) - k) < 1e-12 or t[n][a][b] == [1.0 / E] * E
    trace1 = [[[0], [int(rng.integers(0, E))], [int(rng.integers(0, E))]] for _ in range(400)]
    t1 = build_profile2(trace1, E)
    for b in range(E):
        nb = sum(1 for r in trace1 if r[1] == [b])
        for e in range(E):
            direct = sum(1 for r in trace1 if r[1] == [b] and r[2] == [e]) / nb
            assert abs(t1[2][0][b][e] - direct) < 1e-12


def test_rank_experts2_equals_brute_force_and_first_order_on_a_separable_table():
    rng = np.random.default_rng(4)
    E = 6
    tab = rng.random((E, E, E))
    for _ in range(20):
        p2 = rng.integers(0, E, size=2).tolist()
        p1 = rng.integers(0, E, size=2).tolist()
        score = np.einsum("abe->e", tab[np.ix_(p2, p1)])
        assert rank_experts2(tab.tolist(), p2, p1) == sorted(range(E), key=lambda e: (-score[e], e))
    # a table that ignores layer n-2 ranks exactly as the first-order one
    first = rng.random((E, E))
    tab2 = np.broadcast_to(first[None, :, :], (E, E, E))
    for _ in range(10):
        p1 = rng.integers(0, E, size=2).tolist()
        assert rank_experts2(tab2.tolist(), [3], p1) == rank_experts(first.tolist(), p1)
