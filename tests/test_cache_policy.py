"""The library's cache bookkeeping (emoe_policy_*: the same host code that drives the device
cache) against the plain model, operation by operation, on random traces: slots, evictions and
counters are integer work and must agree exactly.  Runs without a GPU."""
import random

import numpy as np
import pytest

from oracle.cache_sim import ExpertBufferModel, build_profile2, rank_experts, rank_experts2
from paper_2308_14352_b200 import binding as B

def _bookkeeping(stats):
    """The counters the bookkeeping model has (the library adds its timing fields)."""
    return {k: v for k, v in stats.items() if k not in ("exposed_copy_ns", "timed_acquires")}


RULES = [("forward", B.EVICT_FORWARD), ("printed", B.EVICT_PRINTED), ("lru", B.EVICT_LRU), ("lfu", B.EVICT_LFU),
         ("fifo", B.EVICT_FIFO)]


@pytest.mark.parametrize("rule,code", RULES)
@pytest.mark.parametrize("n_slots,n_layers,per_layer,seed", [(3, 4, 2, 0), (8, 6, 4, 1), (16, 12, 8, 2), (5, 32, 8, 3)])
def test_random_traces_agree(rule, code, n_slots, n_layers, per_layer, seed):
    rng = random.Random(seed)
    model = ExpertBufferModel(n_slots, n_layers, rule)
    h = B.emoe_policy_create(n_slots, n_layers, code)
    try:
        ids = []
        for layer in range(n_layers):
            for j in range(per_layer):
                eid = 1000 * layer + j
                nbytes = rng.randrange(1, 1 << 20)
                model.register(eid, layer, nbytes)
                B.emoe_policy_register(h, eid, layer, nbytes)
                ids.append(eid)
        held = []
        for step in range(3000):
            layer = step % n_layers
            op = rng.random()
            if op < 0.35:
                eid = rng.choice(ids)
                s_ref, ev_ref = model.prefetch(eid, layer)
                s, ev = B.emoe_policy_prefetch(h, eid, layer)
                assert (s, ev) == (-1 if s_ref is None else s_ref, -1 if ev_ref is None else ev_ref), step
            elif op < 0.8:
                eid = rng.choice([e for e in ids if e // 1000 == layer])    # activations come from the current layer
                s_ref, ld_ref, ev_ref = model.acquire(eid, layer)
                s, ld, ev = B.emoe_policy_acquire(h, eid, layer)
                assert (s, ld, ev) == (-1 if s_ref is None else s_ref, ld_ref, -1 if ev_ref is None else ev_ref), step
                if s_ref is not None:
                    held.append(eid)
            elif held:
                eid = held.pop(rng.randrange(len(held)))
                assert B.emoe_policy_release(h, eid) == model.release(eid)
            if len(held) >= n_slots - 1:                                 # keep the trace moving
                eid = held.pop(0)
                assert B.emoe_policy_release(h, eid) == model.release(eid)
            if step % 97 == 0:
                assert _bookkeeping(B.emoe_policy_get_stats(h)) == model.counters
        assert _bookkeeping(B.emoe_policy_get_stats(h)) == model.counters
        assert model.counters["evictions"] > 0
    finally:
        B.emoe_policy_destroy(h)


def test_policy_argument_errors():
    with pytest.raises(B.EmoeError):
        B.emoe_policy_create(0, 4, B.EVICT_FORWARD)
    with pytest.raises(B.EmoeError):
        B.emoe_policy_create(4, 4, 17)
    h = B.emoe_policy_create(2, 4, B.EVICT_LRU)
    try:
        B.emoe_policy_register(h, 5, 1, 10)
        with pytest.raises(B.EmoeError):
            B.emoe_policy_register(h, 5, 2, 10)       # same id twice
        with pytest.raises(B.EmoeError):
            B.emoe_policy_acquire(h, 6, 0)            # unknown id
        assert B.emoe_policy_release(h, 5) == -1      # not held
    finally:
        B.emoe_policy_destroy(h)


def test_rank_experts_matches_the_model():
    rng = np.random.default_rng(3)
    for E, k in ((8, 2), (8, 1), (32, 4), (5, 5)):
        prior = rng.random((E, E)).astype(np.float32)
        prior /= prior.sum(axis=1, keepdims=True)
        prior[1] = prior[0]                                   # equal rows: ties within a sum stay possible
        prior[:, 3] = prior[:, 2]                             # equal columns: exact ties between experts 2 and 3
        for _ in range(20):
            prev = rng.integers(0, E, size=k)
            got = B.emoe_rank_experts(prior, prev)
            assert got.tolist() == rank_experts(prior.tolist(), prev.tolist())


def test_profile_keyed_on_two_previous_layers_matches_the_model():
    """emoe_build_profile2 / emoe_rank_experts2 (Section 3.3: key = the two previous layers)
    against the model, entry by entry and rank by rank, incl. keys never seen and exact ties."""
    rng = np.random.default_rng(6)
    for E, k, L, n in ((4, 1, 5, 60), (6, 2, 4, 200), (3, 3, 3, 10)):
        trace = np.stack([np.stack([np.sort(rng.choice(E, size=k, replace=False)) for _ in range(L)]) for _ in range(n)])
        got = B.emoe_build_profile2(trace, E)
        ref = np.array(build_profile2(trace.tolist(), E))
        assert got.shape == ref.shape
        np.testing.assert_allclose(got, ref, rtol=0, atol=1e-7)
        for _ in range(20):
            layer = int(rng.integers(2, L))
            p2 = rng.choice(E, size=k, replace=False)
            p1 = rng.choice(E, size=k, replace=False)
            assert B.emoe_rank_experts2(got[layer], p2, p1).tolist() == rank_experts2(got[layer].astype(np.float64).tolist(),
                                                                                    p2.tolist(), p1.tolist())
    with pytest.raises(B.EmoeError):
        B.emoe_build_profile2(np.full((2, 3, 1), 9, dtype=np.int32), 4)      # id outside [0, E)
