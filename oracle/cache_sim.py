"""Plain, slow model of the expert buffer and its eviction rule (test infrastructure: only tests,
the smoke check and the bench's CPU arms may use it; it shares no code with the CUDA library).

What it follows (EdgeMoE, arXiv 2308.14352, Section 3.3):
* "Cache eviction policy": a buffer of fixed size holds experts; an activated expert found in
  the buffer is a hit, otherwise it is fetched and, when the buffer is full, an expert is
  evicted.  Every expert j of layer i has the score  L = -f / D,  f its activation count so far,
  D a distance between its layer i and the current layer I out of S layers; the expert with the
  HIGHEST score is evicted.
* "Preloading and pipeline": before a layer's router is known, experts are preloaded in the
  order of their estimated activation probability, unless present already.
* "Estimating expert activation a priori": the probability estimate comes from a table keyed by
  earlier layers' activations (here: one previous layer, as the workload definition asks).

Two more textbook rules are modelled for comparison, as in the paper's evaluation of eviction
policies (its cache-hit-ratio figure compares five): `lfu` (the expert with the fewest activations
so far leaves; ties: the one loaded earliest, then the lowest slot) and `fifo` (the expert loaded
earliest leaves, whatever its use).

Readings where the paper is silent or at odds with itself:
* D: the printed formula is (S - i + I) mod S; the text wants layers "going to be executed
  soon" kept, which is (i - I) mod S.  Both exist: `forward` (default) and `printed`.
* D = 0 (an expert of the current layer): the formula divides by zero; such experts are
  protected and leave only when no other candidate exists (then lowest f first).
* f: the paper's f comes from an offline profile; there is none here, so f = 1 + the running
  count of activations (acquire calls) of that expert: a preloaded expert that has not been used
  yet is then ranked by its layer distance instead of leaving first with L = 0.
* ties: the lowest slot index leaves.
* an expert in use (acquired, not released) is never evicted; a preload that finds no
  candidate is dropped; an activation that finds none is an error.
Scores are compared as exact fractions."""
from fractions import Fraction


class ExpertBufferModel:
    def __init__(self, n_slots, n_layers, rule="forward"):
        assert rule in ("forward", "printed", "lru", "lfu", "fifo")
        self.n_slots, self.S, self.rule = n_slots, n_layers, rule
        self.layer_of, self.bytes_of = {}, {}
        self.slot_content = [None] * n_slots     # expert id or None
        self.where = {}                          # expert id -> slot
        self.freq = {}                           # expert id -> activations so far
        self.in_use = {}                         # expert id -> acquire count not yet released
        self.fresh_from_preload = set()
        self.touched = [0] * n_slots
        self.loaded_at = [0] * n_slots           # tick at which the slot's present content was put there
        self.tick = 0
        self.counters = dict(hits=0, misses=0, prefetch_hits=0, prefetched=0, prefetch_redundant=0,
                             prefetch_refused=0, evictions=0, bytes_copied=0)

    def register(self, eid, layer, nbytes=0):
        assert eid not in self.layer_of
        self.layer_of[eid], self.bytes_of[eid] = layer, nbytes
        self.freq[eid], self.in_use[eid] = 0, 0

    # -- the score of Section 3.3 ----------------------------------------------------------
    def distance(self, eid, current_layer):
        i, I, S = self.layer_of[eid], current_layer, self.S
        return (S - i + I) % S if self.rule == "printed" else (i - I) % S

    def eviction_order(self, current_layer):
        """Slots that may be evicted, first to leave first."""
        cands = [s for s in range(self.n_slots)
                 if self.slot_content[s] is not None and self.in_use[self.slot_content[s]] == 0]
        if self.rule == "lru":
            return sorted(cands, key=lambda s: (self.touched[s], s))
        if self.rule == "fifo":
            return sorted(cands, key=lambda s: (self.loaded_at[s], s))
        if self.rule == "lfu":
            return sorted(cands, key=lambda s: (self.freq[self.slot_content[s]], self.loaded_at[s], s))

        def key(s):
            eid = self.slot_content[s]
            D = self.distance(eid, current_layer)
            if D == 0:                      # protected: after everybody else, lowest count first
                return (1, Fraction(self.freq[eid]), s)
            return (0, Fraction(self.freq[eid] + 1, D), s)   # highest L = -f/D first  <=>  smallest f/D first
        return sorted(cands, key=key)

    def _put(self, eid, current_layer):
        """-> (slot, evicted id or None), or (None, None) when nothing can leave"""
        free = [s for s in range(self.n_slots) if self.slot_content[s] is None]
        evicted = None
        if free:
            s = free[0]
        else:
            order = self.eviction_order(current_layer)
            if not order:
                return None, None
            s = order[0]
            evicted = self.slot_content[s]
            del self.where[evicted]
            self.fresh_from_preload.discard(evicted)
            self.counters["evictions"] += 1
        self.slot_content[s] = eid
        self.where[eid] = s
        self.tick += 1
        self.touched[s] = self.tick
        self.loaded_at[s] = self.tick
        self.counters["bytes_copied"] += self.bytes_of[eid]
        return s, evicted

    # -- preloading -----------------------------------------------------------------------
    def prefetch(self, eid, current_layer):
        """-> (slot loaded into or None, evicted id or None)"""
        if eid in self.where:
            self.counters["prefetch_redundant"] += 1
            return None, None
        s, ev = self._put(eid, current_layer)
        if s is None:
            self.counters["prefetch_refused"] += 1
            return None, None
        self.fresh_from_preload.add(eid)
        self.counters["prefetched"] += 1
        return s, ev

    # -- activation -----------------------------------------------------------------------
    def acquire(self, eid, current_layer):
        """-> (slot, loaded now?, evicted id or None); slot None = every slot is in use"""
        loaded, ev = False, None
        if eid in self.where:
            s = self.where[eid]
            self.counters["hits"] += 1
            if eid in self.fresh_from_preload:
                self.counters["prefetch_hits"] += 1
        else:
            s, ev = self._put(eid, current_layer)
            if s is None:
                return None, False, None
            self.counters["misses"] += 1
            loaded = True
        self.fresh_from_preload.discard(eid)
        self.freq[eid] += 1
        self.in_use[eid] += 1
        self.tick += 1
        self.touched[s] = self.tick
        return s, loaded, ev

    def release(self, eid):
        if eid not in self.where or self.in_use[eid] <= 0:
            return None
        self.in_use[eid] -= 1
        return self.where[eid]


def rank_experts(prior, prev_ids):
    """Next layer's experts by descending estimated probability (first-order table: row p of
    `prior` is the distribution given that the previous layer picked p; several picks: their rows
    are added), ties by lower index."""
    E = len(prior)
    score = [sum(float(prior[p][e]) for p in prev_ids) for e in range(E)]
    return sorted(range(E), key=lambda e: (-score[e], e))


def build_profile2(trace, n_experts):
    """The offline statistical profile of Section 3.3 ("Opportunistic preloading"): a dictionary
    whose key is the activation status of the two previous MoE layers and whose value is the
    probability of each expert of the next layer being activated.  trace[token][layer] lists the
    experts a token activated in a layer.  Returned: table[n][a][b][e] for every layer n >= 2 =
    (times e was active in layer n while a was active in layer n-2 and b in layer n-1) / (times a
    and b were active in layers n-2 and n-1); keys never seen get the uniform distribution; layers
    0 and 1 (no two previous layers) get all zeros.  With Top-K > 1 a key is every (a, b) pair of
    the two layers' picks."""
    n_layers = len(trace[0])
    E = n_experts
    table = [[[[0.0] * E for _ in range(E)] for _ in range(E)] for _ in range(n_layers)]
    seen = [[[0] * E for _ in range(E)] for _ in range(n_layers)]
    for row in trace:
        for n in range(2, n_layers):
            for a in row[n - 2]:
                for b in row[n - 1]:
                    seen[n][a][b] += 1
                    for e in row[n]:
                        table[n][a][b][e] += 1.0
    for n in range(2, n_layers):
        for a in range(E):
            for b in range(E):
                c = seen[n][a][b]
                for e in range(E):
                    table[n][a][b][e] = table[n][a][b][e] / c if c else 1.0 / E
    return table


def rank_experts2(table_n, prev2_ids, prev1_ids):
    """Next layer's experts by descending estimated probability given the picks of the two previous
    layers (table_n[a][b] = distribution for the key (a, b); several picks per layer: the rows of
    every (a, b) pair are added), ties by lower index."""
    E = len(table_n)
    score = [sum(float(table_n[a][b][e]) for a in prev2_ids for b in prev1_ids) for e in range(E)]
    return sorted(range(E), key=lambda e: (-score[e], e))
