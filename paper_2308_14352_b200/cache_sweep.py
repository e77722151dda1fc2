"""Hit ratio of the expert cache over cache sizes and eviction rules on a synthetic activation
trace (the experiment behind the paper's cache-policy figure in Section 4, without its datasets):
decode tokens walk through S layers, every layer activates top_k of E experts, and the picks of
a layer follow the previous layer's picks through a seeded layer-transition prior.  Only the
library's host-side bookkeeping runs (emoe_policy_*): no GPU is needed.

    python -m paper_2308_14352_b200.cache_sweep [--layers 32 --experts 8 --top-k 2 --steps 512]
    python -m paper_2308_14352_b200.cache_sweep --predictor-orders      # one previous layer as key vs two
"""
from __future__ import annotations

import argparse

import numpy as np

from . import binding as B

RULES = (("forward", B.EVICT_FORWARD), ("printed", B.EVICT_PRINTED), ("lru", B.EVICT_LRU), ("lfu", B.EVICT_LFU),
         ("fifo", B.EVICT_FIFO))


def make_trace(n_layers: int, n_experts: int, top_k: int, steps: int, beta: float, seed: int):
    """picks[step][layer] = sorted expert indices; the prior that generated them."""
    rng = np.random.default_rng(seed)
    prior = rng.random((n_experts, n_experts)) ** 4
    prior /= prior.sum(axis=1, keepdims=True)
    trace = []
    for _ in range(steps):
        prev, row = None, []
        for _l in range(n_layers):
            logit = rng.gumbel(size=n_experts)                       # sampling without replacement from p^beta
            if prev is not None:
                logit = logit + beta * np.log(prior[prev].mean(axis=0) + 1e-9)
            prev = np.sort(np.argsort(-logit, kind="stable")[:top_k])
            row.append(prev)
        trace.append(row)
    return trace, prior.astype(np.float32)


def make_trace2(n_layers: int, n_experts: int, top_k: int, steps: int, beta: float, seed: int, table_seed: int):
    """A trace whose layer n depends on the picks of layers n-1 AND n-2 (the statistics Section 3.3
    reports: two previous layers observed): two seeded transition tables, one per distance, shared by
    every trace drawn with the same table_seed."""
    trng = np.random.default_rng(table_seed)
    near = trng.random((n_experts, n_experts)) ** 4
    far = trng.random((n_experts, n_experts)) ** 4
    near /= near.sum(axis=1, keepdims=True)
    far /= far.sum(axis=1, keepdims=True)
    rng = np.random.default_rng(seed)
    trace = []
    for _ in range(steps):
        row = []
        for l in range(n_layers):
            logit = rng.gumbel(size=n_experts)
            if l >= 1:
                logit = logit + beta * np.log(near[row[l - 1]].mean(axis=0) + 1e-9)
            if l >= 2:
                logit = logit + beta * np.log(far[row[l - 2]].mean(axis=0) + 1e-9)
            row.append(np.sort(np.argsort(-logit, kind="stable")[:top_k]))
        trace.append(row)
    return trace


def first_order_profile(trace, n_layers, n_experts):
    """P(e active in layer n | p active in layer n-1), counted over a trace: [n_layers][E][E]."""
    cnt = np.zeros((n_layers, n_experts, n_experts))
    for row in trace:
        for l in range(1, n_layers):
            for p in row[l - 1]:
                cnt[l, p, row[l]] += 1
    tot = cnt.sum(axis=2, keepdims=True)
    return np.where(tot > 0, cnt / np.maximum(tot, 1), 1.0 / n_experts).astype(np.float32)


def run(trace, prior, n_layers, n_experts, n_slots, rule_code, n_prefetch, warm_steps, rank_fn=None):
    """rank_fn(next_layer, row, picks) -> order of the next layer's experts; default: the first-order
    prior shared by all layers."""
    h = B.emoe_policy_create(n_slots, n_layers, rule_code)
    try:
        for l in range(n_layers):
            for e in range(n_experts):
                B.emoe_policy_register(h, l * n_experts + e, l, 1)
        base = None
        for step, row in enumerate(trace):
            if step == warm_steps:
                base = B.emoe_policy_get_stats(h)
            for l, picks in enumerate(row):
                if n_prefetch and l + 1 < n_layers:
                    order = (rank_fn(l + 1, row, picks) if rank_fn is not None
                             else B.emoe_rank_experts(prior, picks.astype(np.int32)))
                    for e in order[:n_prefetch]:
                        B.emoe_policy_prefetch(h, (l + 1) * n_experts + int(e), l)
                ids = [l * n_experts + int(e) for e in picks]
                for i in ids:
                    B.emoe_policy_acquire(h, i, l)
                for i in ids:
                    B.emoe_policy_release(h, i)
        st = B.emoe_policy_get_stats(h)
        d = {k: st[k] - base[k] for k in st}
        loads = d["misses"] + d["prefetched"]
        return d["hits"] / max(1, d["hits"] + d["misses"]), loads / max(1, len(trace) - warm_steps)
    finally:
        B.emoe_policy_destroy(h)


def predictor_orders(args) -> None:
    """Profiles built from one trace (the offline phase), used on another drawn from the same
    statistics: preload hit ratio and Top-K prediction accuracy with one and with two previous layers
    as key."""
    L, E, k = args.layers, args.experts, args.top_k
    prof = make_trace2(L, E, k, 4 * args.steps, args.beta, args.seed + 100, args.seed)
    test = make_trace2(L, E, k, args.steps + args.warm, args.beta, args.seed + 200, args.seed)
    p1 = first_order_profile(prof, L, E)
    p2 = B.emoe_build_profile2(np.array([[list(x) for x in row] for row in prof], dtype=np.int32), E)

    def rank1(nl, row, picks):
        return B.emoe_rank_experts(p1[nl], picks.astype(np.int32))

    def rank2(nl, row, picks):
        if nl < 2:
            return rank1(nl, row, picks)
        return B.emoe_rank_experts2(p2[nl], row[nl - 2].astype(np.int32), picks.astype(np.int32))

    def accuracy(rank):
        good = total = 0
        for row in test[args.warm:]:
            for l in range(L - 1):
                top = set(int(e) for e in rank(l + 1, row, row[l])[:k])
                good += len(top & set(int(e) for e in row[l + 1]))
                total += k
        return good / total

    print(f"{L} layers x {E} experts, top-{k}; layer n drawn from the picks of layers n-1 and n-2 (beta = {args.beta}); "
          f"profile from {4 * args.steps} tokens, evaluated on {args.steps} others")
    print(f"share of the activated experts among the top-{k} predicted: one previous layer as key {accuracy(rank1):.3f}, "
          f"two previous layers {accuracy(rank2):.3f}")
    print(f"| slots | hit ratio, key = 1 layer (loads per step) | hit ratio, key = 2 layers (loads per step) |")
    print("|---|---|---|")
    total = L * E
    for n in sorted({max(2 * E, total * f // 16) for f in (2, 4, 8, 12)}):
        cells = []
        for fn in (rank1, rank2):
            hit, loads = run(test, None, L, E, n, B.EVICT_FORWARD, k, args.warm, fn)
            cells.append(f"{hit:.3f} ({loads:.1f})")
        print(f"| {n} | " + " | ".join(cells) + " |")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--experts", type=int, default=8)
    ap.add_argument("--top-k", type=int, default=2)
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--warm", type=int, default=64)
    ap.add_argument("--beta", type=float, default=4.0)
    ap.add_argument("--seed", type=int, default=4)
    ap.add_argument("--predictor-orders", action="store_true",
                    help="compare the profile keyed on one previous layer with the one keyed on two (Section 3.3)")
    args = ap.parse_args()
    if args.predictor_orders:
        predictor_orders(args)
        return
    trace, prior = make_trace(args.layers, args.experts, args.top_k, args.steps + args.warm, args.beta, args.seed)
    total = args.layers * args.experts
    sizes = sorted({max(2 * args.experts, total * f // 16) for f in (2, 4, 6, 8, 12, 16)})
    print(f"{args.layers} layers x {args.experts} experts, top-{args.top_k}, {args.steps} decode steps after {args.warm} warm-up steps, "
          f"beta = {args.beta}, seed {args.seed}; hit ratio (expert loads per step)")
    print("| slots | " + " | ".join(f"{r}, no preload | {r}, preload top-{args.top_k}" for r, _ in RULES) + " |")
    print("|---|" + "---|" * (2 * len(RULES)))
    for n in sizes:
        cells = []
        for _, code in RULES:
            for p in (0, args.top_k):
                hit, loads = run(trace, prior, args.layers, args.experts, n, code, p, args.warm)
                cells.append(f"{hit:.3f} ({loads:.1f})")
        print(f"| {n} | " + " | ".join(cells) + " |")


if __name__ == "__main__":
    main()
