"""Hit ratio of the expert cache over cache sizes and eviction rules on a synthetic activation
trace (the experiment behind the paper's cache-policy figure in Section 4, without its datasets):
decode tokens walk through S layers, every layer activates top_k of E experts, and the picks of
a layer follow the previous layer's picks through a seeded layer-transition prior.  Only the
library's host-side bookkeeping runs (emoe_policy_*): no GPU is needed.

    python -m paper_2308_14352_b200.cache_sweep [--layers 32 --experts 8 --top-k 2 --steps 512]
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


def run(trace, prior, n_layers, n_experts, n_slots, rule_code, n_prefetch, warm_steps):
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
                    order = B.emoe_rank_experts(prior, picks.astype(np.int32))
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--experts", type=int, default=8)
    ap.add_argument("--top-k", type=int, default=2)
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--warm", type=int, default=64)
    ap.add_argument("--beta", type=float, default=4.0)
    ap.add_argument("--seed", type=int, default=4)
    args = ap.parse_args()
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
