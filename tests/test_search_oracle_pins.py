"""Pins for the search oracle (Algorithms 1 and 2): evaluation-count bounds stated in the paper's
captions, exact recovery of a planted threshold, agreement with brute force on tiny problems."""
import itertools
import math

import numpy as np
import pytest

from oracle import search_oracle as so


def additive_model(cost, bs):
    """Accuracy = 1 - sum of per-layer penalties; penalty grows as bits shrink (monotone, separable)."""
    top = max(bs)

    def evaluate(cfg):
        return 1.0 - sum(cost[l] * (top - b) for l, b in enumerate(cfg))
    return evaluate


@pytest.mark.parametrize("n,seed", [(54, 0), (144, 1), (7, 2), (1, 3)])
def test_evaluation_counts_within_paper_bounds(n, seed):
    rng = np.random.default_rng(seed)
    cost = rng.uniform(0, 1e-3, n)
    order = list(np.argsort(cost, kind="stable"))
    bs = [16, 8, 4]
    nb = len(bs) - 1                                            # bit widths actually searched
    for target in (0.5, 0.98, 0.999, 1.1):
        calls = []
        ev = additive_model(cost, bs)
        w, vis = so.bisection_search(n, order, bs, target, lambda c: (calls.append(1), ev(c))[1])
        assert len(vis) == len(calls) <= nb * (math.ceil(math.log2(n + 1)) + 2)    # O(b log N)
        calls.clear()
        w, vis = so.greedy_search(n, order, bs, target, lambda c: (calls.append(1), ev(c))[1])
        assert n <= len(vis) <= nb * n                           # between N and bN
        if target > 1:
            assert w == [16] * n                                 # nothing can be lowered


def test_bisection_finds_planted_threshold_and_greedy_the_planted_set():
    n = 40
    bs = [16, 8]
    # lowering any of the first k layers (in sensitivity order) is free, any other one breaks the model
    for k in (0, 1, 13, 39, 40):
        order = list(np.random.default_rng(k).permutation(n))
        free = set(order[:k])
        ev = lambda cfg: 1.0 if all(b == 16 or l in free for l, b in enumerate(cfg)) else 0.0
        w, _ = so.bisection_search(n, order, bs, 0.5, ev)
        # with floor halving the threshold approaches but never reaches the full list length
        assert {l for l in range(n) if w[l] == 8} == set(order[:min(k, n - 1)])
        # greedy does not need the order to be right
        shuffled = list(np.random.default_rng(100 + k).permutation(n))
        w, vis = so.greedy_search(n, shuffled, bs, 0.5, ev)
        assert {l for l in range(n) if w[l] == 8} == free and len(vis) == n


def test_second_bit_width_only_revisits_layers_that_took_the_first():
    n, bs = 10, [16, 8, 4]
    cost = np.linspace(1e-3, 1e-2, n)
    order = list(range(n))
    ev = additive_model(cost, bs)
    for search in (so.bisection_search, so.greedy_search):
        w, vis = search(n, order, bs, 0.8, ev)
        assert ev(w) >= 0.8
        eight_or_less = [l for l in range(n) if w[l] <= 8]
        assert all(w[l] == 16 for l in range(n) if l not in eight_or_less)
        # every configuration with a 4 was evaluated after the 8-bit pass, and only on 8-bit layers
        first4 = next((i for i, c in enumerate(vis) if 4 in c), len(vis))
        assert all(4 not in c for c in vis[:first4])
        for c in vis[first4:]:
            assert all(w8 in (8, 4) for l, w8 in enumerate(c) if c[l] == 4)


@pytest.mark.parametrize("seed", range(5))
def test_against_brute_force_on_tiny_problems(seed):
    """For a separable monotone model the best prefix (bisection) and the greedy result can be
    checked against all 2^N configurations."""
    rng = np.random.default_rng(seed)
    n, bs = 6, [16, 8]
    cost = np.sort(rng.uniform(0, 0.05, n))
    ev = additive_model(cost, bs)
    target = 1.0 - 8 * float(rng.uniform(0, cost.sum()))
    order = list(range(n))
    wb, _ = so.bisection_search(n, order, bs, target, ev)
    wg, _ = so.greedy_search(n, order, bs, target, ev)
    assert ev(wb) >= target and ev(wg) >= target
    # bisection returns the longest feasible prefix of the order
    kb = sum(1 for b in wb if b == 8)
    assert wb == [8] * kb + [16] * (n - kb)
    assert kb >= n - 1 or ev([8] * (kb + 1) + [16] * (n - kb - 1)) < target
    # greedy quantizes at least as many layers as the best prefix, and no feasible single addition remains
    assert sum(b == 8 for b in wg) >= kb
    best = max(sum(b == 8 for b in cfg) for cfg in itertools.product(bs, repeat=n) if ev(list(cfg)) >= target)
    assert sum(b == 8 for b in wg) == best          # cheapest-first greedy is optimal in count for additive costs
