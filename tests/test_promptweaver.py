"""Cluster-combination selection (Algorithm 1) and the online prefix lookup (Sec. 4.2): the oracle against
what the definition fixes, and the library's host code against the oracle.  No GPU needed."""
import itertools
import os

import numpy as np
import pytest

from oracle.promptweaver import coverage, longest_reusable_prefix, select_combinations
from paper_2605_10380_b200 import agx

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "algorithm1_hand_example.txt")


def synthetic_samples(seed, n, clusters=8):
    """Activation sequences with skewed co-activation: a few themes of clusters that fire together, each
    sample activating one theme's leading clusters plus the odd extra one, in the fixed cluster order."""
    rng = np.random.default_rng(seed)
    themes = [[0, 1, 2], [1, 3], [4, 5, 6, 7], [2, 5]]
    out = []
    for _ in range(n):
        t = themes[int(rng.choice(len(themes), p=[0.5, 0.25, 0.15, 0.10]))]
        k = int(rng.integers(1, len(t) + 1))
        s = set(t[:k])
        if rng.random() < 0.2:
            s.add(int(rng.integers(0, clusters)))
        out.append(tuple(sorted(s)))
    return out


def test_hand_worked_example():
    lines = [l for l in open(GOLDEN) if not l.startswith("#")]
    fields = dict(l.strip().split(": ", 1) for l in lines if ": " in l)
    samples = []
    for part in fields["samples"].split(", "):
        cnt, seq = part.split(" x ")
        samples += [tuple(int(c) for c in seq.split("-"))] * int(cnt)
    want = [tuple(int(c) for c in s.split("-")) for s in fields["selected"].split(" | ")]
    cov = [int(v) for v in fields["coverage_after_each_step"].split()]
    got = select_combinations(samples, 4)
    assert got == want
    assert [coverage(samples, got[:k + 1]) for k in range(4)] == cov
    assert agx.pw_select_combinations(samples, 4)[0] == want


def test_coverage_closed_forms():
    samples = [(0, 1, 2), (0, 1), (3,), (0, 2)]
    assert coverage(samples, []) == 0
    assert coverage(samples, [(0,)]) == 3                       # three samples start with cluster 0
    assert coverage(samples, [(0,), (0, 1)]) == 5
    assert coverage(samples, [(0, 1)]) == 4                     # (0,) itself is not cached: only the two 0-1.. samples hit
    every = {s[:n] for s in samples for n in range(1, len(s) + 1)}
    assert coverage(samples, every) == sum(len(s) for s in samples)


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_selection_is_greedy_monotone_and_prefix_closed(seed):
    samples = synthetic_samples(seed, 300)
    order = select_combinations(samples, 15)
    cached, prev = [], 0
    for p in order:
        assert len(p) == 1 or p[:-1] in cached                    # candidates extend what is cached by one cluster
        # brute force: no admissible candidate would have gained more
        prefixes = {s[:n] for s in samples for n in range(1, len(s) + 1)}
        options = [c for c in prefixes if c not in cached and (len(c) == 1 or c[:-1] in cached)]
        gains = {c: coverage(samples, cached + [c]) - prev for c in options}
        assert gains[p] == max(gains.values())
        cached.append(p)
        cov = coverage(samples, cached)
        assert cov >= prev                                          # coverage never decreases with the budget
        prev = cov
    assert coverage(samples, select_combinations(samples, 10 ** 6)) == sum(len(s) for s in samples)


def test_greedy_is_optimal_on_tiny_instances_with_at_most_two_picks():
    """For budgets 1 and 2 the greedy choice is optimal among prefix-closed sets (checked by brute force)."""
    samples = synthetic_samples(9, 40, clusters=5)
    prefixes = sorted({s[:n] for s in samples for n in range(1, len(s) + 1)})
    for budget in (1, 2):
        best = 0
        for comb in itertools.combinations(prefixes, budget):
            if all(len(p) == 1 or p[:-1] in comb for p in comb):
                best = max(best, coverage(samples, comb))
        assert coverage(samples, select_combinations(samples, budget)) == best


@pytest.mark.parametrize("seed,n,budget", [(4, 0, 5), (5, 1, 3), (6, 50, 0), (7, 500, 15), (8, 3000, 40), (9, 200, 1000)])
def test_library_selection_matches_oracle(seed, n, budget):
    samples = synthetic_samples(seed, n)
    want = select_combinations(samples, budget)
    got, gains = agx.pw_select_combinations(samples, budget)
    assert got == want
    cov = [coverage(samples, want[:k]) for k in range(len(want) + 1)]
    assert gains == [cov[k + 1] - cov[k] for k in range(len(want))]


def test_longest_prefix_lookup_with_tail_cut():
    stored = [(0,), (0, 1, 2), (0, 1, 3, 5), (4, 5)]
    cases = [((0, 1, 3), (2, 3)), ((0, 1, 4), (1, 2)), ((0, 1, 2, 3), (1, 3)), ((4,), (3, 1)), ((7, 0), (-1, 0)),
             ((), (-1, 0)), ((0,), (0, 1)), ((0, 1, 3, 5, 6), (2, 4))]
    for query, want in cases:
        assert longest_reusable_prefix(stored, query) == want
        assert agx.pw_longest_prefix(stored, query) == want
    assert agx.pw_longest_prefix([], (1, 2)) == (-1, 0)
    rng = np.random.default_rng(3)
    samples = synthetic_samples(11, 400)
    stored = select_combinations(samples, 15)
    for _ in range(200):
        q = samples[int(rng.integers(0, len(samples)))]
        assert agx.pw_longest_prefix(stored, q) == longest_reusable_prefix(stored, q)
