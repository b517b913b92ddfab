"""Cluster-combination selection and prefix lookup of the prompt-rewriting half of the method
(Sec. 4.2, Algorithm 1), as plain Python.  TEST INFRASTRUCTURE ONLY (part of the CPU oracle).

A training sample is the ordered sequence of clusters it activates (clusters have one fixed order, so
a sample is an increasing tuple of cluster ids).  The cached set C is a set of such sequences; the
coverage of C is, summed over samples, the length of the longest prefix of the sample that is in C.
Algorithm 1 adds, N times, the candidate (a single cluster, or a cached sequence extended by one
cluster) that raises the coverage most.

The paper does not say which candidate wins when several raise the coverage equally: here the shortest
one, and among those the lexicographically smallest.  Candidates are drawn from the prefixes of the
samples, as Algorithm 1 states; a step at which no candidate is left ends the selection early.
"""
from __future__ import annotations


def coverage(samples, cached) -> int:
    """Sum over samples of the number of leading clusters whose KV can be reused: the length of the
    longest prefix of the sample that is in ``cached``."""
    cached = set(tuple(c) for c in cached)
    total = 0
    for s in samples:
        s = tuple(s)
        best = 0
        for n in range(1, len(s) + 1):
            if s[:n] in cached:
                best = n
        total += best
    return total


def select_combinations(samples, budget: int):
    """Algorithm 1.  Returns the list of selected sequences in the order they were added."""
    samples = [tuple(int(c) for c in s) for s in samples]
    prefixes = sorted({s[:n] for s in samples for n in range(1, len(s) + 1)}, key=lambda p: (len(p), p))
    cached, order = set(), []
    for _ in range(int(budget)):
        options = [p for p in prefixes if p not in cached and (len(p) == 1 or p[:-1] in cached)]
        if not options:
            break
        base = coverage(samples, cached)
        best, best_gain = None, -1
        for p in options:                       # options are sorted by (length, value): the first maximum wins
            gain = coverage(samples, cached | {p}) - base
            if gain > best_gain:
                best, best_gain = p, gain
        cached.add(best)
        order.append(best)
    return order


def longest_reusable_prefix(stored, query):
    """Online lookup with tail cut (Sec. 4.2): the stored combination sharing the longest run of
    leading clusters with the query, and that run's length; a stored combination may be longer than
    the run (its mismatched tail is cut off).  Ties go to the first stored combination.  Returns
    (index, length), (-1, 0) when nothing matches."""
    query = tuple(int(c) for c in query)
    best_i, best_n = -1, 0
    for i, comb in enumerate(stored):
        n = 0
        for a, b in zip(comb, query):
            if int(a) != b:
                break
            n += 1
        if n > best_n:
            best_i, best_n = i, n
    return best_i, best_n
