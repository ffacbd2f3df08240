"""Pins of the oracle's tree construction (``oracle/tree_dp.py``): exhaustive enumeration of small ordered trees,
the best-first characterisation of the optimum for non-increasing acceptance vectors, closed forms, the
proposition F = sum of scores applied to the rebuilt tree, and the hardware-aware search on a hand-worked case."""
import heapq
import math
import os

import numpy as np
import pytest

from oracle import tree_dp as D

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "acceptance_vector_llama3_70b.txt")


def paper_vector():
    rows = [ln for ln in open(GOLDEN) if not ln.startswith("#")]
    return np.array(" ".join(rows).split(), dtype=np.float64)


def all_ordered_trees(n):
    """Every ordered rooted tree with n nodes as a nested tuple of children (Catalan(n-1) of them)."""
    if n == 1:
        return [()]
    out = []

    def forests(k):  # ordered forests with k nodes in total
        if k == 0:
            return [()]
        res = []
        for first in range(1, k + 1):
            for t in all_ordered_trees(first):
                for rest in forests(k - first):
                    res.append((t,) + rest)
        return res

    return forests(n - 1)


def score_nested(tree, R, depth=0, f=1.0):
    """F by the definition, on the nested form: a node's score is its parent's times P[parent depth][rank]."""
    total = f
    for rank, child in enumerate(tree, start=1):
        total += score_nested(child, R, depth + 1, f * R[depth][rank - 1])
    return total


def depth_nested(tree):
    return 0 if not tree else 1 + max(depth_nested(c) for c in tree)


def max_branch_nested(tree):
    return max([len(tree)] + [max_branch_nested(c) for c in tree])


@pytest.mark.parametrize("kind", ["sorted", "unsorted", "matrix"])
def test_dp_equals_enumeration_of_all_small_trees(kind):
    rng = np.random.default_rng({"sorted": 0, "unsorted": 1, "matrix": 2}[kind])
    Bmax, Dmax, N = 4, 4, 7
    for trial in range(4):
        if kind == "matrix":
            P = rng.random((Dmax, Bmax)) * 0.9
        else:
            P = rng.random(Bmax) * 0.9
            if kind == "sorted":
                P = np.sort(P)[::-1]
        R = np.tile(P[None], (Dmax, 1)) if P.ndim == 1 else P
        trees = {n: all_ordered_trees(n) for n in range(1, N + 1)}
        for Dd in (1, 2, 4):
            for B in (1, 2, 4):
                _, Tmax, _, _ = D.dp_tables(P, N, Dd, B)
                for n in range(1, N + 1):
                    feasible = [t for t in trees[n] if depth_nested(t) <= Dd and max_branch_nested(t) <= B]
                    want = max((score_nested(t, R) for t in feasible), default=-math.inf)
                    assert Tmax[n, Dd] == pytest.approx(want, rel=1e-13, abs=0) or (Tmax[n, Dd] == want == -math.inf)


def best_first_value(P, N, Dd, B):
    """Sum of the N largest scores among the nodes of the full B-ary tree of depth Dd: for a non-increasing P
    every prefix of that order is a valid tree (a node's parent and earlier siblings score at least as much), so
    this is the optimum.  A different algorithm from the recursion: a heap instead of a table."""
    heap = [(-1.0, 0, 0)]  # (-score, depth, tiebreak)
    total, taken, tick = 0.0, 0, 0
    # lazily generated: popping a node pushes its first child and its next sibling
    items = {0: (1.0, 0, None, 0)}  # id -> (score, depth, parent score, rank)
    while heap and taken < N:
        neg, depth, ident = heapq.heappop(heap)
        score, depth, pscore, rank = items.pop(ident)
        total += score
        taken += 1
        if depth < Dd:
            tick += 1
            items[tick] = (score * P[0], depth + 1, score, 1)
            heapq.heappush(heap, (-score * P[0], depth + 1, tick))
        if pscore is not None and rank < B:
            tick += 1
            items[tick] = (pscore * P[rank], depth, pscore, rank + 1)
            heapq.heappush(heap, (-pscore * P[rank], depth, tick))
    return total, taken


@pytest.mark.parametrize("N,Dd,B", [(64, 10, 8), (128, 6, 31), (120, 119, 31), (40, 3, 3)])
def test_dp_equals_the_n_best_scores_for_the_papers_vector(N, Dd, B):
    P = paper_vector()
    assert len(P) == 31 and np.all(np.diff(P[:15]) <= 0)
    P = np.sort(P)[::-1]  # the printed tail is not monotone in the 4th decimal; the characterisation needs order
    _, Tmax, _, _ = D.dp_tables(P, N, Dd, B)
    want, taken = best_first_value(P, N, Dd, B)
    n_feasible = max(n for n in range(1, N + 1) if Tmax[n, Dd] > -math.inf)
    assert taken == n_feasible
    assert Tmax[n_feasible, Dd] == pytest.approx(want, rel=1e-12)


def test_closed_forms_chain_and_star():
    P = np.array([0.8, 0.1, 0.05, 0.02])
    # B = 1: the only tree is a chain, F = 1 + p + p^2 + ... ; bounded by 1/(1 - p) (Section 3.1's remark)
    _, Tmax, _, _ = D.dp_tables(P, 12, 11, 1)
    for n in range(1, 13):
        assert Tmax[n, 11] == pytest.approx((1 - 0.8 ** n) / (1 - 0.8), rel=1e-13)
        assert Tmax[n, 11] < 1 / (1 - 0.8)
    # depth 1: a star, F = 1 + P[1] + ... + P[n-1]; more nodes than B + 1 do not fit
    _, Tmax, _, _ = D.dp_tables(P, 8, 1, 4)
    for n in range(1, 6):
        assert Tmax[n, 1] == pytest.approx(1 + P[: n - 1].sum(), rel=1e-13)
    assert all(Tmax[n, 1] == -math.inf for n in (6, 7, 8))
    # depth 0: the root alone
    _, Tmax, _, _ = D.dp_tables(P, 3, 0, 4)
    assert Tmax[1, 0] == 1.0 and Tmax[2, 0] == -math.inf


def test_expected_tokens_is_the_sum_of_path_products():
    """A hand-worked tree: root with children a, b; a with child c.  F = 1 + p1 + p2 + p1*p1 for a vector, and with
    a matrix the grandchild uses the second row."""
    parent = [-1, 0, 0, 1]
    assert D.expected_tokens(parent, [0.5, 0.25]) == pytest.approx(1 + 0.5 + 0.25 + 0.25)
    assert D.expected_tokens(parent, [[0.5, 0.25], [0.1, 0.9]]) == pytest.approx(1 + 0.5 + 0.25 + 0.5 * 0.1)
    assert D.expected_tokens([-1], [0.3]) == 1.0


@pytest.mark.parametrize("N,Dd,B", [(16, 6, 8), (64, 10, 8), (128, 12, 31), (30, 2, 5), (9, 20, 1)])
def test_rebuilt_tree_is_valid_and_scores_the_optimum(N, Dd, B):
    P = paper_vector()
    parent, value = D.build_tree(P, N, Dd, B)
    n = len(parent)
    feasible_max = min(N, sum(B ** k for k in range(Dd + 1)))
    assert n == feasible_max and parent[0] == -1 and all(0 <= parent[i] < i for i in range(1, n))
    depth = np.zeros(n, int)
    for i in range(1, n):
        depth[i] = depth[parent[i]] + 1
    assert depth.max() <= Dd and np.bincount(parent[1:], minlength=n).max() <= B
    assert np.all(np.diff(depth) >= 0) and np.all(np.diff(parent) >= 0)  # level order, siblings contiguous
    assert D.expected_tokens(parent, P) == pytest.approx(value, rel=1e-12)
    _, Tmax, _, _ = D.dp_tables(P, N, Dd, B)
    assert value == Tmax[n, Dd]


def test_value_grows_with_budget_and_depth_and_beats_independent_chains():
    P = paper_vector()
    _, Tmax, _, _ = D.dp_tables(P, 96, 12, 16)
    G = Tmax[1:, 12]
    assert np.all(np.diff(G) >= 0)
    assert np.all(np.diff(Tmax[64, 1:]) >= -1e-15)
    # k independent sequences (a root whose k children each start a chain) are one of the trees the recursion
    # searches over, so the optimum is at least as good; a single chain is bounded by 1/(1-P1) and the tree is not
    k, L = 4, 16
    parent = [-1]
    for j in range(k):
        parent.append(0)
    heads = list(range(1, k + 1))
    for step in range(L - 1):
        for j in range(k):
            parent.append(heads[j])
            heads[j] = len(parent) - 1
    n = len(parent)
    assert n == 1 + k * L
    _, T2, _, _ = D.dp_tables(P, n, L, 16)
    assert T2[n, L] >= D.expected_tokens(parent, P) - 1e-12
    assert T2[n, L] > 1 / (1 - P[0]) - 1e-9 or n < 30


def test_speedup_search_hand_worked():
    """G(n, d) for n <= 3, d <= 2 with P = [0.5, 0.25]; t(n) = 1, 1, 1.5; c = 0.1.
    G(1, .) = 1; G(2, d >= 1) = 1.5; G(3, 1) = 1.75 (star); G(3, 2) = max(1.75, 1 + .5 + .25) = 1.75.
    Speedups: (1,0): 1; (2,1): 1.5/1.1 = 1.3636; (2,2): 1.5/1.2; (3,1): 1.75/1.6; (3,2): 1.75/1.7 -> (2, 1)."""
    _, Tmax, _, _ = D.dp_tables([0.5, 0.25], 3, 2, 2)
    assert Tmax[1].tolist() == [1.0, 1.0, 1.0]
    assert Tmax[2].tolist() == [-math.inf, 1.5, 1.5] and Tmax[3].tolist() == [-math.inf, 1.75, 1.75]
    n, d, s = D.speedup_search(Tmax, [0.0, 1.0, 1.0, 1.5], 0.1)
    assert (n, d) == (2, 1) and s == pytest.approx(1.5 / 1.1)
    # a cheaper drafter and a flat t(n) move the optimum to the larger tree
    n, d, s = D.speedup_search(Tmax, [0.0, 1.0, 1.0, 1.0], 0.01)
    assert (n, d) == (3, 1) and s == pytest.approx(1.75 / 1.01)
