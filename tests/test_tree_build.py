"""Host logic: seq_tree_build / seq_tree_speedup_search (the library's C++ dynamic program) against the oracle's
plain statement of the recursion.  The optimum F and the whole G(n, d) table are unique and must agree to rounding;
the tree itself is only required to be valid, within the bounds, and to score F under the oracle's definition."""
import math
import os

import numpy as np
import pytest

from oracle import tree_dp as D
from paper_2402_12374_b200 import binding as B

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "acceptance_vector_llama3_70b.txt")


def paper_vector():
    rows = [ln for ln in open(GOLDEN) if not ln.startswith("#")]
    return np.array(" ".join(rows).split(), dtype=np.float64)


def test_workload_constant_is_the_papers_vector():
    from paper_2402_12374_b200 import workloads as W

    assert np.array_equal(np.array(W.PAPER_ACCEPTANCE_VECTOR), paper_vector())


def check_tree(parent, P, N, Dd, Bb, F):
    n = len(parent)
    assert 1 <= n <= N and parent[0] == -1 and all(0 <= parent[i] < i for i in range(1, n))
    depth = np.zeros(n, int)
    for i in range(1, n):
        depth[i] = depth[parent[i]] + 1
    assert depth.max() <= Dd
    if n > 1:
        assert np.bincount(parent[1:], minlength=n).max() <= Bb
        assert np.all(np.diff(depth) >= 0) and np.all(np.diff(parent) >= 0)  # level order, siblings contiguous
    assert D.expected_tokens(parent, P) == pytest.approx(F, rel=1e-12)


@pytest.mark.parametrize("N,Dd,Bb", [(1, 0, 1), (1, 5, 3), (2, 1, 1), (16, 6, 8), (64, 10, 8), (100, 12, 31), (30, 2, 5),
                                     (9, 20, 1), (40, 3, 3), (50, 49, 4)])
def test_build_matches_the_oracle_on_the_papers_vector(N, Dd, Bb):
    P = paper_vector()
    parent, F, table = B.seq_tree_build(P, N, Dd, Bb, want_table=True)
    oparent, oF = D.build_tree(P, N, Dd, Bb)
    assert F == pytest.approx(oF, rel=1e-12) and len(parent) == len(oparent)
    check_tree(parent, P, N, Dd, Bb, F)
    _, Tmax, _, _ = D.dp_tables(P, N, Dd, Bb)
    assert table.shape == (N + 1, Dd + 1)
    assert np.array_equal(np.isinf(table[1:]), np.isinf(Tmax[1:])) and np.all(np.isinf(table[0]))
    fin = np.isfinite(Tmax[1:])
    assert np.allclose(table[1:][fin], Tmax[1:][fin], rtol=1e-12, atol=0)


def test_build_with_unsorted_rates_and_an_acceptance_matrix():
    rng = np.random.default_rng(0)
    for trial in range(6):
        N, Dd, Bb = int(rng.integers(2, 40)), int(rng.integers(1, 7)), int(rng.integers(1, 6))
        P = rng.random((Dd, Bb)) if trial % 2 else rng.random(Bb)
        parent, F, table = B.seq_tree_build(P, N, Dd, Bb, want_table=True)
        _, oF = D.build_tree(P, N, Dd, Bb)
        assert F == pytest.approx(oF, rel=1e-12)
        check_tree(parent, P, N, Dd, Bb, F)
        _, Tmax, _, _ = D.dp_tables(P, N, Dd, Bb)
        fin = np.isfinite(Tmax[1:, Dd])
        assert np.array_equal(np.isfinite(table[1:, Dd]), fin)
        assert np.allclose(table[1:, Dd][fin], Tmax[1:, Dd][fin], rtol=1e-12, atol=0)


def test_build_zero_rates_and_full_size():
    # rates of 0: every tree scores 1; still a valid tree of the largest feasible size
    parent, F = B.seq_tree_build(np.zeros(4), 20, 3, 4)
    assert F == 1.0 and len(parent) == 20
    # the largest tree the library handles, at the paper's largest configuration's bounds
    P = paper_vector()
    parent, F = B.seq_tree_build(P, 768, 20, 31)
    assert len(parent) == 768
    check_tree(parent, P, 768, 20, 31, F)
    # more budget and more depth never hurt
    _, F2 = B.seq_tree_build(P, 512, 20, 31)
    _, F3 = B.seq_tree_build(P, 768, 10, 31)
    assert F2 <= F and F3 <= F


def test_build_refuses_bad_arguments():
    P = paper_vector()
    for kw in (dict(max_size=0), dict(max_size=1025), dict(max_depth=-1)):
        args = dict(max_size=16, max_depth=4)
        args.update(kw)
        with pytest.raises(B.SeqTreeError):
            B.seq_tree_build(P, args["max_size"], args["max_depth"], 8)
    bad = P.copy()
    bad[2] = float("nan")
    with pytest.raises(B.SeqTreeError):
        B.seq_tree_build(bad, 16, 4, 8)
    bad[2] = 1.5
    with pytest.raises(B.SeqTreeError):
        B.seq_tree_build(bad, 16, 4, 8)
    with pytest.raises(B.SeqTreeError):  # a matrix needs one row per depth
        B.seq_tree_build(np.tile(P[None], (3, 1)), 16, 4, 8)


def test_speedup_search_matches_the_oracle():
    P = paper_vector()
    N, Dd = 96, 12
    _, _, table = B.seq_tree_build(P, N, Dd, 16, want_table=True)
    rng = np.random.default_rng(1)
    for trial in range(8):
        knee = int(rng.integers(8, 80))
        t = np.ones(N + 1)
        t[knee:] = 1.0 + rng.random() * 0.05 * (np.arange(knee, N + 1) - knee)  # flat, then linear (the shape of t(n))
        c = float(rng.random() * 0.2)
        got = B.seq_tree_speedup_search(table, t, c)
        want = D.speedup_search(table, t, c)
        assert got[:2] == want[:2] and got[2] == pytest.approx(want[2], rel=1e-13)
    # the hand-worked case of the oracle's pin
    _, _, small = B.seq_tree_build([0.5, 0.25], 3, 2, 2, want_table=True)
    assert B.seq_tree_speedup_search(small, [0.0, 1.0, 1.0, 1.5], 0.1)[:2] == (2, 1)
    with pytest.raises(B.SeqTreeError):
        B.seq_tree_speedup_search(small, [0.0, 1.0, 0.0, 1.5], 0.1)
