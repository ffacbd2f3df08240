"""Tree construction by dynamic programming -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

A plain, slow statement of Sequoia's tree construction (Section 3.1: the score function, the proposition
F(tree) = sum of the nodes' scores, the recursion of Algorithm 1; Appendix "Dynamic programming details" for
the two extensions: a bound on the depth and an acceptance-rate matrix with one row per depth) and of the
hardware-aware choice of the tree's size and depth (Section 4.1, Speedup(n, d) = G(n, d) / (t(n) + d c)).

Notation as in the paper: P[b] is the probability that the b-th child (b = 1 .. B) of a node is accepted, given
that the node was reached and its earlier children were rejected ("positional acceptance"); the score f(v) of a
node is the product of the P's along its path; F(tree) is the expected number of generated tokens.  Depth is
counted in edges here (the root alone has depth 0).  Nothing is blocked or vectorised: the loops are the
recursion.  It shares no code with the CUDA library; only tests, the smoke check and the benchmark's
cpu_baseline leg may import it.

Pins (tests marked "not gpu"): enumeration of every ordered tree of up to 7 nodes; for non-increasing acceptance
vectors the optimum is the n best-scored nodes of the infinite tree (best-first search on a library heap);
closed forms for chains and stars; the reconstructed tree re-scored by the proposition; a hand-worked
speedup search.
"""
from __future__ import annotations

import math

import numpy as np

NEG = -math.inf


def _rates(P, D: int, B: int) -> np.ndarray:
    """Acceptance rates as a [max(D,1)][B+1] fp64 matrix, column 0 unused; row = depth of the parent."""
    P = np.asarray(P, dtype=np.float64)
    if P.ndim == 1:
        P = np.tile(P[None, :], (max(D, 1), 1))
    assert P.shape[0] >= max(D, 1) and P.shape[1] >= B, "one row per parent depth, one column per child rank"
    out = np.zeros((max(D, 1), B + 1))
    out[:, 1:] = P[: max(D, 1), :B]
    return out


def expected_tokens(parent, P) -> float:
    """F(tree) = sum over nodes of f(v), f(v) = product over the path of P[depth of the parent][rank of the
    child], f(root) = 1 (the proposition of Section 3.1).  A child's rank is its position among its siblings in
    ascending node order."""
    parent = np.asarray(parent)
    n = len(parent)
    depth = np.zeros(n, dtype=np.int64)
    rank = np.zeros(n, dtype=np.int64)
    seen = np.zeros(n, dtype=np.int64)
    for i in range(1, n):
        p = int(parent[i])
        assert 0 <= p < i
        depth[i] = depth[p] + 1
        seen[p] += 1
        rank[i] = seen[p]
    R = _rates(P, int(depth.max()) if n > 1 else 0, int(rank.max()) if n > 1 else 1)
    f = np.ones(n)
    for i in range(1, n):
        f[i] = f[int(parent[i])] * R[depth[i] - 1, rank[i]]
    return float(f.sum())


def dp_tables(P, N: int, D: int, B: int):
    """T[n][d][b] = the largest F over trees of exactly n nodes, depth <= d, whose root has exactly b children and
    in which no node has more than B; Tmax[n][d] = max over b (= G(n, d)); -inf where no such tree exists.  With
    an acceptance matrix, a tree "of depth <= d" here hangs below a node at depth D - d of the final tree, so its
    root's children use row D - d.  Also returns the arg-max bookkeeping needed to rebuild a best tree."""
    R = _rates(P, D, B)
    T = np.full((N + 1, D + 1, B + 1), NEG)
    Tmax = np.full((N + 1, D + 1), NEG)
    arg_m = np.zeros((N + 1, D + 1, B + 1), dtype=np.int64)   # size of the last child's subtree
    arg_b = np.zeros((N + 1, D + 1), dtype=np.int64)          # best number of root children
    T[1, :, 0] = 1.0          # the root alone: one token per step even when nothing is speculated
    Tmax[1, :] = 1.0
    for n in range(2, N + 1):
        for d in range(1, D + 1):
            row = R[D - d]
            for b in range(1, B + 1):
                best, best_m = NEG, 0
                for m in range(1, n):  # m nodes in the subtree of the b-th child, the rest in "tree #1"
                    left, sub = T[n - m, d, b - 1], Tmax[m, d - 1]
                    if left == NEG or sub == NEG:
                        continue
                    val = left + row[b] * sub
                    if val > best:
                        best, best_m = val, m
                T[n, d, b], arg_m[n, d, b] = best, best_m
            b_star = int(np.argmax(T[n, d]))
            Tmax[n, d], arg_b[n, d] = T[n, d, b_star], b_star
    return T, Tmax, arg_m, arg_b


def build_tree(P, N: int, D: int, B: int):
    """A best tree for the budget: at most N nodes, depth <= D, at most B children per node.  Returns the parent
    array in level order (siblings contiguous, in rank order), and its F.  Several trees can share the optimum;
    only F is unique."""
    T, Tmax, arg_m, arg_b = dp_tables(P, N, D, B)
    n_best = max((n for n in range(1, N + 1) if Tmax[n, D] > NEG), key=lambda n: (Tmax[n, D], n))

    def children_sizes(n, d):
        sizes = []
        b = int(arg_b[n, d])
        while b > 0:
            m = int(arg_m[n, d, b])
            sizes.append(m)
            n -= m
            b -= 1
        assert n == 1
        return sizes[::-1]

    parent = [-1]
    level = [(0, n_best, D)]  # (node id, nodes in its subtree, depth still allowed below it)
    while level:
        nxt = []
        for node, n, d in level:
            if n == 1:
                continue
            for m in children_sizes(n, d):
                parent.append(node)
                nxt.append((len(parent) - 1, m, d - 1))
        level = nxt
    return np.array(parent, dtype=np.int32), float(Tmax[n_best, D])


def speedup_search(G, t, c: float):
    """Speedup(n, d) = G(n, d) / (t(n) + d c) maximised over 1 <= n <= N, 0 <= d <= D (Section 4.1,
    "Hardware-Aware Optimization"); G: [N+1][D+1] with -inf where no tree exists, t: [N+1] relative verify
    times.  Returns (n, d, speedup); ties go to the smaller n, then the smaller d."""
    G, t = np.asarray(G, dtype=np.float64), np.asarray(t, dtype=np.float64)
    best = (0, 0, NEG)
    for n in range(1, G.shape[0]):
        for d in range(G.shape[1]):
            if G[n, d] == NEG:
                continue
            s = G[n, d] / (t[n] + d * c)
            if s > best[2]:
                best = (n, d, s)
    return best
