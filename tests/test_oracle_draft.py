"""Pins of the oracle's draft-side sampling without replacement (exponential sort), none of which retypes its
formula: the exact law of ordered draws without replacement (Monte-Carlo), the two degenerate cases that are a
library sort, temperature as a rescaling of the logits, and invariants."""
import numpy as np
import pytest

from oracle import oracle as O


def test_ordered_pairs_follow_the_without_replacement_law():
    """P(first = i, second = j) = q_i q_j / (1 - q_i): the definition of sampling twice without replacement."""
    rng = np.random.default_rng(0)
    logits = np.array([0.3, -1.0, 1.2, 0.0, -0.4], np.float32)
    T = 0.7
    q = np.exp(logits / T - (logits / T).max())
    q /= q.sum()
    N = 60000
    counts = np.zeros((5, 5))
    for _ in range(N):
        t = O.draft_sample(logits, T, rng.random(5).astype(np.float32), 2)["tokens"]
        counts[t[0], t[1]] += 1
    expect = np.outer(q, q) / (1.0 - q)[:, None]
    np.fill_diagonal(expect, 0.0)
    assert np.trace(counts) == 0
    # every cell within 5 standard deviations of its binomial expectation
    sd = np.sqrt(N * expect * (1 - expect))
    assert (np.abs(counts - N * expect) <= 5 * sd + 1).all(), (counts / N, expect)
    # first draws alone: plain sampling from q
    first = counts.sum(axis=1)
    assert (np.abs(first - N * q) <= 5 * np.sqrt(N * q * (1 - q))).all()


def test_degenerate_cases_are_library_sorts():
    rng = np.random.default_rng(1)
    V = 300
    logits = rng.standard_normal(V).astype(np.float32)
    u = rng.random(V).astype(np.float32)
    # all uniforms equal: the order is that of decreasing probability, i.e. of decreasing logit
    same = np.full(V, 0.37, np.float32)
    got = O.draft_sample(logits, 0.9, same, V)["tokens"]
    assert got.tolist() == np.argsort(-logits.astype(np.float64), kind="stable").tolist()
    # all logits equal: the order is that of increasing exponential variate, i.e. of decreasing uniform
    flat = np.zeros(V, np.float32)
    got = O.draft_sample(flat, 1.3, u, V)["tokens"]
    assert got.tolist() == np.argsort(-u.astype(np.float64), kind="stable").tolist()


def test_temperature_is_a_rescaling_of_the_logits():
    rng = np.random.default_rng(2)
    V = 200
    logits = (3 * rng.standard_normal(V)).astype(np.float32)
    u = rng.random(V).astype(np.float32)
    # a power of two, so that logits / T is exact in fp32 and both calls see the same numbers
    a = O.draft_sample(logits, 0.5, u, 16)["tokens"]
    b = O.draft_sample((logits / np.float32(0.5)).astype(np.float32), 1.0, u, 16)["tokens"]
    assert a.tolist() == b.tolist()


def test_invariants_distinct_support_and_exhaustion():
    rng = np.random.default_rng(3)
    V = 64
    logits = rng.standard_normal(V).astype(np.float32)
    logits[rng.choice(V, 50, replace=False)] = -np.inf  # 14 tokens keep mass
    u = rng.random(V).astype(np.float32)
    r = O.draft_sample(logits, 1.0, u, 20)
    tok = r["tokens"]
    live = tok[tok >= 0]
    assert len(live) == 14 and len(set(live.tolist())) == 14 and (tok[14:] == -1).all()
    assert np.isfinite(logits[live]).all()
    keys = r["keys"]
    assert np.isinf(keys[~np.isfinite(logits)]).all()
    assert (np.diff(keys[live]) >= 0).all()  # draw order = ascending key order
    # a prefix of a longer draw is the shorter draw
    assert O.draft_sample(logits, 1.0, u, 5)["tokens"].tolist() == tok[:5].tolist()
    # uniforms outside (0, 1) give a token no chance
    u2 = u.copy()
    u2[live[0]] = 0.0
    u2[live[1]] = 1.0
    tok2 = O.draft_sample(logits, 1.0, u2, 20)["tokens"]
    assert live[0] not in tok2 and live[1] not in tok2 and (tok2 >= 0).sum() == 12


def test_min_rel_gap_reports_the_closest_neighbours():
    logits = np.zeros(4, np.float32)
    u = np.exp(-np.array([1.0, 2.0, 2.0002, 4.0])).astype(np.float32)  # keys 4, 8, 8.0008, 16 (q = 1/4)
    r = O.draft_sample(logits, 1.0, u, 2)
    assert r["tokens"].tolist() == [0, 1]
    assert 5e-5 < r["min_rel_gap"] < 2e-4   # between the second draw and the first token left out
