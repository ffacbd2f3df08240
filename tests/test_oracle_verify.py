"""Pins of the oracle's Algorithm 2 walk against what the paper and the mathematics fix:
exact enumeration of the output distribution (must equal P), the paper's printed example,
the optimal-transport and cover properties, the rejection lemma, reductions to Algorithm 3,
to plain sampling and to arg-max matching, invariants, and Monte-Carlo."""
import ctypes as C
import json
import os

import numpy as np
import pytest

from oracle import oracle as O
from paper_2402_12374_b200 import workloads as W

GOLDEN = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_examples.json")))
REJECT = 1.0  # a "uniform" that rejects whenever ratio <= 1 (enumeration never recurses when ratio >= 1)


def enumerate_alg2(P, Q, k, variant=O.VARIANT_SEQUOIA):
    """Exact output distribution of Algorithm 2 with k speculated children.

    Every quantity comes from the oracle's own state: child i is drawn from the oracle's current
    D, accepted with probability min(1, ratio) where ratio is the one the oracle tested, and on k
    rejections the token comes from the oracle's final R.  Returns (distribution, P(all rejected))."""
    P, Q = np.asarray(P, float), np.asarray(Q, float)
    V = len(P)
    out = np.zeros(V)
    rejected_mass = [0.0]

    def rec(prefix, reach):
        st = O.alg2_node(P, Q, prefix, [REJECT] * len(prefix), variant)
        assert st["accepted"] == -1
        if len(prefix) == k or st["D"].sum() == 0.0:
            out[:] += reach * st["R"]
            rejected_mass[0] += reach
            return
        for s in range(V):
            ds = st["D"][s]
            if ds == 0.0:
                continue
            ratio = O.alg2_node(P, Q, prefix + [s], [REJECT] * (len(prefix) + 1), variant)["ratio"][-1]
            a = min(1.0, ratio)
            out[s] += reach * ds * a
            if a < 1.0:
                rec(prefix + [s], reach * ds * (1.0 - a))

    rec([], 1.0)
    return out, rejected_mass[0]


def _rand_dist(rng, V, zeros=0):
    p = rng.random(V) + 0.05
    if zeros:
        p[rng.choice(V, zeros, replace=False)] = 0.0
    return p / p.sum()


def test_paper_printed_cover_counterexample():
    g = GOLDEN["cover_counterexample"]
    _, rej_seq = enumerate_alg2(g["P"], g["Q"], g["k"], O.VARIANT_SEQUOIA)
    out_si, rej_si = enumerate_alg2(g["P"], g["Q"], g["k"], O.VARIANT_SPECINFER)
    assert abs((1.0 - rej_seq) - g["sequoia_acceptance"]) < 1e-15
    assert abs(rej_si - g["specinfer_all_rejected_probability"]) < 1e-15
    np.testing.assert_allclose(out_si, g["P"], atol=1e-15)  # SpecInfer still preserves the target


@pytest.mark.parametrize("variant", [O.VARIANT_SEQUOIA, O.VARIANT_SPECINFER])
def test_output_distribution_equals_target_by_exact_enumeration(variant):
    rng = np.random.default_rng(10)
    cases = 0
    for V in (2, 3, 4, 5):
        for k in range(0, V + 1 if variant == O.VARIANT_SEQUOIA else 4):
            for zp, zq in ((0, 0), (1, 0), (0, 1), (V - 1, 0), (0, V - 1), (1, 1)):
                if zp >= V or zq >= V:
                    continue
                P, Q = _rand_dist(rng, V, zp), _rand_dist(rng, V, zq)
                out, _ = enumerate_alg2(P, Q, k, variant)
                np.testing.assert_allclose(out, P, atol=1e-12, err_msg=f"V={V} k={k} P={P} Q={Q}")
                cases += 1
    assert cases > 50


def test_optimal_transport_property_k1():
    rng = np.random.default_rng(11)
    for V in (2, 5, 9):
        P, Q = _rand_dist(rng, V, 1), _rand_dist(rng, V)
        _, rej = enumerate_alg2(P, Q, GOLDEN["optimal_transport"]["k"])
        assert abs((1.0 - rej) - (1.0 - 0.5 * np.abs(P - Q).sum())) < 1e-13


def test_cover_property():
    rng = np.random.default_rng(12)
    V = 5
    for k in (2, 3, 4):
        Q = np.zeros(V)
        supp = rng.choice(V, k, replace=False)
        Q[supp] = _rand_dist(rng, k)
        P = np.zeros(V)
        P[supp[: max(1, k - 1)]] = _rand_dist(rng, max(1, k - 1))
        assert enumerate_alg2(P, Q, k)[1] < 1e-14
        if k > 2:  # one speculation fewer can still fail
            assert enumerate_alg2(P, Q, 1)[1] > 1e-3
    # k = vocabulary size: always accepted, whatever the draft (uniform fallback included)
    P, Q = _rand_dist(rng, V), np.array([0.7, 0.3, 0, 0, 0])
    assert enumerate_alg2(P, Q, V)[1] < 1e-14


def test_rejection_lemma_and_residual_definition():
    """P(no accept at the first iteration) = sum max(0, P-Q); the next residual is norm(max(P-Q,0))."""
    rng = np.random.default_rng(13)
    P, Q = _rand_dist(rng, 6), _rand_dist(rng, 6)
    _, rej = enumerate_alg2(P, Q, 1)
    assert abs(rej - np.maximum(P - Q, 0).sum()) < 1e-14
    s = int(np.argmax(Q - P))  # a token that can be rejected
    st = O.alg2_node(P, Q, [s], [REJECT])
    np.testing.assert_allclose(st["R"], np.maximum(P - Q, 0) / np.maximum(P - Q, 0).sum(), atol=1e-15)
    expect_D = Q.copy()
    expect_D[s] = 0
    np.testing.assert_allclose(st["D"], expect_D / expect_D.sum(), atol=1e-15)


def test_inverse_cdf_when_the_cumulative_sum_never_exceeds_the_uniform():
    """x ~ R by inverse CDF (Algorithm 2's last line, reading: first index whose inclusive sum exceeds u, else
    the LAST index with R > 0).  The second branch by hand: trailing zeros must not be returned, nor -1, nor V-1."""
    assert O.sample_inverse_cdf([0.5, 0.5, 0.0, 0.0], 1.0) == 1          # total == u, two trailing zeros
    assert O.sample_inverse_cdf([0.0, 0.3, 0.0], 0.9) == 1               # total well below u, zeros on both sides
    assert O.sample_inverse_cdf([0.25, 0.0, 0.25, 0.25, 0.0], 0.75) == 3  # c == u is not "exceeds"
    assert O.sample_inverse_cdf([1.0], 1.0) == 0
    assert O.sample_inverse_cdf([0.0, 0.0], 0.5) == -1                   # no mass at all: nothing to return
    # a total that rounding left below 1 (ten times 0.1 sums to 0.9999999999999999) and u just above it
    R = [0.1] * 10 + [0.0, 0.0]
    c = 0.0
    for x in R:  # the sequential sum (Python's built-in sum compensates)
        c += x
    assert c < 1.0 and O.sample_inverse_cdf(R, float(np.nextafter(c, 2.0))) == 9 and O.sample_inverse_cdf(R, c) == 9
    # and the first branch for contrast: strict crossing, zeros are never chosen
    assert O.sample_inverse_cdf([0.5, 0.0, 0.5], 0.5) == 2
    assert O.sample_inverse_cdf([0.5, 0.0, 0.5], 0.4999) == 0
    # the whole walk reaches that branch too: a single node whose uniform is 1 (outside [0,1), legal for the oracle)
    tl = np.log(np.array([[0.5, 0.5, 1e-300, 1e-300]])).astype(np.float32)
    tl[0, 2:] = -np.inf
    r = O.tree_verify(np.array([-1], np.int32), np.array([0], np.int32), tl, tl, 1.0, np.array([0.0, 1.0], np.float32))
    assert r["bonus"] == 1 and r["path"].tolist() == [0]


def test_hand_checked_three_token_example():
    P, Q = [0.5, 0.3, 0.2], [0.2, 0.5, 0.3]
    st = O.alg2_node(P, Q, [1, 2], [0.7, 0.1])
    assert st["accepted"] == -1
    np.testing.assert_allclose(st["ratio"], [0.6, 0.0], atol=1e-15)
    np.testing.assert_allclose(st["R"], [1, 0, 0], atol=1e-15)
    assert O.sample_inverse_cdf(st["R"], 0.999) == 0
    assert O.alg2_node(P, Q, [1, 2], [0.5, 0.1])["accepted"] == 0
    assert O.alg2_node(P, Q, [1, 2], [0.6, 0.1])["accepted"] == -1  # strict '<'


def test_uniform_fallback_and_duplicates():
    P, Q = np.array([0.1, 0.2, 0.3, 0.4]), np.array([1.0, 0, 0, 0])
    st = O.alg2_node(P, Q, [0], [REJECT])  # the only draft token is rejected -> D uniform over the rest
    np.testing.assert_allclose(st["D"], [0, 1 / 3, 1 / 3, 1 / 3], atol=1e-15)
    np.testing.assert_allclose(st["R"], [0, 0.2 / 0.9, 0.3 / 0.9, 0.4 / 0.9], atol=1e-15)
    st = O.alg2_node(P, Q, [0, 2], [REJECT, 0.99])  # R[2]/D[2] = 1 -> accepted
    assert st["accepted"] == 1 and abs(st["ratio"][1] - 1.0) < 1e-15
    # a duplicate of a rejected sibling has R = D = 0 there: ratio 0, rejected, S does not grow
    st = O.alg2_node(P, Q, [0, 0, 1], [REJECT, 0.0, REJECT])
    assert st["accepted"] == -1 and st["ratio"][1] == 0.0 and st["ratio"][2] == 0.0
    np.testing.assert_allclose(st["R"], [0, 0, 0, 1], atol=1e-15)
    np.testing.assert_allclose(st["D"], [0, 0, 0.5, 0.5], atol=1e-15)  # |S| = 2 although three were rejected
    # token out of range: flagged, nothing else changes
    a = O.alg2_node(P, Q, [7, 0], [0.0, REJECT])
    b = O.alg2_node(P, Q, [0], [REJECT])
    assert a["flags"] & O.BAD_TOKEN and np.array_equal(a["R"], b["R"]) and np.array_equal(a["D"], b["D"])


def _alg3_textbook(p, q, x, r, u_final):
    """Sequence speculative sampling as in the textbook statement (Algorithm 3)."""
    s = 0
    for i in range(len(x)):
        if r[i] < p[i, x[i]] / q[i, x[i]]:
            s += 1
        else:
            break
    dist = p[s].copy()
    if s < len(x):
        dist = np.maximum(p[s] - q[s], 0)
        dist /= dist.sum()
    return s, int(np.searchsorted(np.cumsum(dist), u_final, side="right"))


def _softmax64(x, T):
    z = np.asarray(x, np.float64) / T
    e = np.exp(z - z.max(-1, keepdims=True))
    return e / e.sum(-1, keepdims=True)


@pytest.mark.parametrize("T", [1.0, 0.6])
def test_chain_tree_reduces_to_algorithm3(T):
    rng = np.random.default_rng(14)
    V, n = 50, 7
    hits = set()
    for trial in range(60):
        tl = (2 * rng.standard_normal((n, V))).astype(np.float32)
        dl = (tl + rng.standard_normal((n, V))).astype(np.float32)
        parent = W.chain_tree(n)
        tokens = W.draw_children_tokens(parent, dl, T, rng)
        u = rng.random(n + 1, dtype=np.float32)
        res = O.tree_verify(parent, tokens, tl, dl, T, u)
        p, q = _softmax64(tl, T), _softmax64(dl[: n - 1], T)
        s, t = _alg3_textbook(p, q, tokens[1:], u[1:n].astype(np.float64), float(u[n]))
        assert res["path_len"] == s + 1 and list(res["path"]) == list(range(s + 1))
        assert res["bonus"] == t
        s2, t2 = O.alg3_chain(p, q, tokens[1:], u[1:n].astype(np.float64), float(u[n]))
        assert (s2, t2) == (s, t)
        hits.add(s)
    assert len(hits) >= 3  # several different accepted lengths were exercised


def test_single_node_tree_samples_from_target():
    rng = np.random.default_rng(15)
    V = 300
    tl = (3 * rng.standard_normal((1, V))).astype(np.float32)
    for T in (1.0, 0.6, 0.2):
        cdf = np.cumsum(_softmax64(tl[0], T))
        for u in rng.random(20, dtype=np.float32):
            res = O.tree_verify([-1], [0], tl, tl, T, np.array([0.0, u], np.float32))
            assert res["path_len"] == 1 and res["bonus"] == int(np.searchsorted(cdf, float(u), side="right"))
            np.testing.assert_allclose(res["residual"], _softmax64(tl[0], T), atol=1e-15)


def test_draft_equals_target_follows_first_children_to_a_leaf():
    rng = np.random.default_rng(16)
    n, V = 30, 40
    parent = W.random_tree(n, None, 4, rng)
    tl = rng.standard_normal((n, V)).astype(np.float32)
    tokens = W.draw_children_tokens(parent, tl, 0.8, rng)
    res = O.tree_verify(parent, tokens, tl, tl, 0.8, rng.random(n + 1, dtype=np.float32))
    kids = W.children_lists(parent)
    cur, expect = 0, [0]
    while kids[cur]:
        cur = kids[cur][0]
        expect.append(cur)
    assert list(res["path"]) == expect and abs(res["min_gap"]) > 0


def test_greedy_and_its_low_temperature_limit():
    rng = np.random.default_rng(17)
    n, V = 40, 64
    agree = 0
    for trial in range(30):
        parent = W.random_tree(n, None, 4, rng)
        tl = np.round(3 * rng.standard_normal((n, V)), 1).astype(np.float32)
        tl[np.arange(n), rng.integers(0, V, n)] += 20.0  # unique arg-max with a wide gap
        dl = (tl + rng.standard_normal((n, V))).astype(np.float32)
        tokens = W.draw_children_tokens(parent, dl, 0.0, rng)  # children = draft top-k
        u = rng.random(n + 1, dtype=np.float32)
        g = O.tree_verify(parent, tokens, tl, dl, 0.0, u)
        # direct statement of greedy: follow the child whose token is the target arg-max
        kids, cur, expect = W.children_lists(parent), 0, [0]
        while True:
            a = int(np.argmax(tl[cur]))
            nxt = [c for c in kids[cur] if tokens[c] == a]
            if not nxt:
                break
            cur = nxt[0]
            expect.append(cur)
        assert list(g["path"]) == expect and g["bonus"] == int(np.argmax(tl[cur]))
        assert g["residual"][g["bonus"]] == 1.0 and g["residual"].sum() == 1.0
        # the general loop at a tiny temperature gives the same outcome
        s = O.tree_verify(parent, tokens, tl, dl, 1e-3, u)
        assert list(s["path"]) == expect and s["bonus"] == g["bonus"]
        agree += len(expect) > 1
    assert agree >= 5
    # ties -> lowest index
    tl = np.zeros((1, 5), np.float32)
    tl[0, [1, 3]] = 2.0
    assert O.tree_verify([-1], [0], tl, tl, 0.0, np.array([0, 0.9], np.float32))["bonus"] == 1


def test_walk_invariants_on_a_config_shaped_workload():
    cfg = W.CONFIGS["tiny"]
    for seed in range(4):
        vi = W.make_verify_inputs(cfg, 0.6, seed, vocab=2000)
        parent = vi.parent.numpy()
        res = O.tree_verify(parent, vi.tokens, vi.target_logits, vi.draft_logits, 0.6, vi.uniforms)
        R = res["residual"]
        assert (R >= 0).all() and abs(R.sum() - 1) < 1e-12 and R[res["bonus"]] > 0
        path = res["path"]
        assert path[0] == 0 and all(parent[path[i]] == path[i - 1] for i in range(1, len(path)))
        last = path[-1]
        assert res["next_child"][last] == -1
        rejected = [int(vi.tokens[c]) for c in W.children_lists(parent)[last]]
        assert all(R[t] == 0.0 for t in rejected)  # a rejected token leaves the residual for good
        assert set(np.flatnonzero(R)) <= set(np.flatnonzero(O.softmax_T(vi.target_logits[last], 0.6)))
        # rows off the path (and draft rows of leaves) do not matter
        tl, dl = vi.target_logits.numpy().copy(), vi.draft_logits.numpy().copy()
        off = [i for i in range(len(parent)) if i not in set(path)]
        tl[off] = 123.0
        dl[off] = -7.0
        dl[last] = 0.0 if not rejected else dl[last]
        res2 = O.tree_verify(parent, vi.tokens, tl, dl, 0.6, vi.uniforms)
        assert list(res2["path"]) == list(path) and res2["bonus"] == res["bonus"]


def _chi2_ok(counts, probs, trials):
    exp = probs * trials
    keep = exp >= 5
    stat = ((counts[keep] - exp[keep]) ** 2 / exp[keep]).sum()
    dof = keep.sum() - 1
    return stat < dof + 6 * np.sqrt(2 * dof), stat, dof  # ~6 sigma of the chi-square law


@pytest.mark.parametrize("T", [1.0, 0.6, 0.2])
@pytest.mark.parametrize("k", [1, 4, 24])
def test_monte_carlo_output_distribution_equals_target(T, k):
    """Root + k children drawn without replacement from the draft; the emitted token (accepted
    child's token, else the bonus) must be distributed as softmax(target/T)."""
    V, trials = 24, 60000
    rng = np.random.default_rng(1000 + k)
    tl = (2.0 * rng.standard_normal(V)).astype(np.float32)
    dl = (tl + 1.5 * rng.standard_normal(V)).astype(np.float32)
    n = k + 1
    parent = W.star_tree(n)
    TL = np.ascontiguousarray(np.broadcast_to(tl, (n, V)))
    DL = np.ascontiguousarray(np.broadcast_to(dl, (n, V)))
    keys = dl.astype(np.float64) / T + rng.gumbel(size=(trials, V))
    kids = np.argsort(-keys, axis=1)[:, :k].astype(np.int32)
    U = rng.random((trials, n + 1), dtype=np.float32)
    L = O.lib()
    pi, pf, pd = C.POINTER(C.c_int32), C.POINTER(C.c_float), C.POINTER(C.c_double)
    tokens = np.zeros(n, np.int32)
    path = np.zeros(n, np.int32)
    plen, bonus = C.c_int32(), C.c_int32()
    counts = np.zeros(V)
    accepted = 0
    for t in range(trials):
        tokens[1:] = kids[t]
        u = U[t]
        L.orc_tree_verify(n, V, parent.ctypes.data_as(pi), tokens.ctypes.data_as(pi), TL.ctypes.data_as(pf), V,
                          DL.ctypes.data_as(pf), V, T, u.ctypes.data_as(pf), 0, path.ctypes.data_as(pi),
                          C.byref(plen), C.byref(bonus), None, None, None, None)
        if plen.value == 2:
            counts[tokens[path[1]]] += 1
            accepted += 1
        else:
            counts[bonus.value] += 1
    ok, stat, dof = _chi2_ok(counts, _softmax64(tl, T), trials)
    assert ok, (stat, dof)
    if k == V:
        assert accepted == trials  # cover property: k = vocabulary size always accepts
    # the check has teeth: the draft distribution would fail it
    assert not _chi2_ok(counts, _softmax64(dl, T), trials)[0]


def test_monte_carlo_greedy_is_exact():
    rng = np.random.default_rng(18)
    V, k = 24, 4
    tl = rng.standard_normal((k + 1, V)).astype(np.float32)
    dl = (tl + rng.standard_normal((k + 1, V))).astype(np.float32)
    for _ in range(200):
        tokens = np.zeros(k + 1, np.int32)
        tokens[1:] = rng.choice(V, k, replace=False)
        r = O.tree_verify(W.star_tree(k + 1), tokens, tl, dl, 0.0, rng.random(k + 2, dtype=np.float32))
        emitted = tokens[r["path"][1]] if r["path_len"] == 2 else r["bonus"]
        assert emitted == int(np.argmax(tl[0]))
