"""Pins of the oracle's verification by sampling from the target ("naive" / "top-k sampling", Section 2.2):
on a chain it is plain autoregressive sampling (library inverse CDF), the emitted first token follows the
target distribution whatever the tree (Monte-Carlo), T = 0 is arg-max matching, and invariants."""
import numpy as np

from oracle import oracle as O
from paper_2402_12374_b200 import workloads as W


def _softmax(x, T):
    z = np.exp((x.astype(np.float64) - x.max()) / T)
    return z / z.sum()


def test_chain_is_plain_autoregressive_sampling_with_a_library_inverse_cdf():
    rng = np.random.default_rng(0)
    n, V, T = 9, 40, 0.8
    parent = W.chain_tree(n)
    for trial in range(200):
        tl = (2 * rng.standard_normal((n, V))).astype(np.float32)
        u = rng.random(n + 1).astype(np.float32)
        # what the target would emit position by position, with numpy's own cumulative sum and search
        want = [int(np.searchsorted(np.cumsum(_softmax(tl[v], T)), np.float64(u[v]), side="right")) for v in range(n)]
        tokens = np.zeros(n, np.int32)
        tokens[1:] = rng.integers(0, V, n - 1)
        agree = rng.integers(0, n)           # the chain guesses the first `agree` tokens right
        tokens[1:1 + agree] = want[:agree]
        if agree < n - 1 and tokens[1 + agree] == want[agree]:
            tokens[1 + agree] = (want[agree] + 1) % V
        r = O.tree_verify_target_sample(parent, tokens, tl, T, u)
        assert r["path"].tolist() == list(range(agree + 1)), (agree, r["path"])
        assert r["bonus"] == want[agree] and r["path_len"] == agree + 1
        np.testing.assert_allclose(r["residual"], _softmax(tl[agree], T), atol=1e-12)


def test_first_emitted_token_follows_the_target_whatever_the_tree():
    rng = np.random.default_rng(1)
    V, n, T = 12, 7, 0.9
    parent = W.star_tree(n)
    tl = np.tile((1.5 * rng.standard_normal(V)).astype(np.float32), (n, 1))
    tokens = np.array([0, 3, 5, 7, 8, 9, 11], np.int32)
    P = _softmax(tl[0], T)
    N = 40000
    cnt = np.zeros(V)
    for _ in range(N):
        u = rng.random(n + 1).astype(np.float32)
        r = O.tree_verify_target_sample(parent, tokens, tl, T, u)
        first = tokens[r["path"][1]] if r["path_len"] > 1 else r["bonus"]
        cnt[first] += 1
    assert (np.abs(cnt - N * P) <= 5 * np.sqrt(N * P * (1 - P)) + 1).all()


def test_temperature_zero_is_argmax_matching_and_agrees_with_the_greedy_walk():
    cfg = W.CONFIGS["tiny"]
    for seed in range(6):
        vi = W.make_verify_inputs(cfg, 0.0, seed, vocab=512)
        a = O.tree_verify_target_sample(vi.parent, vi.tokens, vi.target_logits, 0.0, vi.uniforms)
        b = O.tree_verify(vi.parent, vi.tokens, vi.target_logits, vi.draft_logits, 0.0, vi.uniforms)
        assert a["path"].tolist() == b["path"].tolist() and a["bonus"] == b["bonus"]
        v = int(a["path"][-1])
        assert a["bonus"] == int(np.argmax(vi.target_logits[v].numpy()))


def test_invariants_on_a_config_shaped_tree():
    cfg = W.CONFIGS["tiny"]
    for seed in range(5):
        vi = W.make_verify_inputs(cfg, 0.6, seed, vocab=1024)
        r = O.tree_verify_target_sample(vi.parent, vi.tokens, vi.target_logits, 0.6, vi.uniforms)
        par = vi.parent.numpy()
        path = r["path"]
        assert path[0] == 0 and all(par[path[i + 1]] == path[i] for i in range(len(path) - 1))
        assert (r["next_child"][path[:-1]] == path[1:]).all() and r["next_child"][path[-1]] == -1
        visited = r["next_child"] != -2
        assert visited.sum() == r["path_len"]
        last_kids = [c for c in range(len(par)) if par[c] == path[-1]]
        assert all(int(vi.tokens[c]) != r["bonus"] for c in last_kids)
        assert abs(r["residual"].sum() - 1) < 1e-12 and r["flags"] == 0


def _accept_measure(parent, tokens, tl, T, N=20000):
    """Lebesgue measure of the root uniforms for which some child is accepted: the walk is a deterministic
    function of uniforms[0], so the measure is read off a midpoint grid (exact when the CDF steps lie on it)."""
    n = len(parent)
    hits = 0
    for j in range(N):
        u = np.zeros(n + 1, np.float32)
        u[0] = (j + 0.5) / N
        hits += O.tree_verify_target_sample(parent, tokens, tl, T, u)["path_len"] > 1
    return hits / N


def test_printed_top_k_example_accepts_with_probability_0_6():
    """The value the paper prints for this verifier (appendix, proof of the robustness theorem, item on top-k
    naive sampling and optimal transport): P = Q = [0.6, 0.4], one speculated token (the draft's top-1, token 0)
    is accepted with probability 0.6, although 1 - |P - Q|_1 / 2 = 1."""
    import json
    import os

    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_examples.json")))["top_k_naive_sampling"]
    P, Q, k = np.array(g["P"]), np.array(g["Q"]), g["k"]
    top = np.argsort(-Q, kind="stable")[:k]                 # the draft's top-k tokens are the children
    parent = W.star_tree(1 + k)
    tokens = np.concatenate([[0], top]).astype(np.int32)
    tl = np.tile(np.log(P).astype(np.float32), (1 + k, 1))
    assert abs(_accept_measure(parent, tokens, tl, 1.0) - g["naive_acceptance"]) < 1e-9
    assert abs((1 - np.abs(P - Q).sum() / 2) - g["optimal_transport_acceptance"]) < 1e-12
    # Algorithm 2 on the same pair accepts always (optimal transport at k = 1)
    st = O.alg2_node(P, Q, top, [0.999999])
    assert st["accepted"] == 0


def test_top_k_cover_property_of_sampling_from_the_target():
    """Same proof, next item: when the k children are the draft's top-k and contain the target's support, or
    k = V, the sample from the target is always among them."""
    P = np.array([0.5, 0.0, 0.3, 0.0, 0.2])
    tl = np.log(np.maximum(P, 1e-300)).astype(np.float32)
    tl[P == 0] = -np.inf
    for kids in ([0, 2, 4], [4, 2, 0, 1], [0, 1, 2, 3, 4]):
        parent = W.star_tree(1 + len(kids))
        tokens = np.array([0] + kids, np.int32)
        assert _accept_measure(parent, tokens, np.tile(tl, (len(parent), 1)), 1.0, N=2000) == 1.0
    # one token of the support missing: accepted exactly with the mass that is covered
    parent = W.star_tree(3)
    assert abs(_accept_measure(parent, np.array([0, 0, 4], np.int32), np.tile(tl, (3, 1)), 1.0, N=2000) - 0.7) < 1e-9
