"""Pins of the oracle's cache commit (``orc_kv_commit``): a library gather, hand-written cases, and the identity
that ties the commit to the attention oracle — after the commit, plain causal attention over the new prefix gives
every accepted node exactly what tree attention gave it before."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2402_12374_b200 import workloads as W


def _random_path(rng, parent, min_len=1):
    """A root-to-node path of the tree: walk down taking a random child until a leaf or a coin says stop."""
    kids = W.children_lists(parent)
    path, cur = [0], 0
    while kids[cur] and (len(path) < min_len or rng.random() < 0.8):
        cur = int(rng.choice(kids[cur]))
        path.append(cur)
    return np.array(path, np.int32)


def test_commit_equals_library_gather_and_leaves_other_rows_alone():
    rng = np.random.default_rng(0)
    for dtype, d in ((np.uint16, 128), (np.float32, 64), (np.uint8, 48)):
        L, n, planes, rows = 37, 29, 5, 37 + 29 + 3
        cache = rng.integers(0, 250, size=(planes, rows, d)).astype(dtype)
        parent = W.make_tree(W.CONFIGS["tiny"], 3)
        parent = np.concatenate([parent, np.arange(len(parent) - 1, n - 1)]).astype(np.int32)[:n]
        path = _random_path(rng, parent, min_len=3)
        out, flags = O.kv_commit(cache, L, n, path)
        assert flags == 0
        expect = cache.copy()
        expect[:, L:L + len(path)] = np.take(cache, L + path, axis=1)  # the library's gather
        assert np.array_equal(out, expect)
        assert np.array_equal(out[:, :L], cache[:, :L]) and np.array_equal(out[:, L + len(path):], cache[:, L + len(path):])


def test_commit_hand_written_overlap_case():
    """path = [0, 2, 3, 6]: row L+2 is read (for slot 1) and overwritten (slot 2 <- node 3) in the same commit;
    the result must be made of the OLD rows."""
    L, n = 2, 7
    cache = (np.arange(1 * (L + n) * 4).reshape(1, L + n, 4)).astype(np.float32)
    old = cache.copy()
    out, flags = O.kv_commit(cache, L, n, [0, 2, 3, 6])
    assert flags == 0 and np.array_equal(cache, old)  # the input is not touched
    for slot, node in enumerate([0, 2, 3, 6]):
        assert np.array_equal(out[0, L + slot], old[0, L + node])
    for r in (0, 1, 6, 7, 8):
        assert np.array_equal(out[0, r], old[0, r])


def test_commit_identity_path_and_empty_path_change_nothing():
    cache = np.random.default_rng(1).standard_normal((3, 20, 8)).astype(np.float32)
    for path in ([0, 1, 2, 3, 4], [0], []):
        out, flags = O.kv_commit(cache, 10, 10, path)
        assert flags == 0 and np.array_equal(out, cache)


@pytest.mark.parametrize("path", [[1, 2], [0, 2, 2], [0, 3, 2], [0, 10], [0, -1], list(range(11))])
def test_commit_invalid_path_is_flagged_and_moves_nothing(path):
    cache = np.random.default_rng(2).standard_normal((2, 20, 8)).astype(np.float32)
    out, flags = O.kv_commit(cache, 10, 10, path)
    assert flags == O.BAD_PATH and np.array_equal(out, cache)


def test_attention_over_committed_cache_equals_tree_attention_of_the_path():
    """The reason the commit exists: node path[m] saw the prefix and path[0..m]; after the commit those keys are rows
    [0, L+m], so causal (chain-tree) attention of the same queries over the committed cache returns the same
    vectors.  Checked with the attention oracle on a chain parent array."""
    rng = np.random.default_rng(5)
    cfg = W.CONFIGS["tiny"]
    for seed in range(3):
        ai = W.make_attention_inputs(cfg, seed, dtype="fp32")
        parent = ai.parent.numpy()
        n, L = len(parent), ai.prefix_len
        path = _random_path(rng, parent, min_len=3)
        q, k, v = ai.q.double().numpy(), ai.k_cache.double().numpy(), ai.v_cache.double().numpy()
        tree_out, _, f0 = O.tree_attention(q, k, v, parent, L)
        k2, fk = O.kv_commit(k, L, n, path)
        v2, fv = O.kv_commit(v, L, n, path)
        m = len(path)
        chain = np.arange(-1, m - 1, dtype=np.int32)
        chain_out, _, f1 = O.tree_attention(np.ascontiguousarray(q[path]), k2, v2, chain, L)
        assert f0 == f1 == fk == fv == 0
        assert np.abs(chain_out - tree_out[path]).max() < 1e-13
        # and a path that is NOT the accepted one gives something else (the pin can fail)
        other = path.copy()
        sib = [c for c in range(1, n) if c not in set(path.tolist()) and parent[c] == path[-2]]
        if sib:
            other[-1] = sib[0]
            other.sort()
            k3, _ = O.kv_commit(k, L, n, other)
            v3, _ = O.kv_commit(v, L, n, other)
            wrong, _, _ = O.tree_attention(np.ascontiguousarray(q[path]), k3, v3, chain, L)
            assert np.abs(wrong[-1] - tree_out[path[-1]]).max() > 1e-6
