"""Pins of the oracle's ancestor mask and tree attention against things fixed outside it:
library causal attention (chain tree), single-query decode (star tree, n = 1), explicit-sequence
brute force over every 5-node tree, and invariants of the definition."""
import itertools

import numpy as np
import pytest
import torch
from scipy.special import logsumexp

from oracle import oracle as O
from paper_2402_12374_b200 import workloads as W


def _closure(parent):
    """Ancestor-or-self relation by repeated boolean squaring of the parent adjacency."""
    n = len(parent)
    A = np.eye(n, dtype=bool)
    for i, p in enumerate(parent):
        if p >= 0:
            A[i, p] = True
    for _ in range(int(np.ceil(np.log2(max(n, 2)))) + 1):
        A = (A.astype(np.int64) @ A.astype(np.int64)) > 0
    return A


def _unpack(mask, n):
    bits = ((mask[:, :, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(mask.shape[0], -1)
    return bits[:, :n].astype(bool)


@pytest.mark.parametrize("n,seed", [(1, 0), (2, 0), (17, 1), (64, 2), (100, 3), (130, 4), (768, 5)])
def test_mask_matches_transitive_closure(n, seed):
    parent = W.random_tree(n, None, None, np.random.default_rng(seed))
    mask, depth, flags = O.mask_from_parents(parent)
    assert flags == 0
    M = _unpack(mask, n)
    assert np.array_equal(M, _closure(parent))
    assert np.array_equal(M.sum(1), depth + 1)
    assert M[0].sum() == 1 and M[0, 0]
    assert not np.triu(M, 1).any() and M.diagonal().all()
    for i in range(1, n):
        expect = M[parent[i]].copy()
        expect[i] = True
        assert np.array_equal(M[i], expect)
    # bits beyond n in the last word stay clear
    assert _unpack(mask, mask.shape[1] * 32)[:, n:].sum() == 0


def test_mask_chain_star_forest_and_bad_parent():
    M = _unpack(O.mask_from_parents(W.chain_tree(40))[0], 40)
    assert np.array_equal(M, np.tril(np.ones((40, 40), bool)))
    M = _unpack(O.mask_from_parents(W.star_tree(40))[0], 40)
    expect = np.eye(40, dtype=bool)
    expect[:, 0] = True
    assert np.array_equal(M, expect)
    # forest: a second parentless node sees only itself
    mask, depth, flags = O.mask_from_parents(np.array([-1, 0, -1, 2], np.int32))
    assert flags == 0 and list(depth) == [0, 1, 0, 1]
    assert np.array_equal(_unpack(mask, 4), np.array([[1, 0, 0, 0], [1, 1, 0, 0], [0, 0, 1, 0], [0, 0, 1, 1]], bool))
    # a parent that is not an earlier node is flagged and read as "no parent"
    mask, depth, flags = O.mask_from_parents(np.array([-1, 0, 2, 5], np.int32))
    assert flags & O.BAD_PARENT
    assert np.array_equal(_unpack(mask, 4)[2:], np.array([[0, 0, 1, 0], [0, 0, 0, 1]], bool))


def _rand_qkv(rng, n, L, Hq, Hkv, d, extra=0):
    q = rng.standard_normal((n, Hq, d))
    k = rng.standard_normal((Hkv, L + n + extra, d))
    v = rng.standard_normal((Hkv, L + n + extra, d))
    return q, k, v


def test_chain_tree_is_library_causal_attention():
    rng = np.random.default_rng(0)
    n, L, H, d = 9, 13, 3, 16
    q, k, v = _rand_qkv(rng, n, L, H, H, d)
    out, lse, _ = O.tree_attention(q, k, v, W.chain_tree(n), L)
    tq = torch.from_numpy(q).permute(1, 0, 2)  # [H, n, d]
    mask = torch.ones(n, L + n, dtype=torch.bool)
    mask[:, L:] = torch.tril(torch.ones(n, n, dtype=torch.bool))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, torch.from_numpy(k), torch.from_numpy(v), attn_mask=mask)
    np.testing.assert_allclose(out, ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)
    s = np.einsum("ihc,hjc->hij", q, k) / np.sqrt(d)
    s = np.where(mask.numpy()[None], s, -np.inf)
    np.testing.assert_allclose(lse, logsumexp(s, axis=2), rtol=0, atol=1e-12)


def test_star_tree_and_single_node_are_plain_decode():
    rng = np.random.default_rng(1)
    n, L, H, d = 6, 10, 2, 8
    q, k, v = _rand_qkv(rng, n, L, H, H, d)
    out, _, _ = O.tree_attention(q, k, v, W.star_tree(n), L)
    for i in range(n):
        keys = list(range(L)) + [L] + ([L + i] if i else [])
        for h in range(H):
            w = torch.softmax(torch.from_numpy(k[h, keys] @ q[i, h]) / np.sqrt(d), 0).numpy()
            np.testing.assert_allclose(out[i, h], w @ v[h, keys], atol=1e-12)
    # n = 1 with and without a prefix (L = 0: the root sees only itself -> output is its own V row)
    out1, _, _ = O.tree_attention(q[:1], k[:, : L + 1], v[:, : L + 1], np.array([-1], np.int32), L)
    np.testing.assert_allclose(out1, out[:1], atol=1e-12)
    out0, lse0, _ = O.tree_attention(q[:1], k[:, :1], v[:, :1], np.array([-1], np.int32), 0)
    np.testing.assert_allclose(out0[0], v[:, 0], atol=1e-12)
    np.testing.assert_allclose(lse0[:, 0], np.einsum("hc,hc->h", q[0], k[:, 0]) / np.sqrt(d), atol=1e-12)


def test_brute_force_every_five_node_tree():
    """For each of the 24 parent arrays with parent[i] < i: row i must equal unmasked dense softmax
    attention over the explicit sequence prefix + path(i)."""
    rng = np.random.default_rng(2)
    n, L, H, d = 5, 3, 2, 4
    q, k, v = _rand_qkv(rng, n, L, H, H, d)
    count = 0
    for tail in itertools.product(*[range(i) for i in range(1, n)]):
        parent = np.array((-1,) + tail, np.int32)
        out, _, _ = O.tree_attention(q, k, v, parent, L, scale=0.7)
        for i in range(n):
            path, j = [], i
            while j >= 0:
                path.append(j)
                j = parent[j]
            seq = list(range(L)) + [L + a for a in reversed(path)]
            for h in range(H):
                s = 0.7 * (k[h, seq] @ q[i, h])
                w = np.exp(s - s.max())
                np.testing.assert_allclose(out[i, h], (w / w.sum()) @ v[h, seq], atol=1e-12)
        count += 1
    assert count == 24


def test_gqa_maps_consecutive_query_heads_to_one_kv_head():
    rng = np.random.default_rng(3)
    n, L, Hq, Hkv, d = 7, 5, 8, 2, 8
    q, k, v = _rand_qkv(rng, n, L, Hq, Hkv, d)
    parent = W.random_tree(n, None, None, rng)
    out, lse, _ = O.tree_attention(q, k, v, parent, L)
    out_mha, lse_mha, _ = O.tree_attention(q, np.repeat(k, 4, axis=0), np.repeat(v, 4, axis=0), parent, L)
    assert np.array_equal(out, out_mha) and np.array_equal(lse, lse_mha)


def test_attention_invariants():
    rng = np.random.default_rng(4)
    n, L, H, d = 12, 6, 2, 8
    parent = W.random_tree(n, None, None, rng)
    q, k, v = _rand_qkv(rng, n, L, H, H, d, extra=3)
    k[:, L + n:] = np.nan
    v[:, L + n:] = np.nan
    out, lse, _ = O.tree_attention(q, k, v, parent, L)
    assert np.isfinite(out).all() and np.isfinite(lse).all()  # rows past L+n are never read
    M = _closure(parent)
    # (i) junk in every non-ancestor tree row leaves row i bitwise unchanged
    for i in range(n):
        k2, v2 = k.copy(), v.copy()
        for a in range(n):
            if not M[i, a]:
                k2[:, L + a] = 1e4 * (-1) ** a
                v2[:, L + a] = -1e4
        o2, l2, _ = O.tree_attention(q, k2, v2, parent, L)
        assert np.array_equal(o2[i], out[i]) and np.array_equal(l2[:, i], lse[:, i])
    # (iii) relabelling the nodes by another topological order permutes the rows
    order = [0] + sorted(range(1, n), key=lambda i: (int(M[i].sum()), -i))  # by depth, then reversed index
    inv = np.empty(n, np.int64)
    inv[order] = np.arange(n)
    parent2 = np.array([-1 if parent[o] < 0 else inv[parent[o]] for o in order], np.int32)
    assert all(parent2[i] < i for i in range(n))
    k3, v3 = k.copy(), v.copy()
    k3[:, L:L + n] = k[:, L + np.array(order)]
    v3[:, L:L + n] = v[:, L + np.array(order)]
    o3, _, _ = O.tree_attention(q[order], k3, v3, parent2, L)
    np.testing.assert_allclose(o3, out[order], atol=1e-12)
    # (iv) all V rows equal r -> output r
    r = rng.standard_normal(d)
    vr = np.broadcast_to(r, v[:, :L + n].shape).copy()
    o4, _, _ = O.tree_attention(q, k[:, :L + n], vr, parent, L)
    np.testing.assert_allclose(o4, np.broadcast_to(r, o4.shape), atol=1e-12)
    # a change of one key the row does see changes the row (mask is not over-restrictive)
    i = n - 1
    k5 = k.copy()
    k5[:, L + parent[i]] += 1.0
    o5, _, _ = O.tree_attention(q, k5, v, parent, L)
    assert not np.allclose(o5[i], out[i])


def test_sixteen_bit_inputs_are_taken_at_their_exact_value():
    rng = np.random.default_rng(5)
    q = torch.from_numpy(rng.standard_normal((3, 2, 8)).astype(np.float32)).to(torch.bfloat16)
    k = torch.from_numpy(rng.standard_normal((2, 7, 8)).astype(np.float32)).to(torch.bfloat16)
    v = torch.from_numpy(rng.standard_normal((2, 7, 8)).astype(np.float32)).to(torch.bfloat16)
    a, _, _ = O.tree_attention(q, k, v, W.chain_tree(3), 4)
    b, _, _ = O.tree_attention(q.double().numpy(), k.double().numpy(), v.double().numpy(), W.chain_tree(3), 4)
    assert np.array_equal(a, b)
