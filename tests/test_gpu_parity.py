"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded
inputs.  Integer results bit-exact; attention within 2e-2 abs (16-bit inputs) / 1e-5 (fp32 mode);
residual probabilities within 1e-5 abs; accepted path and bonus identical outside the band
|u - ratio| < 1e-5."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2402_12374_b200 import binding as B
from paper_2402_12374_b200 import workloads as W
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


# ---------------------------------------------------------------- mask ------------------------------
@pytest.mark.parametrize("n,seed", [(1, 0), (2, 0), (16, 1), (17, 2), (64, 3), (100, 4), (130, 5), (768, 6), (1024, 7)])
def test_mask_bit_exact(n, seed):
    parent = W.random_tree(n, 20, 16, np.random.default_rng(seed))
    for p in (parent, W.chain_tree(n), W.star_tree(n)):
        mask, depth, st = G.gpu_mask(p)
        omask, odepth, _ = O.mask_from_parents(p)
        assert np.array_equal(mask.cpu().numpy().view(np.uint32), omask)
        assert np.array_equal(depth.cpu().numpy(), odepth) and int(st.item()) == 0


def test_mask_wide_rows_forest_and_bad_parent():
    d = G.dev()
    parent = np.array([-1, 0, -1, 2, 9, 1, -5], np.int32)
    st = torch.zeros(1, dtype=torch.int32, device=d)
    mask = torch.full((7, 3), -1, dtype=torch.int32, device=d)
    B.seq_tree_mask_from_parents(torch.from_numpy(parent).to(d), words_per_row=3, mask_bits=mask, dev_status=st)
    omask, odepth, oflags = O.mask_from_parents(parent, words_per_row=3)
    assert np.array_equal(mask.cpu().numpy().view(np.uint32), omask)
    assert int(st.item()) == B.SEQ_DEV_BAD_PARENT and oflags == O.BAD_PARENT


# ---------------------------------------------------------------- attention -------------------------
def _cfg(name, **kw):
    return dataclasses.replace(W.CONFIGS[name], **kw)


@pytest.mark.parametrize("seed", range(4))
def test_attention_tiny_config(seed):
    G.check_attention(W.make_attention_inputs(W.CONFIGS["tiny"], seed))


@pytest.mark.parametrize("dtype", ["fp16", "bf16", "fp32"])
@pytest.mark.parametrize("kernel", [B.KERNEL_AUTO, B.KERNEL_CUDA_CORE])
def test_attention_dtypes_small(dtype, kernel):
    cfg = _cfg("tiny", num_q_heads=8, num_kv_heads=8, prefix_len=300, n_tree=40)
    G.check_attention(W.make_attention_inputs(cfg, 1, dtype=dtype), kernel=kernel)


def test_attention_fp32_mode_config_shapes():
    G.check_attention(W.make_attention_inputs(W.CONFIGS["tiny"], 0, dtype="fp32"))
    cfg = _cfg("llama2-7b", num_q_heads=8, num_kv_heads=8)  # config-2 shape, fewer heads for the oracle's sake
    G.check_attention(W.make_attention_inputs(cfg, 0, dtype="fp32"))


@pytest.mark.parametrize("n,L", [(1, 0), (1, 77), (5, 0), (17, 33), (100, 129), (130, 1000)])
def test_attention_edge_sizes(n, L):
    cfg = _cfg("tiny", num_q_heads=4, num_kv_heads=2, prefix_len=L, n_tree=n, max_depth=12)
    for dtype in ("bf16", "fp32"):
        G.check_attention(W.make_attention_inputs(cfg, 2, dtype=dtype))


@pytest.mark.parametrize("tree", ["chain", "star"])
def test_attention_chain_and_star(tree):
    cfg = _cfg("tiny", num_q_heads=4, num_kv_heads=4, prefix_len=200, n_tree=64)
    parent = W.chain_tree(64) if tree == "chain" else W.star_tree(64)
    G.check_attention(W.make_attention_inputs(cfg, 3, parent=parent))


def test_attention_gqa_and_custom_scale():
    cfg = _cfg("tiny", num_q_heads=16, num_kv_heads=2, prefix_len=150, n_tree=48)
    G.check_attention(W.make_attention_inputs(cfg, 4, dtype="bf16"), scale=0.05)


def test_attention_masked_keys_contribute_exactly_zero_and_nan_tail_is_never_read():
    cfg = _cfg("tiny", num_q_heads=4, num_kv_heads=4, prefix_len=96, n_tree=40)
    ai = W.make_attention_inputs(cfg, 5, dtype="bf16", extra_capacity=24)  # NaN rows past L+n
    base, lse, st = G.run_attention(ai)
    assert st == 0 and torch.isfinite(base).all() and torch.isfinite(lse).all()
    G.check_attention(ai)
    # junk in every tree row that node i cannot see leaves row i bitwise unchanged
    M, _, _ = O.mask_from_parents(ai.parent)
    n, L = 40, 96
    for i in (0, 7, 23, 39):
        k2, v2 = ai.k_cache.clone(), ai.v_cache.clone()
        for a in range(n):
            if not (M[i, a >> 5] >> (a & 31)) & 1:
                k2[:, L + a] = 1e4 * (-1) ** a
                v2[:, L + a] = -1e4
        out2, lse2, _ = G.run_attention(dataclasses.replace(ai, k_cache=k2, v_cache=v2))
        assert torch.equal(out2[i], base[i]) and torch.equal(lse2[:, i], lse[:, i])


def test_attention_strided_views():
    """q/out as slices of a fused [n, Hq+2Hkv, d] projection; K/V cache with spare capacity."""
    cfg = _cfg("tiny", num_q_heads=8, num_kv_heads=4, prefix_len=64, n_tree=20)
    ai = W.make_attention_inputs(cfg, 6, dtype="bf16", extra_capacity=16, tail_fill=0.0)
    d = G.dev()
    fused = torch.zeros((20, 16, 128), dtype=torch.bfloat16, device=d)
    fused[:, :8] = ai.q.to(d)
    out_buf = torch.zeros((20, 12, 128), dtype=torch.bfloat16, device=d)
    mask, _, _ = G.gpu_mask(ai.parent.numpy())
    B.seq_tree_attention(fused[:, :8], ai.k_cache.to(d), ai.v_cache.to(d), mask, 64, out=out_buf[:, 2:10])
    torch.cuda.synchronize()
    ref, _, _ = O.tree_attention(ai.q, ai.k_cache, ai.v_cache, ai.parent, 64)
    assert np.abs(out_buf[:, 2:10].double().cpu().numpy() - ref).max() < 2e-2
    assert out_buf[:, :2].abs().sum() == 0 and out_buf[:, 10:].abs().sum() == 0


# ---------------------------------------------------------------- verification ----------------------
def _verify_cases(name, T, seeds, vocab=None, parent=None):
    cfg = W.CONFIGS[name]
    outcomes = []
    for seed in seeds:
        vi = W.make_verify_inputs(cfg, T, seed, vocab=vocab, parent=parent)
        outcomes.append(G.check_verify(vi))
    assert outcomes.count("ok") >= max(1, len(outcomes) - 1), outcomes
    return outcomes


def test_verify_tiny_config():
    _verify_cases("tiny", 0.6, range(8))


@pytest.mark.parametrize("T", [0.0, 0.6, 1.0])
def test_verify_llama2_7b_config(T):
    _verify_cases("llama2-7b", T, range(8) if T == 0.6 else range(4))


def test_verify_llama2_13b_config():
    _verify_cases("llama2-13b", 1.0, range(2))


def test_verify_vicuna_33b_config():
    _verify_cases("vicuna-33b", 0.6, range(2))


@pytest.mark.parametrize("V", [1, 2, 7, 8, 33, 1000, 4099, 50257])
def test_verify_ragged_vocab_sizes(V):
    cfg = _cfg("tiny", n_tree=min(12, V + 1), max_fanout=max(1, min(3, V)))
    for seed in range(3):
        G.check_verify(W.make_verify_inputs(cfg, 0.8, seed, vocab=V))


@pytest.mark.parametrize("T", [0.0, 0.6])
def test_verify_every_node_hook(T):
    vi = W.make_verify_inputs(W.CONFIGS["llama2-13b"], T, 0, vocab=8192)
    checked, excluded = G.check_verify_all_nodes(vi)
    assert checked >= 20 and excluded <= 2


def test_verify_chain_star_single_node():
    cfg = W.CONFIGS["tiny"]
    for parent in (W.chain_tree(24), W.star_tree(24), np.array([-1], np.int32)):
        for seed in range(3):
            G.check_verify(W.make_verify_inputs(cfg, 0.7, seed, parent=parent, vocab=3000))


def test_verify_uniform_fallback_duplicates_and_bad_tokens():
    """A node with more children than the draft's support (-inf draft logits) drives the uniform
    fallback; a duplicated sibling token and an out-of-range token take their documented paths."""
    rng = np.random.default_rng(0)
    V, n = 64, 12
    parent = W.star_tree(n)
    for trial in range(20):
        tl = (2 * rng.standard_normal((n, V))).astype(np.float32)
        dl = np.full((n, V), -np.inf, np.float32)
        supp = rng.choice(V, 4, replace=False)
        dl[:, supp] = tl[:, supp] + rng.standard_normal((n, 4)).astype(np.float32)
        tokens = W.draw_children_tokens(parent, dl, 0.9, rng)
        u = (0.9 + 0.1 * rng.random(n + 1)).astype(np.float32)  # large uniforms: many rejections
        u[-1] = rng.random()
        vi = W.VerifyInputs(torch.from_numpy(parent), torch.from_numpy(tokens), torch.from_numpy(tl),
                            torch.from_numpy(dl), torch.from_numpy(u), 0.9)
        G.check_verify(vi)
    # bad tokens first (always reached), then a duplicated sibling
    dl = (tl + 2 * rng.standard_normal((n, V))).astype(np.float32)
    tokens = W.draw_children_tokens(parent, dl, 0.9, rng)
    tokens[1] = V + 3
    tokens[2] = -1
    tokens[4] = tokens[3]
    u = np.full(n + 1, 0.999, np.float32)
    vi = W.VerifyInputs(torch.from_numpy(parent), torch.from_numpy(tokens), torch.from_numpy(tl),
                        torch.from_numpy(dl), torch.from_numpy(u), 0.9)
    got = G.run_verify(vi)
    ref = O.tree_verify(parent, tokens, tl, dl, 0.9, u)
    assert got["status"] == B.SEQ_DEV_BAD_TOKEN and ref["flags"] == O.BAD_TOKEN
    assert ref["min_gap"] > 1e-5 and ref["ratio"][4] == 0.0  # the duplicate was tested and had ratio 0
    assert got["path"].tolist() == ref["path"].tolist() and got["bonus"] == ref["bonus"]
    assert np.abs(got["residual"] - ref["residual"]).max() < 1e-5


@pytest.mark.parametrize("name,T,seeds", [("tiny", 0.6, range(8)), ("llama2-7b", 0.6, range(4)), ("llama2-7b", 1.0, range(3)),
                                          ("llama2-13b", 1.0, range(2))])
def test_verify_specinfer_variant_configs(name, T, seeds):
    """SEQ_VERIFY_SPECINFER: Algorithm 2 without lines 10-16 (D untouched after a rejection), against the
    oracle's walk of the same variant."""
    cfg = W.CONFIGS[name]
    outcomes = [G.check_verify(W.make_verify_inputs(cfg, T, seed), specinfer=True) for seed in seeds]
    assert outcomes.count("ok") >= max(1, len(outcomes) - 1), outcomes


def test_verify_specinfer_children_with_replacement_and_many_rejections():
    """Children drawn WITH replacement (repeated sibling tokens), large uniforms so that most tests
    reject: every repeated token is tested again (ratio 0 by then) and costs one more residual round."""
    rng = np.random.default_rng(3)
    V, n = 96, 14
    parent = W.star_tree(n)
    checked = 0
    for trial in range(25):
        tl = (2 * rng.standard_normal((n, V))).astype(np.float32)
        dl = (tl + 1.5 * rng.standard_normal((n, V))).astype(np.float32)
        q = np.exp((dl[0] - dl[0].max()) / 0.8)
        tokens = np.zeros(n, np.int32)
        tokens[1:] = rng.choice(V, n - 1, replace=True, p=q / q.sum())  # repeats are likely with 13 draws
        if trial == 0:
            tokens[2] = tokens[1]
        u = (0.85 + 0.15 * rng.random(n + 1)).astype(np.float32)
        u[-1] = rng.random()
        vi = W.VerifyInputs(torch.from_numpy(parent), torch.from_numpy(tokens), torch.from_numpy(tl),
                            torch.from_numpy(dl), torch.from_numpy(u), 0.8)
        checked += G.check_verify(vi, specinfer=True) == "ok"
        # the two variants are different algorithms: on these inputs they must not be interchangeable
    assert checked >= 20
    ref_a = O.tree_verify(parent, tokens, tl, dl, 0.8, u, variant=O.VARIANT_SEQUOIA)
    ref_b = O.tree_verify(parent, tokens, tl, dl, 0.8, u, variant=O.VARIANT_SPECINFER)
    assert np.abs(ref_a["residual"] - ref_b["residual"]).max() > 1e-4 or ref_a["path"].tolist() != ref_b["path"].tolist()


@pytest.mark.parametrize("name,T,seeds", [("tiny", 0.6, range(8)), ("llama2-7b", 0.6, range(4)), ("llama2-7b", 1.0, range(3)),
                                          ("llama2-13b", 1.0, range(2)), ("llama3-70b", 0.6, range(1))])
def test_verify_target_sample_configs(name, T, seeds):
    """SEQ_VERIFY_TARGET_SAMPLE (Section 2.2, naive / top-k sampling): the walk that samples from the target at
    every node, against the oracle's; no draft row is passed."""
    cfg = W.CONFIGS[name]
    outcomes = [G.check_verify_target_sample(W.make_verify_inputs(cfg, T, seed)) for seed in seeds]
    assert outcomes.count("ok") >= max(1, len(outcomes) - 1), outcomes


@pytest.mark.parametrize("name,T,vocab", [("tiny", 0.6, None), ("llama2-7b", 1.0, None), ("llama2-7b", 0.3, 5003)])
def test_verify_target_sample_deep_walks(name, T, vocab):
    """Children carrying exactly the token that is drawn at their parent: the walk follows them to a leaf, one
    cluster-wide draw per level, and the bonus is the leaf's own draw.  (Vocabulary 5003: ragged slices.)"""
    cfg = W.CONFIGS[name]
    ok = 0
    for seed in range(3):
        vi = W.make_verify_inputs(cfg, T, seed, vocab=vocab)
        assert G.steer_tokens_to_samples(vi) > 1
        ref = O.tree_verify_target_sample(vi.parent, vi.tokens, vi.target_logits, vi.temperature, vi.uniforms)
        assert ref["path_len"] >= 3  # the steering worked: root, its first child, that child's first child ...
        ok += G.check_verify_target_sample(vi, with_draft=(seed == 1)) == "ok"
    assert ok >= 2


def test_verify_target_sample_greedy_is_argmax_matching():
    """T = 0 with the flag set: the arg-max matching of the default mode (the draw degenerates to the arg-max)."""
    vi = W.make_verify_inputs(W.CONFIGS["tiny"], 0.0, 2)
    a = G.run_verify(vi, target_sample=True)
    b = G.run_verify(vi)
    ref = O.tree_verify_target_sample(vi.parent, vi.tokens, vi.target_logits, 0.0, vi.uniforms)
    assert a["path"].tolist() == b["path"].tolist() == ref["path"].tolist()
    assert a["bonus"] == b["bonus"] == ref["bonus"] and a["status"] == 0
    assert np.array_equal(a["residual"], ref["residual"])


def test_verify_nonfinite_logits_are_flagged_not_trapped():
    vi = W.make_verify_inputs(W.CONFIGS["tiny"], 0.6, 0, vocab=512)
    vi.target_logits[0, 5] = float("nan")
    got = G.run_verify(vi)
    assert got["status"] & B.SEQ_DEV_NONFINITE and 0 <= got["bonus"] < 512 and got["path_len"] >= 1


# ---------------------------------------------------------------- tensor-core attention kernel ------
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("n,L,Hq,Hkv", [(1, 0, 2, 2), (1, 77, 2, 1), (5, 0, 4, 2), (17, 33, 4, 4), (64, 128, 2, 2),
                                        (100, 129, 8, 2), (130, 1000, 4, 4), (257, 5, 16, 1), (40, 300, 128, 1)])
def test_tensor_core_attention_edge_sizes(dtype, n, L, Hq, Hkv):
    cfg = _cfg("tiny", num_q_heads=Hq, num_kv_heads=Hkv, prefix_len=L, n_tree=n, max_depth=12)
    G.check_attention(W.make_attention_inputs(cfg, 7, dtype=dtype), kernel=B.KERNEL_TENSOR_CORE)


@pytest.mark.parametrize("tree", ["chain", "star"])
def test_tensor_core_attention_chain_and_star(tree):
    cfg = _cfg("tiny", num_q_heads=4, num_kv_heads=2, prefix_len=200, n_tree=160)
    parent = W.chain_tree(160) if tree == "chain" else W.star_tree(160)
    G.check_attention(W.make_attention_inputs(cfg, 3, parent=parent, dtype="bf16"), kernel=B.KERNEL_TENSOR_CORE)


def test_tensor_core_attention_masked_keys_are_exactly_zero_and_nan_tail_is_never_read():
    cfg = _cfg("tiny", num_q_heads=4, num_kv_heads=2, prefix_len=96, n_tree=150, max_depth=12)
    ai = W.make_attention_inputs(cfg, 5, dtype="bf16", extra_capacity=200)  # NaN rows past L+n
    base, lse, st = G.run_attention(ai, kernel=B.KERNEL_TENSOR_CORE)
    assert st == 0 and torch.isfinite(base).all() and torch.isfinite(lse).all()
    G.check_attention(ai, kernel=B.KERNEL_TENSOR_CORE)
    M, _, _ = O.mask_from_parents(ai.parent)
    n, L = 150, 96
    for i in (0, 31, 77, 149):
        k2, v2 = ai.k_cache.clone(), ai.v_cache.clone()
        for a in range(n):
            if not (M[i, a >> 5] >> (a & 31)) & 1:
                k2[:, L + a] = 1e4 * (-1) ** a
                v2[:, L + a] = -1e4
        out2, lse2, _ = G.run_attention(dataclasses.replace(ai, k_cache=k2, v_cache=v2), kernel=B.KERNEL_TENSOR_CORE)
        assert torch.equal(out2[i], base[i]) and torch.equal(lse2[:, i], lse[:, i])


def test_tensor_core_attention_garbage_in_unused_mask_words_is_ignored():
    cfg = _cfg("tiny", num_q_heads=2, num_kv_heads=2, prefix_len=50, n_tree=70)
    ai = W.make_attention_inputs(cfg, 8, dtype="bf16", extra_capacity=64, tail_fill=1.0)
    d = G.dev()
    mask, _, _ = G.gpu_mask(ai.parent.numpy())
    wide = torch.full((70, 6), -1, dtype=torch.int32, device=d)  # all-ones beyond the 3 live words
    wide[:, :3] = mask
    wide[:, 2] |= torch.tensor(-(1 << 6), dtype=torch.int32, device=d)  # bits 70..95 set too
    for kernel in (B.KERNEL_TENSOR_CORE, B.KERNEL_CUDA_CORE):
        out = B.seq_tree_attention(ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d), wide, 50, kernel=kernel)
        torch.cuda.synchronize()
        ref, _, _ = O.tree_attention(ai.q, ai.k_cache, ai.v_cache, ai.parent, 50)
        assert np.abs(out.double().cpu().numpy() - ref).max() < 2e-2


def test_tensor_core_attention_large_magnitude_scores_rescale_path():
    """Scores that grow block after block force the accumulator rescale in tensor memory."""
    cfg = _cfg("tiny", num_q_heads=2, num_kv_heads=2, prefix_len=700, n_tree=64)
    ai = W.make_attention_inputs(cfg, 9, dtype="bf16")
    ramp = torch.linspace(0.2, 6.0, 764).view(1, -1, 1)
    k = (ai.k_cache.float() * ramp).to(torch.bfloat16)
    G.check_attention(dataclasses.replace(ai, k_cache=k), kernel=B.KERNEL_TENSOR_CORE)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("n,L,Hq,Hkv", [(300, 200, 64, 8),    # 19 tiles x 8 heads, tiles about as long as a CTA's range
                                        (600, 100, 32, 2),    # 75 tiles per head (three per lane in the prefix scan)
                                        (1024, 40, 24, 6),    # maximum tree, 32 tiles x 6 heads, ragged last blocks
                                        (150, 3000, 128, 16)])  # 10 tiles x 16 heads, long prefix: tiles cut in three
def test_tensor_core_attention_stream_mode(dtype, n, L, Hq, Hkv):
    """More (tile, kv head) units than SMs: CTAs take equal ranges of the flattened block space and tiles cut
    by a range boundary are completed from workspace pieces.  All rows against the oracle, then repeated
    calls on the same workspace (the arrival counters must have been left at zero), bit for bit."""
    cfg = _cfg("tiny", num_q_heads=Hq, num_kv_heads=Hkv, prefix_len=L, n_tree=n, max_depth=14)
    ai = W.make_attention_inputs(cfg, 11, dtype=dtype)
    d = G.dev()
    mask, _, st = G.gpu_mask(ai.parent.numpy())
    lse = torch.empty((Hq, n), dtype=torch.float32, device=d)
    call = B.AttentionCall(ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d), mask, L, lse=lse, dev_status=st,
                           kernel=B.KERNEL_TENSOR_CORE_STREAM)
    assert call.workspace_bytes_needed > 0, "the stream schedule was asked for"
    first = call.run().clone()
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    ref, rlse, _ = O.tree_attention(ai.q, ai.k_cache, ai.v_cache, ai.parent, L)
    assert np.abs(first.double().cpu().numpy() - ref).max() < G.ATTN_TOL[ai.q.dtype]
    assert np.abs(lse.double().cpu().numpy() - rlse).max() < 2e-2
    # Repeated calls, each after a large fill that empties the L2 and shifts the order in which the CTAs
    # finish their pieces: the result may not depend on which CTA completes a tile.
    junk = torch.empty(160 << 20, dtype=torch.uint8, device=d)
    for it in range(12):
        junk.fill_(it)
        again = call.run()
        if it % 2:
            again = call.run()  # and back to back
        torch.cuda.synchronize()
        assert int(st.item()) == 0 and torch.equal(first, again), f"call {it} differs from the first"


@pytest.mark.parametrize("n,L,Hq,Hkv,tree", [(1, 0, 2, 2, "random"), (17, 33, 4, 4, "random"), (64, 1024, 32, 32, "random"),
                                             (130, 1000, 4, 4, "chain"), (257, 5, 16, 1, "star"), (1024, 40, 24, 6, "random"),
                                             (768, 4096, 64, 8, "random")])
def test_tensor_core_attention_mask_from_parent_array(n, L, Hq, Hkv, tree):
    """mask_bits = NULL, parent given: the kernel walks the parent array itself.  Same bits as with the mask
    of seq_tree_mask_from_parents (grid mode with and without clusters, and stream mode)."""
    cfg = _cfg("tiny", num_q_heads=Hq, num_kv_heads=Hkv, prefix_len=L, n_tree=n, max_depth=14)
    parent = {"random": None, "chain": W.chain_tree(n), "star": W.star_tree(n)}[tree]
    ai = W.make_attention_inputs(cfg, 13, parent=parent, dtype="bf16")
    d = G.dev()
    q, k, v, par = ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d), ai.parent.to(d)
    mask, _, _ = G.gpu_mask(ai.parent.numpy())
    st = torch.zeros(1, dtype=torch.int32, device=d)
    with_mask = B.seq_tree_attention(q, k, v, mask, L, kernel=B.KERNEL_TENSOR_CORE).clone()
    lse = torch.empty((Hq, n), dtype=torch.float32, device=d)
    fused = B.seq_tree_attention(q, k, v, None, L, parent=par, lse=lse, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and torch.equal(with_mask, fused)
    # both schedules of the kernel, whichever of them the shape gets by default: same bits with either mask source
    # (between the schedules the key range is cut differently, so the rounding differs: oracle tolerance)
    for forced in (B.KERNEL_TENSOR_CORE_STREAM, B.KERNEL_TENSOR_CORE_GRID):
        a = B.seq_tree_attention(q, k, v, mask, L, kernel=forced)
        b = B.seq_tree_attention(q, k, v, None, L, parent=par, kernel=forced, dev_status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0 and torch.equal(a, b)
        assert (a.float() - fused.float()).abs().max().item() < 2e-2
    if n <= 300:
        ref, rlse, _ = O.tree_attention(ai.q, ai.k_cache, ai.v_cache, ai.parent, L)
        assert np.abs(fused.double().cpu().numpy() - ref).max() < 2e-2
        assert np.abs(lse.double().cpu().numpy() - rlse).max() < 2e-2


def test_attention_mask_from_parent_array_bad_parent_and_unsupported():
    cfg = _cfg("tiny", num_q_heads=4, num_kv_heads=2, prefix_len=40, n_tree=50)
    ai = W.make_attention_inputs(cfg, 14, dtype="bf16")
    d = G.dev()
    q, k, v = ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d)
    bad = ai.parent.clone()
    bad[20] = 35   # a later node: flagged, read as "no parent"
    bad[30] = -7
    st = torch.zeros(1, dtype=torch.int32, device=d)
    fused = B.seq_tree_attention(q, k, v, None, 40, parent=bad.to(d), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) & B.SEQ_DEV_BAD_PARENT
    st2 = torch.zeros(1, dtype=torch.int32, device=d)
    mask, _ = B.seq_tree_mask_from_parents(bad.to(d), dev_status=st2)   # same reading of the bad entries
    assert torch.equal(fused, B.seq_tree_attention(q, k, v, mask, 40, kernel=B.KERNEL_TENSOR_CORE))
    # the CUDA-core kernel needs mask_bits
    with pytest.raises(B.SeqTreeError) as e:
        B.seq_tree_attention(q, k, v, None, 40, parent=ai.parent.to(d), kernel=B.KERNEL_CUDA_CORE)
    assert e.value.code == B.SEQ_ERR_UNSUPPORTED
    with pytest.raises(B.SeqTreeError) as e:
        B.seq_tree_attention(q.float(), k.float(), v.float(), None, 40, parent=ai.parent.to(d))
    assert e.value.code == B.SEQ_ERR_UNSUPPORTED


@pytest.mark.parametrize("name,rows", [("llama2-7b", [0, 1, 13, 40, 63]), ("llama2-13b", [0, 5, 64, 127]),
                                       ("vicuna-33b", [0, 100, 128, 255]), ("llama3-70b", [0, 31, 32, 400, 767])])
def test_attention_full_size_configs_sampled_rows(name, rows):
    """The full workload sizes, in the launch configuration the benchmark times; the oracle recomputes the
    sampled nodes (and their ancestors) one by one."""
    cfg = W.CONFIGS[name]
    ai = W.make_attention_inputs(cfg, 0)
    G.check_attention(ai, rows=rows)


# ---------------------------------------------------------------- trees from the dynamic program ----
def _dp_parent(cfg):
    parent, _ = B.seq_tree_build(W.PAPER_ACCEPTANCE_VECTOR, cfg.n_tree, cfg.max_depth, cfg.max_fanout or 31)
    assert len(parent) == cfg.n_tree
    return parent


@pytest.mark.parametrize("name", ["tiny", "llama2-7b", "llama2-13b", "vicuna-33b"])
def test_attention_on_dp_shaped_trees(name):
    """Trees from seq_tree_build on the paper's acceptance vector (wide near the root, long first-child chains):
    attention with the mask given and with the mask derived in the kernel, against the oracle."""
    cfg = W.CONFIGS[name]
    parent = _dp_parent(cfg)
    ai = W.make_attention_inputs(cfg, 0, parent=parent)
    G.check_attention(ai)
    out, _, st = G.run_attention(ai)
    d = G.dev()
    fused = B.seq_tree_attention(ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d), None, ai.prefix_len,
                                 parent=ai.parent.to(d))
    torch.cuda.synchronize()
    assert st == 0 and torch.equal(fused, out)


def test_attention_on_the_768_node_dp_tree_sampled_rows():
    cfg = W.CONFIGS["llama3-70b"]
    parent = _dp_parent(cfg)
    ai = W.make_attention_inputs(cfg, 0, parent=parent)
    depth = np.zeros(len(parent), int)
    for i in range(1, len(parent)):
        depth[i] = depth[parent[i]] + 1
    rows = [0, 1, 63, 64, 300, 767, int(np.argmax(depth))]
    G.check_attention(ai, rows=rows)


@pytest.mark.parametrize("name,T", [("tiny", 0.6), ("llama2-7b", 0.6), ("llama2-7b", 1.0), ("llama2-13b", 1.0), ("llama3-70b", 0.6)])
def test_verify_on_dp_shaped_trees(name, T):
    cfg = W.CONFIGS[name]
    parent = _dp_parent(cfg)
    outcomes = []
    for seed in range(3 if cfg.vocab < 100000 else 1):
        vi = W.make_verify_inputs(cfg, T, seed, parent=parent)
        outcomes.append(G.check_verify(vi))
        outcomes.append(G.check_verify_target_sample(vi))
    assert outcomes.count("ok") >= len(outcomes) - 1, outcomes


# ---------------------------------------------------------------- batched verification --------------
@pytest.mark.parametrize("name,T,R,mode", [("tiny", 0.6, 5, "sequoia"), ("llama2-7b", 0.6, 20, "sequoia"), ("llama2-7b", 1.0, 7, "specinfer"),
                                           ("llama2-7b", 0.6, 6, "target"), ("llama2-7b", 0.0, 4, "sequoia"),
                                           ("llama3-70b", 0.6, 3, "sequoia")])  # (up to 9 requests: one cluster of 16 each, rows in registers)
def test_verify_batch_equals_one_request_at_a_time(name, T, R, mode):
    """R requests (own tree, tokens, logits, uniforms) in one launch: every request's path, bonus and residual are
    the oracle's, and equal (to rounding) to what a launch of its own returns."""
    cfg = W.CONFIGS[name]
    d = G.dev()
    vis = [W.make_verify_inputs(cfg, T, seed) for seed in range(R)]
    stack = lambda f: torch.stack([f(v) for v in vis]).to(d)
    parent, tokens = stack(lambda v: v.parent), stack(lambda v: v.tokens)
    tl, dl, un = stack(lambda v: v.target_logits), stack(lambda v: v.draft_logits), stack(lambda v: v.uniforms)
    n, V = cfg.n_tree, cfg.vocab
    resid = torch.full((R, V), float("nan"), dtype=torch.float32, device=d)
    nxt = torch.full((R, n), -9, dtype=torch.int32, device=d)
    st = torch.zeros(1, dtype=torch.int32, device=d)
    path, plen, bonus = B.seq_tree_verify_batch(parent, tokens, tl, None if mode == "target" else dl, T, un, residual_out=resid,
                                                next_child_out=nxt, dev_status=st, specinfer=mode == "specinfer",
                                                target_sample=mode == "target")
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    checked = 0
    for r, vi in enumerate(vis):
        # (a single request may run on a larger cluster than a request of a batch: the vocabulary-wide sums are then
        # rounded differently, so the two agree to rounding, and exactly wherever the oracle's decision is clear)
        one = G.run_verify(vi, specinfer=mode == "specinfer", target_sample=mode == "target")
        k = int(plen[r].item())
        if mode == "target":
            ref = O.tree_verify_target_sample(vi.parent, vi.tokens, vi.target_logits, T, vi.uniforms)
        else:
            ref = O.tree_verify(vi.parent, vi.tokens, vi.target_logits, vi.draft_logits, T, vi.uniforms,
                                variant=O.VARIANT_SPECINFER if mode == "specinfer" else O.VARIANT_SEQUOIA)
        if ref["min_gap"] < G.GAP:
            continue
        assert path[r, :k].cpu().tolist() == one["path"].tolist() == ref["path"].tolist()
        assert np.array_equal(nxt[r].cpu().numpy(), one["next_child"])
        got = resid[r].double().cpu().numpy()
        assert np.abs(got - one["residual"]).max() < 1e-6 and np.abs(got - ref["residual"]).max() < G.RESID_TOL
        if one["bonus"] == ref["bonus"]:
            assert int(bonus[r].item()) == ref["bonus"] or T > 0  # (the bonus draw has its own rounding band)
            checked += int(bonus[r].item()) == ref["bonus"]
    assert checked >= R - 2


# ---------------------------------------------------------------- a batch of requests in one attention launch ----
@pytest.mark.parametrize("name,R", [("tiny", 3), ("llama2-7b", 5), ("llama3-70b", 2)])
def test_attention_batch_of_requests_as_stacked_heads(name, R):  # (llama2-7b x 5: 160 units in two waves of the grid schedule)
    """Requests that share the tree and the prefix length (Sequoia's tree is fixed in advance) go through one launch
    as R times the heads: q laid out [n, R, Hq, d], the caches concatenated along the kv-head axis.  Every request's
    rows against the oracle on that request alone."""
    cfg = W.CONFIGS[name]
    d = G.dev()
    parent = W.make_tree(cfg, 0)
    ais = [W.make_attention_inputs(cfg, seed, parent=parent) for seed in range(R)]
    n, Hq = cfg.n_tree, cfg.num_q_heads
    q = torch.stack([a.q for a in ais], dim=1).reshape(n, R * Hq, cfg.head_dim).contiguous().to(d)
    k = torch.cat([a.k_cache for a in ais], dim=0).contiguous().to(d)
    v = torch.cat([a.v_cache for a in ais], dim=0).contiguous().to(d)
    st = torch.zeros(1, dtype=torch.int32, device=d)
    out = B.seq_tree_attention(q, k, v, None, cfg.prefix_len, parent=torch.from_numpy(parent).to(d), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    out = out.view(n, R, Hq, cfg.head_dim)
    rows = None if n <= 64 else [0, 1, n // 2, n - 1]
    for r, ai in enumerate(ais):
        if rows is None:
            ref, _, _ = O.tree_attention(ai.q, ai.k_cache, ai.v_cache, ai.parent, ai.prefix_len)
            got = out[:, r].double().cpu().numpy()
        else:
            keep = sorted(set(int(a) for i in rows for a in G._path(parent, i)))
            idx = {a: j for j, a in enumerate(keep)}
            psub = np.array([-1 if parent[a] < 0 else idx[int(parent[a])] for a in keep], np.int32)
            L = ai.prefix_len
            sel = torch.tensor(list(range(L)) + [L + a for a in keep])
            ref, _, _ = O.tree_attention(ai.q[keep], ai.k_cache[:, sel], ai.v_cache[:, sel], psub, L)
            got = out[keep, r].double().cpu().numpy()
        assert np.abs(got - ref).max() < G.ATTN_TOL[ai.q.dtype]


@pytest.mark.parametrize("heads", [20, 24, 28, 40, 44])
def test_tensor_core_attention_clusters_of_odd_sizes(heads):
    """(tile, kv head) unit counts for which the plan takes clusters of 7, 6, 5 and 3 CTAs along the key range (the 16
    output slices of the merge do not divide evenly among them): sampled rows against the oracle, and repeated
    calls after L2-emptying fills bit for bit."""
    cfg = _cfg("llama2-13b", num_q_heads=heads, num_kv_heads=heads, prefix_len=2048, n_tree=128)
    ai = W.make_attention_inputs(cfg, 21, dtype="bf16")
    G.check_attention(ai, kernel=B.KERNEL_TENSOR_CORE, rows=[0, 1, 63, 64, 100, 127])
    d = G.dev()
    st = torch.zeros(1, dtype=torch.int32, device=d)
    call = B.AttentionCall(ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d), None, 2048, parent=ai.parent.to(d), dev_status=st)
    assert call.workspace_bytes_needed == 0  # a cluster per unit, not the stream schedule
    first = call.run().clone()
    junk = torch.empty(160 << 20, dtype=torch.uint8, device=d)
    for it in range(6):
        junk.fill_(it)
        again = call.run()
        torch.cuda.synchronize()
        assert int(st.item()) == 0 and torch.equal(first, again)
