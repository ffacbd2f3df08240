"""GPU parity of seq_tree_kv_commit against the oracle: byte-identical caches on the configs' shapes (several
planes, 16-bit and 32-bit rows, padded strides), long paths whose rows are both read and overwritten, invalid
paths, and the whole chain verify -> commit -> attention over the committed prefix."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2402_12374_b200 import binding as B, workloads as W
from tests import gpu_util as G
from tests.gpu_util import steer_tokens_to_samples

pytestmark = pytest.mark.gpu


def _bytes_view(t: torch.Tensor) -> np.ndarray:
    """The exact bits of a cache tensor as an unsigned-integer numpy array of the same item size."""
    it = {1: torch.uint8, 2: torch.int16, 4: torch.int32}[t.element_size()]
    return t.contiguous().view(it).cpu().numpy()


def _random_cache(planes, rows, d, dtype, seed, row_pad=0):
    g = torch.Generator().manual_seed(seed)
    full = torch.randn((planes, rows, d + row_pad), generator=g).to(dtype)
    return full


def _commit_and_compare(k, v, L, n, path, *, row_pad=0):
    """k, v: CPU tensors [planes, rows, d(+pad)]; the first d columns are the cache proper (rows strided)."""
    dev = G.dev()
    d = k.shape[2] - row_pad
    kd, vd = k.to(dev), (v.to(dev) if v is not None else None)
    path_t = torch.full((n,), -7, dtype=torch.int32)
    path_t[: len(path)] = torch.as_tensor(path, dtype=torch.int32)
    plen = torch.tensor([len(path)], dtype=torch.int32)
    newL = torch.full((1,), -1, dtype=torch.int32, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    B.seq_tree_kv_commit(kd[:, :, :d], vd[:, :, :d] if vd is not None else None, L, n, path_t.to(dev), plen.to(dev),
                         new_prefix_len=newL, dev_status=st)
    torch.cuda.synchronize()
    flags = 0
    for host, devt in ((k, kd), (v, vd)):
        if host is None:
            continue
        ref, f = O.kv_commit(_bytes_view(host[:, :, :d]), L, n, np.asarray(path, np.int32))
        flags |= f
        assert np.array_equal(_bytes_view(devt[:, :, :d]), ref)
        if row_pad:  # the padding between rows is not touched
            assert np.array_equal(_bytes_view(devt[:, :, d:]), _bytes_view(host[:, :, d:]))
    assert int(st.item()) == flags
    assert int(newL.item()) == (L if flags else L + len(path))
    return flags


@pytest.mark.parametrize("name,layers", [("tiny", 2), ("llama2-7b", 3), ("llama3-70b", 5)])
def test_commit_of_verified_paths_on_config_shapes(name, layers):
    """Paths produced by the oracle's walk on the config's trees; cache planes = layers x kv heads."""
    cfg = W.CONFIGS[name]
    L, n = (cfg.prefix_len if name != "llama3-70b" else 512), cfg.n_tree
    planes = layers * cfg.num_kv_heads
    moved = 0
    for seed in range(3):
        vi = W.make_verify_inputs(cfg, cfg.temperatures[-1], seed, vocab=2048)
        steer_tokens_to_samples(vi)
        path = O.tree_verify_target_sample(vi.parent, vi.tokens, vi.target_logits, vi.temperature, vi.uniforms)["path"]
        k = _random_cache(planes, L + n + 5, cfg.head_dim, W.TORCH_DTYPES[cfg.dtype], 10 + seed)
        v = _random_cache(planes, L + n + 5, cfg.head_dim, W.TORCH_DTYPES[cfg.dtype], 20 + seed)
        assert _commit_and_compare(k, v, L, n, path) == 0
        moved += sum(int(p != i) for i, p in enumerate(path))
    assert moved > 0  # the paths really moved rows


@pytest.mark.parametrize("dtype,d,row_pad,with_v", [(torch.float32, 128, 0, True), (torch.float16, 8, 0, True),
                                                    (torch.bfloat16, 128, 8, True), (torch.bfloat16, 64, 0, False)])
def test_commit_row_sizes_strides_and_keys_only(dtype, d, row_pad, with_v):
    L, n, planes = 33, 40, 7
    path = [0, 1, 2, 5, 6, 9, 17, 18, 30, 39]
    k = _random_cache(planes, L + n, d, dtype, 1, row_pad)
    v = _random_cache(planes, L + n, d, dtype, 2, row_pad) if with_v else None
    assert _commit_and_compare(k, v, L, n, path, row_pad=row_pad) == 0


def test_commit_long_paths_read_and_overwrite_the_same_rows():
    """n = 1024, 500-node paths (every other node; a dense run followed by jumps): most rows are the source of
    one slot and the destination of a later one, across many load/store batches."""
    n, L, planes = 1024, 7, 3
    k = _random_cache(planes, L + n, 128, torch.bfloat16, 3)
    v = _random_cache(planes, L + n, 128, torch.bfloat16, 4)
    for path in (list(range(0, 1000, 2)), list(range(100)) + list(range(101, 1024, 3)), [0] + list(range(524, 1024)),
                 list(range(1024))):
        assert _commit_and_compare(k, v, L, n, path) == 0


@pytest.mark.parametrize("path", [[1, 2], [0, 2, 2], [0, 3, 2], [0, 16], [0, -1], []])
def test_commit_invalid_or_empty_path(path):
    """An invalid path is flagged and moves nothing; the empty path is valid and moves nothing."""
    k = _random_cache(4, 40, 128, torch.bfloat16, 5)
    flags = _commit_and_compare(k, k.clone(), 24, 16, path)
    assert flags == (0 if path == [] else B.SEQ_DEV_BAD_PATH)


def test_commit_path_len_above_tree_size_is_flagged():
    dev = G.dev()
    k = _random_cache(2, 40, 128, torch.bfloat16, 6).to(dev)
    before = k.clone()
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    B.seq_tree_kv_commit(k, None, 24, 16, torch.arange(16, dtype=torch.int32, device=dev),
                         torch.tensor([17], dtype=torch.int32, device=dev), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == B.SEQ_DEV_BAD_PATH and torch.equal(k, before)


def test_verify_commit_attention_chain_in_one_graph():
    """The whole inter-step sequence on the device, captured in one CUDA graph: verify writes path / path_len,
    the commit consumes them, and attention of the accepted nodes over the committed cache (a chain) returns what
    tree attention gave those nodes."""
    cfg = W.CONFIGS["llama2-7b"]
    dev = G.dev()
    ai = W.make_attention_inputs(cfg, 1)
    vi = W.make_verify_inputs(cfg, 0.6, 1, vocab=4096)
    vi.parent = ai.parent
    steer_tokens_to_samples(vi)
    n, L = cfg.n_tree, ai.prefix_len
    q, k, v = ai.q.to(dev), ai.k_cache.to(dev), ai.v_cache.to(dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    tree_out = B.seq_tree_attention(q, k, v, None, L, parent=ai.parent.to(dev), dev_status=st).clone()
    call = B.VerifyCall(vi.parent.to(dev), vi.tokens.to(dev), vi.target_logits.to(dev), None, 0.6, vi.uniforms.to(dev),
                        dev_status=st, target_sample=True)
    newL = torch.zeros(1, dtype=torch.int32, device=dev)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        call.run(s)  # warm-up outside the capture
        s.synchronize()
        k.copy_(ai.k_cache.to(dev))
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            call.run(s)
            B.seq_tree_kv_commit(k, v, L, n, call.path, call.path_len, new_prefix_len=newL, dev_status=st, stream=s)
        g.replay()
    torch.cuda.synchronize()
    ref = O.tree_verify_target_sample(vi.parent, vi.tokens, vi.target_logits, 0.6, vi.uniforms)
    assert ref["min_gap"] >= G.GAP, "the seed was chosen so that no draw falls inside the rounding band"
    path = ref["path"]
    m = len(path)
    assert m >= 3 and int(newL.item()) == L + m and int(st.item()) == 0
    assert call.path[:m].cpu().tolist() == path.tolist()
    chain = torch.arange(-1, m - 1, dtype=torch.int32, device=dev)
    q_path = q[torch.as_tensor(path, dtype=torch.long, device=dev)].contiguous()
    chain_out = B.seq_tree_attention(q_path, k, v, None, L, parent=chain, dev_status=st)
    torch.cuda.synchronize()
    want = tree_out[torch.as_tensor(path, dtype=torch.long, device=dev)]
    assert (chain_out.float() - want.float()).abs().max().item() < 2e-2
    assert int(st.item()) == 0


def test_whole_step_replayed_from_one_graph_while_the_prefix_grows():
    """Attention -> verification -> commit captured ONCE, with the prefix length in device memory, and replayed three
    times: every replay sees the prefix that the previous one's commit left, and is checked against the oracle
    (attention of the tree at its new rows, the walk, the committed cache bytes, the new length).  Section 4.1: the
    tree is fixed in advance so that CUDA graphs can remove the launch overhead."""
    import dataclasses

    from paper_2402_12374_b200 import workloads as W

    d = G.dev()
    n, L0, cap, Hq, Hkv, V, T = 48, 200, 512, 8, 4, 2048, 0.8
    cfg = dataclasses.replace(W.CONFIGS["tiny"], num_q_heads=Hq, num_kv_heads=Hkv, prefix_len=L0, n_tree=n, max_depth=8, max_fanout=4)
    ai = W.make_attention_inputs(cfg, 3, dtype="bf16", extra_capacity=cap - L0 - n, tail_fill=0.0)
    rng = np.random.default_rng(11)
    k_h = torch.from_numpy(rng.standard_normal((Hkv, cap, 128)).astype(np.float32)).to(torch.bfloat16)  # every row holds
    v_h = torch.from_numpy(rng.standard_normal((Hkv, cap, 128)).astype(np.float32)).to(torch.bfloat16)  # finite values
    vi = W.make_verify_inputs(cfg, T, 3, parent=ai.parent.numpy(), vocab=V)
    q, kc, vc, parent = ai.q.to(d), k_h.to(d), v_h.to(d), ai.parent.to(d)
    L_dev = torch.tensor([L0], dtype=torch.int32, device=d)
    L_new = torch.zeros(1, dtype=torch.int32, device=d)
    st = torch.zeros(1, dtype=torch.int32, device=d)
    uniforms = vi.uniforms.to(d).clone()
    bound = cap - n
    attn = B.AttentionCall(q, kc, vc, None, bound, parent=parent, dev_status=st, prefix_len_dev=L_dev)
    ver = B.VerifyCall(parent, vi.tokens.to(d), vi.target_logits.to(d), vi.draft_logits.to(d), T, uniforms, dev_status=st)
    stream = torch.cuda.Stream()

    def step():
        attn.run(stream)
        ver.run(stream)
        B.seq_tree_kv_commit(kc, vc, bound, n, ver.path, ver.path_len, new_prefix_len=L_new, dev_status=st, stream=stream,
                             prefix_len_dev=L_dev)
        L_dev.copy_(L_new, non_blocking=True)

    with torch.cuda.stream(stream):
        step()  # warm-up outside the graph, then everything back to the start
        stream.synchronize()
        kc.copy_(k_h); vc.copy_(v_h); L_dev.fill_(L0)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            step()
    k_ref, v_ref, L = k_h.clone(), v_h.clone(), L0
    for it in range(3):
        u = rng.random(n + 1).astype(np.float32)
        uniforms.copy_(torch.from_numpy(u))
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        # the oracle on the cache as this replay found it
        ref, _, _ = O.tree_attention(ai.q, k_ref[:, :L + n], v_ref[:, :L + n], ai.parent, L)
        assert np.abs(attn.out.double().cpu().numpy() - ref).max() < 2e-2, f"replay {it}: attention"
        rv = O.tree_verify(vi.parent, vi.tokens, vi.target_logits, vi.draft_logits, T, u)
        plen = int(ver.path_len.item())
        if rv["min_gap"] >= 1e-5:
            assert ver.path[:plen].cpu().tolist() == rv["path"].tolist(), f"replay {it}: path"
        host_path = ver.path[:plen].cpu().numpy()
        for ref_c, got in ((k_ref, kc), (v_ref, vc)):
            want, flags = O.kv_commit(ref_c.view(torch.int16).numpy(), L, n, host_path)
            assert flags == 0 and np.array_equal(got.view(torch.int16).cpu().numpy(), want), f"replay {it}: cache"
            ref_c.copy_(torch.from_numpy(want).view(torch.bfloat16))
        L += plen
        assert int(L_dev.item()) == L == int(L_new.item())
    assert L > L0 + 2  # the prefix did grow (the root alone is a path of one)


def test_attention_reads_the_prefix_length_from_device_memory_on_every_kernel_path():
    """prefix_len_dev on the tensor-core kernel (grid schedule, with and without a cluster split, and the stream
    schedule) and on the CUDA-core kernel: the result is that of a call with the same length given on the host; a
    length outside [0, prefix_len] is flagged and clamped."""
    import dataclasses

    from paper_2402_12374_b200 import workloads as W

    d = G.dev()
    for (n, L, cap, Hq, Hkv, kernel) in [(64, 300, 700, 8, 8, B.KERNEL_TENSOR_CORE), (130, 1000, 1500, 4, 4, B.KERNEL_TENSOR_CORE),
                                         (300, 200, 900, 64, 8, B.KERNEL_TENSOR_CORE_STREAM), (40, 77, 300, 6, 2, B.KERNEL_CUDA_CORE)]:
        cfg = dataclasses.replace(W.CONFIGS["tiny"], num_q_heads=Hq, num_kv_heads=Hkv, prefix_len=L, n_tree=n, max_depth=12)
        ai = W.make_attention_inputs(cfg, 5, dtype="bf16", extra_capacity=cap - L - n)  # NaN past the tree's rows
        q, kc, vc, par = ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d), ai.parent.to(d)
        mask, _, _ = G.gpu_mask(ai.parent.numpy())
        st = torch.zeros(1, dtype=torch.int32, device=d)
        want = B.seq_tree_attention(q, kc, vc, mask, L, kernel=kernel, dev_status=st).clone()
        L_dev = torch.tensor([L], dtype=torch.int32, device=d)
        got = B.seq_tree_attention(q, kc, vc, mask, cap - n, kernel=kernel, dev_status=st, prefix_len_dev=L_dev)
        torch.cuda.synchronize()
        assert int(st.item()) == 0 and torch.isfinite(got).all()
        # (the launch is planned for the bound, so the key range may be cut differently: oracle tolerance, not bits)
        assert (got.float() - want.float()).abs().max().item() < 2e-2
        ref, _, _ = O.tree_attention(ai.q, ai.k_cache[:, :L + n], ai.v_cache[:, :L + n], ai.parent, L)
        assert np.abs(got.double().cpu().numpy() - ref).max() < 2e-2
        L_dev.fill_(cap)  # beyond the bound: flagged, clamped to it
        B.seq_tree_attention(q, kc, vc, mask, cap - n, kernel=kernel, dev_status=st, prefix_len_dev=L_dev)
        torch.cuda.synchronize()
        assert int(st.item()) == B.SEQ_DEV_BAD_LENGTH


@pytest.mark.parametrize("kernel,given_mask,heads_kv,group,n,lengths", [
    (B.KERNEL_AUTO, False, 2, 4, 40, (50, 300, 171)),       # the tensor-core kernel, mask from the parent array
    (B.KERNEL_AUTO, True, 2, 4, 40, (0, 64, 65)),           # ... with the mask given; an empty prefix among them
    (B.KERNEL_CUDA_CORE, True, 2, 4, 40, (50, 300, 171)),   # the CUDA-core kernel
    (B.KERNEL_AUTO, False, 40, 1, 130, (100, 37, 222, 160)),  # 320 (tile, kv head) units: more than SMs, still the grid schedule
])
def test_batch_of_requests_with_a_prefix_length_each(kernel, given_mask, heads_kv, group, n, lengths):
    """Requests stacked as heads, each with its own prefix length in device memory (the tree is common: Section 4.1 fixes
    it in advance): every request's rows against the oracle run on that request alone."""
    import dataclasses

    from paper_2402_12374_b200 import workloads as W

    d = G.dev()
    R, cap = len(lengths), max(lengths) + n + 24
    cfg = dataclasses.replace(W.CONFIGS["tiny"], num_q_heads=heads_kv * group, num_kv_heads=heads_kv, prefix_len=max(lengths),
                              n_tree=n, max_depth=9, max_fanout=5)
    parent = torch.from_numpy(W.make_tree(cfg, 7))
    rng = np.random.default_rng(17)
    q = torch.from_numpy(rng.standard_normal((n, R * heads_kv * group, 128)).astype(np.float32)).to(torch.bfloat16)
    k = torch.from_numpy(rng.standard_normal((R * heads_kv, cap, 128)).astype(np.float32)).to(torch.bfloat16)
    v = torch.from_numpy(rng.standard_normal((R * heads_kv, cap, 128)).astype(np.float32)).to(torch.bfloat16)
    st = torch.zeros(1, dtype=torch.int32, device=d)
    L_dev = torch.tensor(lengths, dtype=torch.int32, device=d)
    mask = G.gpu_mask(parent.numpy())[0] if given_mask else None
    call = B.AttentionCall(q.to(d), k.to(d), v.to(d), mask, max(lengths), parent=parent.to(d), dev_status=st,
                           prefix_len_dev=L_dev, kernel=kernel)
    call.run()
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    got = call.out.double().cpu().numpy()
    hq = heads_kv * group
    for r, L in enumerate(lengths):
        ref, _, _ = O.tree_attention(q[:, r * hq:(r + 1) * hq], k[r * heads_kv:(r + 1) * heads_kv, :L + n],
                                     v[r * heads_kv:(r + 1) * heads_kv, :L + n], parent, L)
        assert np.abs(got[:, r * hq:(r + 1) * hq] - ref).max() < 2e-2, f"request {r} (prefix {L})"


def test_per_request_lengths_are_refused_where_they_cannot_work():
    d = G.dev()
    q = torch.zeros((8, 6, 128), dtype=torch.bfloat16, device=d)
    kv = torch.zeros((6, 64, 128), dtype=torch.bfloat16, device=d)
    parent = torch.tensor([-1, 0, 0, 1, 1, 2, 2, 3], dtype=torch.int32, device=d)
    four = torch.zeros(4, dtype=torch.int32, device=d)   # 4 does not divide 6 kv heads
    with pytest.raises(Exception):
        B.AttentionCall(q, kv, kv.clone(), None, 16, parent=parent, prefix_len_dev=four).run()
    three = torch.zeros(3, dtype=torch.int32, device=d)
    with pytest.raises(Exception):  # the stream schedule works on ranges that cross kv heads
        B.AttentionCall(q, kv, kv.clone(), None, 16, parent=parent, prefix_len_dev=three, kernel=B.KERNEL_TENSOR_CORE_STREAM).run()
