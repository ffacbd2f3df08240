"""The whole step fed from pinned host buffers (`binding.HostStep`): every variant of how the inputs travel — one
stream or two, the whole cache or only the tree's rows — must return what the oracle computes (Section 2.2: one
target pass over the tree, then the walk of Algorithm 2 from the root)."""
from __future__ import annotations

import dataclasses

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2402_12374_b200 import binding as B
from paper_2402_12374_b200 import workloads as W
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("resident_cache", [False, True])
@pytest.mark.parametrize("two_streams", [False, True])
def test_host_step_matches_the_oracle(resident_cache, two_streams):
    d = G.dev()
    cfg = dataclasses.replace(W.CONFIGS["tiny"], num_q_heads=8, num_kv_heads=4, prefix_len=300, n_tree=40, max_depth=8, max_fanout=4)
    T, V = 0.7, 4096
    ai = W.make_attention_inputs(cfg, 5, dtype="bf16")
    vi = W.make_verify_inputs(cfg, T, 5, parent=ai.parent.numpy(), vocab=V)
    hs = B.HostStep(ai.q, ai.k_cache, ai.v_cache, ai.parent, cfg.prefix_len, vi.tokens, vi.target_logits, vi.draft_logits, T,
                    vi.uniforms, device=d, fused_mask=True, resident_cache=resident_cache, two_streams=two_streams)
    full = sum(t.numel() * t.element_size() for t in hs.host_in)
    assert hs.h2d_bytes == full if not resident_cache else hs.h2d_bytes < full
    stream = torch.cuda.Stream()
    ref, _, _ = O.tree_attention(ai.q, ai.k_cache, ai.v_cache, ai.parent, cfg.prefix_len)
    rng = np.random.default_rng(2)
    for it in range(3):  # a new tree row content and new uniforms every step: nothing may be left over from the last one
        if it > 0:
            rows = slice(cfg.prefix_len, cfg.prefix_len + cfg.n_tree)
            hs.host_in[1][:, rows] = torch.from_numpy(rng.standard_normal((4, cfg.n_tree, 128)).astype(np.float32)).to(torch.bfloat16)
            hs.host_in[7].copy_(torch.from_numpy(rng.random(cfg.n_tree + 1).astype(np.float32)))
            ref, _, _ = O.tree_attention(hs.host_in[0], hs.host_in[1], hs.host_in[2], ai.parent, cfg.prefix_len)
        out, path, path_len, bonus = hs.run(stream)
        stream.synchronize()
        assert int(hs.status.item()) == 0
        assert np.abs(out.double().numpy() - ref).max() < 2e-2, f"step {it}: attention"
        rv = O.tree_verify(vi.parent, vi.tokens, vi.target_logits, vi.draft_logits, T, hs.host_in[7].numpy())
        if rv["min_gap"] >= 1e-5:
            plen = int(path_len.item())
            assert path[:plen].tolist() == rv["path"].tolist(), f"step {it}: path"
            assert int(bonus.item()) == rv["bonus"], f"step {it}: bonus token"
