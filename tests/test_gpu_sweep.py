"""A seeded sweep over shapes nobody picked by hand: head counts, group sizes, prefix lengths, tree sizes, vocabulary
sizes and temperatures drawn at random, every case compared with the oracle element by element (attention: Section 1,
one target pass over the tree with each token seeing the prefix and its ancestors; verification: Algorithm 2 walked
from the root, Section 2.2).  The hand-picked cases of the other files cover the edges; this one covers the middle,
where a wrong tile index or a wrong phase count would hide."""
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


def _random_cfg(rng, big_vocab=False):
    group = int(rng.choice([1, 1, 2, 4, 8]))
    hkv = int(rng.integers(1, 5))
    n = int(rng.integers(1, 520))
    L = int(rng.choice([0, int(rng.integers(1, 64)), int(rng.integers(64, 700))]))
    depth, fanout = int(rng.integers(2, 14)), int(rng.integers(1, 9))
    room = sum(min(fanout ** k, 1000) for k in range(depth))  # nodes a tree within these bounds can hold (root at depth 0)
    n = max(1, min(n, room // 2))                              # half of it, so that the random growth always finds a parent
    return dataclasses.replace(W.CONFIGS["tiny"], num_q_heads=hkv * group, num_kv_heads=hkv, prefix_len=L, n_tree=n,
                               max_depth=depth, max_fanout=fanout,
                               vocab=int(rng.integers(33, 9000 if not big_vocab else 70000)))


@pytest.mark.parametrize("case", range(40))
def test_attention_on_random_shapes(case):
    rng = np.random.default_rng(1000 + case)
    cfg = _random_cfg(rng)
    dtype = ["bf16", "fp16"][case % 2]
    ai = W.make_attention_inputs(cfg, case, dtype=dtype, extra_capacity=int(rng.integers(0, 40)))
    kernel = [B.KERNEL_AUTO, B.KERNEL_AUTO, 2, 1][case % 4]  # the default plan, the tensor-core kernel, the CUDA-core kernel
    G.check_attention(ai, kernel=kernel)


@pytest.mark.parametrize("case", range(8))
def test_attention_with_the_mask_from_the_parent_array_and_the_length_from_device_memory(case):
    """The same sweep through the two other ways in: no mask given (the kernel walks the parent array) and the prefix
    length read on the device with the host's value as its upper bound."""
    d = G.dev()
    rng = np.random.default_rng(2000 + case)
    cfg = _random_cfg(rng)
    slack = int(rng.integers(0, 100))
    ai = W.make_attention_inputs(cfg, case, dtype="bf16", extra_capacity=slack + 8, tail_fill=0.0)
    L, n = cfg.prefix_len, cfg.n_tree
    st = torch.zeros(1, dtype=torch.int32, device=d)
    L_dev = torch.tensor([L], dtype=torch.int32, device=d)
    call = B.AttentionCall(ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d), None, L + slack, parent=ai.parent.to(d),
                           dev_status=st, prefix_len_dev=L_dev)
    call.run()
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    ref, _, _ = O.tree_attention(ai.q, ai.k_cache[:, :L + n], ai.v_cache[:, :L + n], ai.parent, L)
    assert np.abs(call.out.double().cpu().numpy() - ref).max() < 2e-2


@pytest.mark.parametrize("verify_schedule", ["nodes", "walk"], indirect=True)
@pytest.mark.parametrize("case", range(40))
def test_verification_on_random_shapes(case, verify_schedule):
    rng = np.random.default_rng(3000 + case)
    cfg = _random_cfg(rng, big_vocab=case % 3 == 0)
    T = float(rng.choice([0.2, 0.6, 1.0, 1.7]))
    vi = W.make_verify_inputs(cfg, T, case)
    G.check_verify(vi, specinfer=case % 4 == 3)
