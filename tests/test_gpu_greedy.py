"""Greedy decoding (T = 0) on the GPU against the oracle: the residual is the one-hot at the target arg-max (lowest index
on ties), a child is accepted iff its token is that arg-max, the bonus token is the arg-max of the last node visited;
draft logits and uniforms play no part (Algorithm 2 at temperature 0; Section 4.1 reports greedy decoding)."""
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


def _steer_to_argmax(vi, every=1):
    """Gives one child of every `every`-th internal node the target's arg-max token of its parent, so that walks are long."""
    parent = vi.parent.numpy()
    tgt = vi.target_logits.numpy()
    seen = set()
    for ch in range(1, len(parent)):
        p = int(parent[ch])
        if p in seen or p % every:
            continue
        seen.add(p)
        vi.tokens[ch] = int(np.argmax(tgt[p]))
    return vi


def _check(vi, bf16=False, expect_flags=0):
    got = G.run_verify(vi, bf16_logits=bf16)
    ref = O.tree_verify(vi.parent, vi.tokens, vi.target_logits, vi.draft_logits, 0.0, vi.uniforms)
    assert got["status"] == ref["flags"] == expect_flags, (got["status"], ref["flags"])
    assert got["path"].tolist() == ref["path"].tolist()
    assert got["bonus"] == ref["bonus"]
    assert np.array_equal(got["next_child"], ref["next_child"])
    assert np.array_equal(got["residual"], ref["residual"])  # a one-hot: exact
    return got


@pytest.mark.parametrize("name,seeds,every", [("tiny", 3, 1), ("llama2-7b", 3, 1), ("llama2-13b", 2, 2), ("vicuna-33b", 2, 1),
                                              ("llama3-70b", 2, 1)])
def test_greedy_walks_on_the_configs(name, seeds, every, verify_schedule):
    for seed in range(seeds):
        vi = _steer_to_argmax(W.make_verify_inputs(W.CONFIGS[name], 0.0, seed), every)
        got = _check(vi)
        if every == 1:
            assert got["path_len"] >= 3  # the steering worked: the walk went down the tree


@pytest.mark.parametrize("V", [1, 8, 9, 31, 33, 127, 129, 1000, 4097, 50257])
def test_greedy_ragged_vocabularies(V, verify_schedule):
    cfg = dataclasses.replace(W.CONFIGS["tiny"], vocab=V)
    _check(_steer_to_argmax(W.make_verify_inputs(cfg, 0.0, V)))


def test_greedy_ties_go_to_the_lowest_index(verify_schedule):
    cfg = dataclasses.replace(W.CONFIGS["tiny"], vocab=9000)
    vi = W.make_verify_inputs(cfg, 0.0, 1)
    top = float(vi.target_logits.max()) + 1.0
    for node, toks in ((0, (8999, 4097, 511)), (1, (4096, 4095)), (2, (0, 8999))):  # equal maxima in different CTAs, warps and lanes
        for t in toks:
            vi.target_logits[node, t] = top
    vi.tokens[1] = 511    # node 1 is a child of the root: it carries the lowest of the root's tied maxima
    got = _check(vi)
    assert got["path"].tolist()[:2] == [0, 1]


def test_greedy_rows_without_a_finite_logit_and_nonfinite_logits(verify_schedule):
    cfg = dataclasses.replace(W.CONFIGS["tiny"], vocab=3000)
    vi = W.make_verify_inputs(cfg, 0.0, 2)
    vi.target_logits[0, :] = float("-inf")       # arg-max of an all -inf row: token 0
    vi.tokens[1] = 0
    got = _check(vi)
    assert got["path"].tolist()[:2] == [0, 1]
    vi = W.make_verify_inputs(cfg, 0.0, 3)
    vi.target_logits[0, 7] = float("nan")        # never the arg-max
    vi.target_logits[0, 2999] = float("inf")     # the largest finite value: the arg-max
    vi.tokens[1] = 2999
    got = _check(vi, expect_flags=B.SEQ_DEV_NONFINITE)
    assert got["path"].tolist()[:2] == [0, 1]


def test_greedy_bad_tokens_before_and_after_the_match(verify_schedule):
    cfg = dataclasses.replace(W.CONFIGS["tiny"], vocab=2048, n_tree=12, max_depth=3, max_fanout=8)
    vi = W.make_verify_inputs(cfg, 0.0, 4, parent=np.array([-1, 0, 0, 0, 0, 1, 1, 2, 2, 3, 3, 4], np.int32))
    g0 = int(np.argmax(vi.target_logits[0].numpy()))
    vi.tokens[1], vi.tokens[2], vi.tokens[3], vi.tokens[4] = 7, g0, -5, 99999   # the bad ones come after the match: not reported
    _check(vi, expect_flags=0)
    vi.tokens[1] = 2048                                                          # ... and one before it: reported
    _check(vi, expect_flags=B.SEQ_DEV_BAD_TOKEN)
    vi.tokens[2] = 8                                                             # no match at all: every child is looked at
    vi.tokens[1] = 7
    _check(vi, expect_flags=B.SEQ_DEV_BAD_TOKEN)


def test_greedy_single_node_chain_star_and_repeated_tokens(verify_schedule):
    cfg = dataclasses.replace(W.CONFIGS["tiny"], vocab=777)
    for parent in ([-1], [-1, 0, 1, 2, 3, 4, 5], [-1, 0, 0, 0, 0, 0, 0, 0]):
        p = np.array(parent, np.int32)
        vi = _steer_to_argmax(W.make_verify_inputs(dataclasses.replace(cfg, n_tree=len(p)), 0.0, len(p), parent=p))
        _check(vi)
    p = np.array([-1, 0, 0, 0, 1, 2, 3], np.int32)   # three children of the root carry the arg-max: the first is taken
    vi = W.make_verify_inputs(dataclasses.replace(cfg, n_tree=7), 0.0, 9, parent=p)
    g0 = int(np.argmax(vi.target_logits[0].numpy()))
    vi.tokens[1] = 3
    vi.tokens[2] = vi.tokens[3] = g0
    got = _check(vi)
    assert got["path"].tolist()[:2] == [0, 2]


@pytest.mark.parametrize("name", ["llama2-7b", "llama3-70b"])
def test_greedy_on_bfloat16_logits(name):
    vi = W.make_verify_inputs(W.CONFIGS[name], 0.0, 5)
    vi.target_logits = vi.target_logits.to(torch.bfloat16).float()   # exact in bfloat16: the oracle sees the same values
    vi.draft_logits = vi.draft_logits.to(torch.bfloat16).float()
    _check(_steer_to_argmax(vi), bf16=True)
