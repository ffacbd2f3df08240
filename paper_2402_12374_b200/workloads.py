"""Seeded synthetic inputs for the token-tree verification step.

This module only *generates inputs*: it holds none of the arithmetic of tree
attention or of Sequoia's verification, and both the CUDA path and the CPU
oracle are fed the very same bytes it returns.  Everything is drawn on the host
from ``numpy.random.Philox`` streams keyed by ``(BASE_SEED, config id, seed,
tensor id)`` and cast to the stated dtype on the host.

The five named configurations take the *shapes* of the paper's evaluation
(Tables 1-4: Llama2-7B/13B, Vicuna-33B, Llama3-70B; tree sizes 64, 128, 768)
and stand in for its models and datasets, which are not available here:
Q/K/V are i.i.d. N(0,1); target logits are N(0, 3^2); draft logits are the
target's plus Gaussian noise; every internal node's children carry tokens drawn
*without replacement* from softmax(draft_logits/T) in draw order (by the
Gumbel-top-k trick the paper cites for this step, Section 4.1), which is the
precondition Algorithm 2 places on its inputs.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

BASE_SEED = 20240212

# tensor ids for the per-tensor Philox streams
_T_TREE, _T_Q, _T_K, _T_V, _T_TGT, _T_NOISE, _T_GUMBEL, _T_UNIF = range(8)


@dataclass(frozen=True)
class TreeVerifyConfig:
    name: str
    config_id: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    prefix_len: int
    n_tree: int
    max_depth: int
    max_fanout: int | None
    dtype: str  # "fp16" | "bf16" | "fp32"
    vocab: int
    target_sigma: float
    draft_noise_sigma: float
    temperatures: tuple = field(default=(0.6,))


CONFIGS = {
    c.name: c
    for c in [
        TreeVerifyConfig("tiny", 1, 32, 32, 128, 128, 16, 6, None, "fp16", 32000, 3.0, 1.0, (0.6,)),
        TreeVerifyConfig("llama2-7b", 2, 32, 32, 128, 1024, 64, 10, 8, "bf16", 32000, 3.0, 1.0, (0.0, 0.6, 1.0)),
        TreeVerifyConfig("llama2-13b", 3, 40, 40, 128, 2048, 128, 12, None, "bf16", 32000, 3.0, 1.0, (1.0,)),
        TreeVerifyConfig("vicuna-33b", 4, 52, 52, 128, 2048, 256, 16, None, "bf16", 32000, 3.0, 1.0, (0.6,)),
        TreeVerifyConfig("llama3-70b", 5, 64, 8, 128, 4096, 768, 20, 16, "bf16", 128256, 3.0, 1.5, (0.6,)),
    ]
}

# decoder layers of the models the configs are named after (the whole-model key/value cache has layers x kv heads planes)
NUM_LAYERS = {"tiny": 2, "llama2-7b": 32, "llama2-13b": 40, "vicuna-33b": 60, "llama3-70b": 80}

# Acceptance-rate vector the paper prints (appendix "Examples of Sequoia trees": target Llama3-70B-Instruct, draft
# Llama3-8B-Instruct, CNN daily news): entry b-1 = probability that a node's b-th child is accepted.  Input data for
# the tree construction; nothing here computes with it.
PAPER_ACCEPTANCE_VECTOR = (
    0.7732, 0.1039, 0.0402, 0.0206, 0.0128, 0.0081, 0.0064, 0.0043, 0.0035, 0.0026, 0.0025, 0.0021, 0.0016, 0.0014,
    0.0010, 0.0010, 0.0010, 0.0007, 0.0007, 0.0006, 0.0007, 0.0006, 0.0004, 0.0004, 0.0005, 0.0006, 0.0004, 0.0003,
    0.0002, 0.0004, 0.0001,
)

TORCH_DTYPES = {"fp16": torch.float16, "bf16": torch.bfloat16, "fp32": torch.float32}


def _rng(config_id: int, seed: int, tensor_id: int) -> np.random.Generator:
    ss = np.random.SeedSequence([BASE_SEED, config_id, seed, tensor_id])
    return np.random.Generator(np.random.Philox(ss))


def random_tree(n: int, max_depth: int | None, max_fanout: int | None, rng: np.random.Generator) -> np.ndarray:
    """parent[0] = -1; parent[i] uniform over earlier nodes still below the depth and fan-out caps."""
    parent = np.full(n, -1, dtype=np.int32)
    depth = np.zeros(n, dtype=np.int64)
    fanout = np.zeros(n, dtype=np.int64)
    for i in range(1, n):
        ok = np.ones(i, dtype=bool)
        if max_depth is not None:
            ok &= depth[:i] < max_depth
        if max_fanout is not None:
            ok &= fanout[:i] < max_fanout
        cand = np.flatnonzero(ok)
        p = int(cand[rng.integers(0, len(cand))])
        parent[i] = p
        depth[i] = depth[p] + 1
        fanout[p] += 1
    return parent


def chain_tree(n: int) -> np.ndarray:
    return np.arange(-1, n - 1, dtype=np.int32)


def star_tree(n: int) -> np.ndarray:
    p = np.zeros(n, dtype=np.int32)
    p[0] = -1
    return p


def children_lists(parent: np.ndarray) -> list[list[int]]:
    kids: list[list[int]] = [[] for _ in range(len(parent))]
    for i in range(1, len(parent)):
        if parent[i] >= 0:
            kids[int(parent[i])].append(i)
    return kids


def draw_children_tokens(parent: np.ndarray, draft_logits: np.ndarray, T: float,
                         rng: np.random.Generator) -> np.ndarray:
    """tokens[c] for every non-root node: the k children of v get the first k entries of a
    without-replacement draw from softmax(draft_logits[v]/T), in draw order = ascending node
    index (keys logits/T + Gumbel noise, sorted descending).  T = 0: the draft's top-k."""
    n, V = draft_logits.shape
    tokens = np.zeros(n, dtype=np.int32)
    for v, kids in enumerate(children_lists(parent)):
        if not kids:
            continue
        k = len(kids)
        row = draft_logits[v].astype(np.float64)
        if T > 0:
            keys = row / T + rng.gumbel(size=V)
        else:
            keys = row
        finite = np.isfinite(keys)
        order = np.argsort(-np.where(finite, keys, -np.inf), kind="stable")
        n_ok = int(finite.sum())
        if k > n_ok:
            # more children than the draft's support: the remaining draws are uniform over
            # what is left (Algorithm 2's fallback distribution)
            rest = order[n_ok:].copy()
            rng.shuffle(rest)
            order = np.concatenate([order[:n_ok], rest])
        tokens[kids] = order[:k].astype(np.int32)
    return tokens


@dataclass
class AttentionInputs:
    q: torch.Tensor        # [n, Hq, d]
    k_cache: torch.Tensor  # [Hkv, capacity, d]; tree rows at [prefix_len, prefix_len + n)
    v_cache: torch.Tensor
    parent: torch.Tensor   # int32 [n]
    prefix_len: int


@dataclass
class VerifyInputs:
    parent: torch.Tensor         # int32 [n]
    tokens: torch.Tensor         # int32 [n]
    target_logits: torch.Tensor  # fp32 [n, V]
    draft_logits: torch.Tensor   # fp32 [n, V]
    uniforms: torch.Tensor       # fp32 [n+1]
    temperature: float


def make_tree(cfg: TreeVerifyConfig, seed: int = 0) -> np.ndarray:
    return random_tree(cfg.n_tree, cfg.max_depth, cfg.max_fanout, _rng(cfg.config_id, seed, _T_TREE))


def _normal(shape, rng, dtype: torch.dtype) -> torch.Tensor:
    a = rng.standard_normal(size=shape, dtype=np.float32)
    return torch.from_numpy(a).to(dtype)


def make_attention_inputs(cfg: TreeVerifyConfig, seed: int = 0, *, parent: np.ndarray | None = None,
                          dtype: str | None = None, extra_capacity: int = 0,
                          tail_fill: float = float("nan")) -> AttentionInputs:
    """Q/K/V ~ N(0,1).  ``extra_capacity`` appends rows past prefix_len+n filled with ``tail_fill``."""
    td = TORCH_DTYPES[dtype or cfg.dtype]
    if parent is None:
        parent = make_tree(cfg, seed)
    n = len(parent)
    rows = cfg.prefix_len + n
    q = _normal((n, cfg.num_q_heads, cfg.head_dim), _rng(cfg.config_id, seed, _T_Q), td)
    k = _normal((cfg.num_kv_heads, rows, cfg.head_dim), _rng(cfg.config_id, seed, _T_K), td)
    v = _normal((cfg.num_kv_heads, rows, cfg.head_dim), _rng(cfg.config_id, seed, _T_V), td)
    if extra_capacity:
        pad = torch.full((cfg.num_kv_heads, extra_capacity, cfg.head_dim), tail_fill, dtype=td)
        k = torch.cat([k, pad], dim=1).contiguous()
        v = torch.cat([v, pad], dim=1).contiguous()
    return AttentionInputs(q, k, v, torch.from_numpy(parent.copy()), cfg.prefix_len)


def make_verify_inputs(cfg: TreeVerifyConfig, T: float, seed: int = 0, *, parent: np.ndarray | None = None,
                       vocab: int | None = None) -> VerifyInputs:
    if parent is None:
        parent = make_tree(cfg, seed)
    n = len(parent)
    V = vocab or cfg.vocab
    tgt = _rng(cfg.config_id, seed, _T_TGT).standard_normal(size=(n, V), dtype=np.float32)
    tgt *= np.float32(cfg.target_sigma)
    noise = _rng(cfg.config_id, seed, _T_NOISE).standard_normal(size=(n, V), dtype=np.float32)
    noise *= np.float32(cfg.draft_noise_sigma)
    drf = tgt + noise
    del noise
    tokens = draw_children_tokens(parent, drf, T, _rng(cfg.config_id, seed, _T_GUMBEL))
    unif = _rng(cfg.config_id, seed, _T_UNIF).random(size=n + 1, dtype=np.float32)
    return VerifyInputs(torch.from_numpy(parent.copy()), torch.from_numpy(tokens), torch.from_numpy(tgt),
                        torch.from_numpy(drf), torch.from_numpy(unif), float(T))


def attention_algorithmic_bytes(cfg: TreeVerifyConfig, n: int | None = None) -> int:
    """K and V rows [0, L+n) once, Q and O once, at the config's element size."""
    e = {"fp16": 2, "bf16": 2, "fp32": 4}[cfg.dtype]
    n = n or cfg.n_tree
    return 2 * (cfg.prefix_len + n) * cfg.num_kv_heads * cfg.head_dim * e + 2 * n * cfg.num_q_heads * cfg.head_dim * e


def attention_algorithmic_flops(cfg: TreeVerifyConfig, parent: np.ndarray) -> int:
    """2 flops per MAC over unmasked (query, key) pairs only, for QK^T and PV."""
    n = len(parent)
    depth = np.zeros(n, dtype=np.int64)
    for i in range(1, n):
        depth[i] = depth[parent[i]] + 1 if parent[i] >= 0 else 0
    pairs = n * cfg.prefix_len + int((depth + 1).sum())
    return 4 * cfg.head_dim * cfg.num_q_heads * pairs
