"""seq_tree_attention_noalloc, the entry point for callers that cannot hand the library any scratch
memory (a server whose device memory is fixed at start-up, an embedder without a tensor framework):
it must give what seq_tree_attention gives with the CUDA-core kernel, call after call, although every
call reuses the same built-in scratch array.  Collected last on purpose (file name), so a run that
stops at the first failure has already run everything else."""
import ctypes as C
import dataclasses

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2402_12374_b200 import binding as B
from paper_2402_12374_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _inputs(seed, dtype):
    # few rows and a long prefix: the CUDA-core kernel splits the key range, so scratch is really used
    cfg = dataclasses.replace(W.CONFIGS["tiny"], num_q_heads=4, num_kv_heads=2, prefix_len=4096, n_tree=16)
    return W.make_attention_inputs(cfg, seed, dtype=dtype)


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_noalloc_matches_the_workspace_entry_point_on_two_calls_in_a_row(dtype):
    d = torch.device("cuda:0")
    tol = 2e-2 if dtype == "bf16" else 1e-5
    for seed in (11, 12):  # two calls in a row; the second finds the first one's partials in the scratch array
        ai = _inputs(seed, dtype)
        q, k, v = ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d)
        mask, _ = B.seq_tree_mask_from_parents(ai.parent.to(d))
        ref_call = B.AttentionCall(q, k, v, mask, ai.prefix_len, kernel=B.KERNEL_CUDA_CORE,
                                   lse=torch.empty((4, 16), dtype=torch.float32, device=d))
        assert ref_call.workspace_bytes_needed > 0, "the case must exercise scratch memory"
        ref = ref_call.run().clone()
        lse = torch.empty((4, 16), dtype=torch.float32, device=d)
        got = B.seq_tree_attention_noalloc(q, k, v, mask, ai.prefix_len, lse=lse)
        torch.cuda.synchronize()
        assert (got.double() - ref.double()).abs().max().item() <= tol
        assert (lse - ref_call.lse).abs().max().item() <= 1e-5
        oracle_out, _, _ = O.tree_attention(ai.q, ai.k_cache, ai.v_cache, ai.parent, ai.prefix_len)
        assert np.abs(got.double().cpu().numpy() - oracle_out).max() < tol


def test_noalloc_rejects_what_does_not_fit_and_bad_arguments():
    lib = B.load()
    fake = 0x1000  # never dereferenced: the size check comes first
    p = B.AttentionParams()
    p.n_tree, p.prefix_len, p.num_q_heads, p.num_kv_heads, p.head_dim, p.dtype = 8, 1 << 20, 64, 64, 128, B.SEQ_BF16
    p.q = p.k_cache = p.v_cache = p.out = p.mask_bits = fake
    p.q_stride_tok = p.o_stride_tok = 64 * 128
    p.q_stride_head = p.o_stride_head = 128
    p.kv_stride_tok, p.kv_capacity = 128, (1 << 20) + 8
    p.kv_stride_head = p.kv_capacity * 128
    p.mask_words_per_row = 1
    assert lib.seq_tree_attention_noalloc(C.byref(p), None) == B.SEQ_ERR_WORKSPACE
    p.q = None
    assert lib.seq_tree_attention_noalloc(C.byref(p), None) == B.SEQ_ERR_INVALID_ARG
    assert lib.seq_tree_attention_noalloc(None, None) == B.SEQ_ERR_INVALID_ARG
