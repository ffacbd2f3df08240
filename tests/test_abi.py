"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every function the
header declares, the ctypes structs match the C layout, and host-checkable errors are refused
before anything is launched."""
import ctypes as C
import os
import re
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "seq_tree.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2402_12374_b200 import build

    build.build()
    from paper_2402_12374_b200 import binding

    return binding.load()


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(seq_tree_\w+)\s*\(", text)))


def test_library_exports_every_declared_function(lib):
    from paper_2402_12374_b200 import binding

    names = _declared_functions()
    assert len(names) >= 6
    for name in names:
        assert hasattr(lib, name), name
    assert set(binding.EXPORTED_SYMBOLS) <= set(names)
    assert b"sm_100a" in lib.seq_tree_version()


def test_ctypes_structs_match_the_header(tmp_path):
    from paper_2402_12374_b200 import binding

    fields_a = [f[0] for f in binding.AttentionParams._fields_]
    fields_v = [f[0] for f in binding.VerifyParams._fields_]
    others = (("seq_tree_draft_sample_params", binding.DraftSampleParams), ("seq_tree_kv_commit_params", binding.KvCommitParams),
              ("seq_tree_top_p_params", binding.TopPParams), ("seq_tree_build_params", binding.TreeBuildParams),
              ("seq_tree_verify_batch_params", binding.VerifyBatchParams))
    src = tmp_path / "layout.c"
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "seq_tree.h"', "int main(void){",
             'printf("%zu\\n", sizeof(seq_tree_attention_params));']
    lines += [f'printf("%zu\\n", offsetof(seq_tree_attention_params, {f}));' for f in fields_a]
    lines += ['printf("%zu\\n", sizeof(seq_tree_verify_params));']
    lines += [f'printf("%zu\\n", offsetof(seq_tree_verify_params, {f}));' for f in fields_v]
    for cname, st in others:
        lines += [f'printf("%zu\\n", sizeof({cname}));']
        lines += [f'printf("%zu\\n", offsetof({cname}, {f[0]}));' for f in st._fields_]
    lines += ["return 0;}"]
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    nums = [int(x) for x in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()]
    assert nums[0] == C.sizeof(binding.AttentionParams)
    assert nums[1:1 + len(fields_a)] == [getattr(binding.AttentionParams, f).offset for f in fields_a]
    rest = nums[1 + len(fields_a):]
    assert rest[0] == C.sizeof(binding.VerifyParams)
    assert rest[1:1 + len(fields_v)] == [getattr(binding.VerifyParams, f).offset for f in fields_v]
    rest = rest[1 + len(fields_v):]
    for cname, st in others:
        names = [f[0] for f in st._fields_]
        assert rest[0] == C.sizeof(st), cname
        assert rest[1:1 + len(names)] == [getattr(st, f).offset for f in names], cname
        rest = rest[1 + len(names):]
    assert not rest


def test_host_checkable_errors_are_refused_before_launch(lib):
    from paper_2402_12374_b200 import binding as B

    fake = 0x1000  # never dereferenced: validation fails first
    assert lib.seq_tree_mask_from_parents(None, 4, fake, 1, None, None, None) == B.SEQ_ERR_INVALID_ARG
    assert lib.seq_tree_mask_from_parents(fake, 0, fake, 1, None, None, None) == B.SEQ_ERR_INVALID_ARG
    assert lib.seq_tree_mask_from_parents(fake, 2000, fake, 63, None, None, None) == B.SEQ_ERR_INVALID_ARG
    assert lib.seq_tree_mask_from_parents(fake, 64, fake, 1, None, None, None) == B.SEQ_ERR_INVALID_ARG

    def attn(**kw):
        p = B.AttentionParams()
        p.n_tree, p.prefix_len, p.num_q_heads, p.num_kv_heads, p.head_dim, p.dtype = 16, 128, 32, 32, 128, B.SEQ_BF16
        p.q = p.k_cache = p.v_cache = p.out = p.mask_bits = fake
        p.q_stride_tok, p.q_stride_head = 32 * 128, 128
        p.o_stride_tok, p.o_stride_head = 32 * 128, 128
        p.kv_stride_tok, p.kv_stride_head, p.kv_capacity = 128, 144 * 128, 144
        p.mask_words_per_row = 1
        for k, v in kw.items():
            setattr(p, k, v)
        return p

    bad = [dict(q=None), dict(n_tree=0), dict(n_tree=1025), dict(num_kv_heads=5), dict(kv_capacity=100),
           dict(dtype=7), dict(q_stride_head=100), dict(kv_stride_tok=129), dict(k_cache=fake + 2),
           dict(mask_words_per_row=0), dict(softmax_scale=float("nan")), dict(kernel=9), dict(prefix_len=-1),
           # one prefix length per request: a negative count, no lengths given, a count that does not divide the kv heads,
           # the stream schedule forced
           dict(prefix_len_dev_count=-1), dict(prefix_len_dev_count=4), dict(prefix_len_dev_count=5, prefix_len_dev=fake),
           dict(prefix_len_dev_count=4, prefix_len_dev=fake, kernel=3)]
    for kw in bad:
        assert lib.seq_tree_attention(C.byref(attn(**kw)), None) == B.SEQ_ERR_INVALID_ARG, kw
        assert lib.seq_tree_attention_workspace_bytes(C.byref(attn(**kw))) == 0
    assert lib.seq_tree_attention(C.byref(attn(head_dim=64)), None) == B.SEQ_ERR_UNSUPPORTED
    assert lib.seq_tree_attention(None, None) == B.SEQ_ERR_INVALID_ARG
    # a split-KV launch without workspace is refused
    big = attn(n_tree=16, prefix_len=4096, kv_capacity=4112, kv_stride_head=4112 * 128, num_q_heads=8, num_kv_heads=8,
               q_stride_tok=8 * 128, o_stride_tok=8 * 128, kernel=1)
    assert lib.seq_tree_attention_workspace_bytes(C.byref(big)) > 0
    assert lib.seq_tree_attention(C.byref(big), None) == B.SEQ_ERR_WORKSPACE

    def ver(**kw):
        p = B.VerifyParams()
        p.n_tree, p.vocab, p.temperature = 16, 32000, 0.6
        p.parent = p.tokens = p.target_logits = p.draft_logits = p.uniforms = fake
        p.path = p.path_len = p.bonus_token = fake
        p.target_row_stride = p.draft_row_stride = 32000
        for k, v in kw.items():
            setattr(p, k, v)
        return p

    bad = [dict(parent=None), dict(n_tree=0), dict(n_tree=5000), dict(vocab=0), dict(temperature=-1.0),
           dict(temperature=float("nan")), dict(temperature=float("inf")), dict(target_row_stride=31999),
           dict(target_row_stride=32001), dict(draft_logits=None), dict(uniforms=None), dict(path=None),
           dict(flags=64), dict(flags=6), dict(flags=1, next_child_out=None), dict(target_logits=fake + 4)]
    for kw in bad:
        assert lib.seq_tree_verify(C.byref(ver(**kw)), None) == B.SEQ_ERR_INVALID_ARG, kw
    assert lib.seq_tree_verify(C.byref(ver(vocab=400000, target_row_stride=400000, draft_row_stride=400000)), None) \
        == B.SEQ_ERR_UNSUPPORTED
    # the node-parallel schedule keeps a few words per node in a workspace; the walk (the default) none
    assert 0 < lib.seq_tree_verify_workspace_bytes(C.byref(ver(flags=B.SEQ_VERIFY_SCHED_NODES))) <= 16384
    assert lib.seq_tree_verify_workspace_bytes(C.byref(ver())) == 0
    assert lib.seq_tree_verify_workspace_bytes(C.byref(ver(flags=B.SEQ_VERIFY_SCHED_WALK))) == 0
    assert lib.seq_tree_verify_workspace_bytes(C.byref(ver(flags=B.SEQ_VERIFY_ALL_NODES, next_child_out=fake))) == 0
    assert lib.seq_tree_verify(C.byref(ver(flags=B.SEQ_VERIFY_SCHED_WALK | B.SEQ_VERIFY_SCHED_NODES)), None) == B.SEQ_ERR_INVALID_ARG
    assert lib.seq_tree_verify(C.byref(ver(flags=B.SEQ_VERIFY_SCHED_NODES)), None) == B.SEQ_ERR_WORKSPACE
    assert lib.seq_tree_verify(C.byref(ver(flags=B.SEQ_VERIFY_SCHED_NODES, vocab=400000, target_row_stride=400000,
                                           draft_row_stride=400000)), None) == B.SEQ_ERR_UNSUPPORTED

    def verb(**kw):
        p = B.VerifyBatchParams()
        p.request0 = ver()
        p.batch, p.tree_stride, p.logits_stride, p.uniforms_stride = 4, 16, 16 * 32000, 17
        for k, v in kw.items():
            setattr(p, k, v)
        return p

    for kw in (dict(batch=0), dict(tree_stride=15), dict(logits_stride=15 * 32000), dict(logits_stride=16 * 32000 + 2),
               dict(uniforms_stride=16), dict(request0=ver(flags=1, next_child_out=fake)), dict(request0=ver(vocab=0)),
               dict(request0=ver(residual_out=fake), residual_stride=31999)):
        assert lib.seq_tree_verify_batch(C.byref(verb(**kw)), None) == B.SEQ_ERR_INVALID_ARG, kw
    assert lib.seq_tree_verify_batch(None, None) == B.SEQ_ERR_INVALID_ARG

    def commit(**kw):
        p = B.KvCommitParams()
        p.num_planes, p.row_bytes, p.prefix_len, p.n_tree = 64, 256, 128, 16
        p.k_cache = p.v_cache = p.path = p.path_len = fake
        p.row_stride_bytes, p.plane_stride_bytes = 256, 144 * 256
        for k, v in kw.items():
            setattr(p, k, v)
        return p

    bad = [dict(k_cache=None), dict(path=None), dict(path_len=None), dict(num_planes=0), dict(n_tree=0), dict(n_tree=1025),
           dict(prefix_len=-1), dict(row_bytes=8), dict(row_bytes=250), dict(row_stride_bytes=128), dict(row_stride_bytes=264),
           dict(plane_stride_bytes=143 * 256), dict(plane_stride_bytes=144 * 256 + 8), dict(k_cache=fake + 4),
           dict(v_cache=fake + 8)]
    for kw in bad:
        assert lib.seq_tree_kv_commit(C.byref(commit(**kw)), None) == B.SEQ_ERR_INVALID_ARG, kw
    assert lib.seq_tree_kv_commit(None, None) == B.SEQ_ERR_INVALID_ARG

    def topp(**kw):
        p = B.TopPParams()
        p.n_rows, p.vocab, p.temperature, p.top_p = 4, 32000, 0.6, 0.9
        p.logits = p.out = fake
        p.logits_row_stride = p.out_row_stride = 32000
        for k, v in kw.items():
            setattr(p, k, v)
        return p

    bad = [dict(logits=None), dict(out=None), dict(n_rows=0), dict(vocab=0), dict(temperature=0.0), dict(temperature=float("nan")),
           dict(temperature=float("inf")), dict(top_p=0.0), dict(top_p=-0.5), dict(top_p=float("nan")),
           dict(logits_row_stride=31996), dict(out_row_stride=32002), dict(logits=fake + 4), dict(out=fake + 8)]
    for kw in bad:
        assert lib.seq_tree_top_p_filter(C.byref(topp(**kw)), None) == B.SEQ_ERR_INVALID_ARG, kw


def test_binding_refuses_cpu_tensors():
    import torch

    from paper_2402_12374_b200 import binding as B

    with pytest.raises(ValueError, match="no CPU path"):
        B.seq_tree_mask_from_parents(torch.tensor([-1, 0], dtype=torch.int32))


def test_attention_schedule_choice_is_visible_through_the_workspace_size(lib):
    """Host logic of the tensor-core kernel's plan, observable without a GPU: only its stream schedule needs a
    workspace.  Taken for long tiles on many (tile, kv head) units (the llama3-70b shape) or when the last wave of
    plain waves would be thin; never for short tiles; forced either way by kernel = 3 / 4."""
    from paper_2402_12374_b200 import binding as B

    fake = 0x1000

    def shape(n, L, Hq, Hkv, kernel=0):
        p = B.AttentionParams()
        p.n_tree, p.prefix_len, p.num_q_heads, p.num_kv_heads, p.head_dim, p.dtype = n, L, Hq, Hkv, 128, B.SEQ_BF16
        p.q = p.k_cache = p.v_cache = p.out = fake
        p.parent = fake
        p.q_stride_tok, p.q_stride_head = Hq * 128, 128
        p.o_stride_tok, p.o_stride_head = Hq * 128, 128
        p.kv_stride_tok, p.kv_stride_head, p.kv_capacity = 128, (L + n) * 128, L + n
        p.mask_words_per_row = (n + 31) // 32
        p.kernel = kernel
        return lib.seq_tree_attention_workspace_bytes(C.byref(p))

    assert shape(768, 4096, 64, 8) > 0             # 384 units of 76 blocks: stream schedule
    assert shape(64, 1024, 32, 32) == 0            # 32 units: a cluster per unit
    assert shape(64, 1024, 8 * 32, 8 * 32) == 0    # 256 units of 17 blocks (8 requests as heads): plain waves
    assert shape(128, 2048, 4 * 40, 4 * 40) > 0    # 160 units of 34 blocks: the second wave would hold 12 CTAs
    assert shape(128, 2048, 6 * 40, 6 * 40) == 0   # 240 units: waves
    assert shape(64, 1024, 8 * 32, 8 * 32, kernel=3) > 0 and shape(768, 4096, 64, 8, kernel=4) == 0
    assert shape(64, 1024, 32, 32, kernel=3) > 0   # forced even where one wave would do
