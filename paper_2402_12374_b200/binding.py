"""Thin ctypes binding of ``libseqtree.so`` (see ``include/seq_tree.h``).

Argument marshalling only: every step of the token-tree verification path runs in the
library's CUDA kernels.  torch supplies device memory and streams.  There is no CPU fallback:
if the library is missing or a tensor is not on a CUDA device the call raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libseqtree.so")

SEQ_OK, SEQ_ERR_INVALID_ARG, SEQ_ERR_UNSUPPORTED, SEQ_ERR_WORKSPACE, SEQ_ERR_CUDA = 0, -1, -2, -3, -4
SEQ_F16, SEQ_BF16, SEQ_F32 = 0, 1, 2
SEQ_DEV_BAD_PARENT, SEQ_DEV_BAD_TOKEN, SEQ_DEV_NONFINITE, SEQ_DEV_DEGENERATE, SEQ_DEV_TIMEOUT = 1, 2, 4, 8, 16
SEQ_VERIFY_ALL_NODES = 1
SEQ_VERIFY_SPECINFER = 2
SEQ_VERIFY_TARGET_SAMPLE = 4
SEQ_VERIFY_SCHED_WALK, SEQ_VERIFY_SCHED_NODES = 16, 32
SEQ_VERIFY_LOGITS_BF16 = 8
SEQ_DEV_BAD_PATH = 32
SEQ_DEV_BAD_LENGTH = 64
SEQ_MAX_TREE = 1024
SEQ_NOALLOC_SCRATCH_BYTES = 384 << 10
KERNEL_AUTO, KERNEL_CUDA_CORE, KERNEL_TENSOR_CORE = 0, 1, 2
KERNEL_TENSOR_CORE_STREAM, KERNEL_TENSOR_CORE_GRID = 3, 4  # the tensor-core kernel with one of its two schedules forced

_STATUS_NAMES = {0: "SEQ_OK", -1: "SEQ_ERR_INVALID_ARG", -2: "SEQ_ERR_UNSUPPORTED", -3: "SEQ_ERR_WORKSPACE",
                 -4: "SEQ_ERR_CUDA"}
_DTYPES = {torch.float16: SEQ_F16, torch.bfloat16: SEQ_BF16, torch.float32: SEQ_F32}

EXPORTED_SYMBOLS = (
    "seq_tree_mask_from_parents",
    "seq_tree_attention_workspace_bytes",
    "seq_tree_attention",
    "seq_tree_attention_noalloc",
    "seq_tree_verify_workspace_bytes",
    "seq_tree_verify",
    "seq_tree_verify_batch",
    "seq_tree_draft_sample_workspace_bytes",
    "seq_tree_draft_sample",
    "seq_tree_kv_commit",
    "seq_tree_top_p_filter",
    "seq_tree_build",
    "seq_tree_speedup_search",
    "seq_tree_probe_stream_read",
    "seq_tree_probe_dependent_load",
    "seq_tree_version",
)


class SeqTreeError(RuntimeError):
    def __init__(self, fn: str, code: int):
        super().__init__(f"{fn} returned {_STATUS_NAMES.get(code, code)}")
        self.code = code


class AttentionParams(C.Structure):
    _fields_ = [
        ("n_tree", C.c_int32), ("prefix_len", C.c_int32), ("num_q_heads", C.c_int32),
        ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("dtype", C.c_int32),
        ("softmax_scale", C.c_float),
        ("q", C.c_void_p), ("q_stride_tok", C.c_int64), ("q_stride_head", C.c_int64),
        ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
        ("kv_stride_tok", C.c_int64), ("kv_stride_head", C.c_int64), ("kv_capacity", C.c_int32),
        ("mask_bits", C.c_void_p), ("mask_words_per_row", C.c_int32),
        ("out", C.c_void_p), ("o_stride_tok", C.c_int64), ("o_stride_head", C.c_int64),
        ("lse", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("dev_status", C.c_void_p), ("kernel", C.c_int32),
        ("parent", C.c_void_p), ("prefix_len_dev", C.c_void_p), ("prefix_len_dev_count", C.c_int32),
    ]


class VerifyParams(C.Structure):
    _fields_ = [
        ("n_tree", C.c_int32), ("vocab", C.c_int32),
        ("parent", C.c_void_p), ("tokens", C.c_void_p),
        ("target_logits", C.c_void_p), ("target_row_stride", C.c_int64),
        ("draft_logits", C.c_void_p), ("draft_row_stride", C.c_int64),
        ("temperature", C.c_float), ("uniforms", C.c_void_p),
        ("path", C.c_void_p), ("path_len", C.c_void_p), ("bonus_token", C.c_void_p),
        ("residual_out", C.c_void_p), ("next_child_out", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("dev_status", C.c_void_p), ("flags", C.c_int32),
    ]


_lib = None


def load() -> C.CDLL:
    """Load the CUDA library; raises if it has not been built (``python -m paper_2402_12374_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2402_12374_b200.build`; "
                               "there is no fallback path")
        lib = C.CDLL(LIB_PATH)
        lib.seq_tree_mask_from_parents.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                                   C.c_void_p, C.c_void_p]
        lib.seq_tree_mask_from_parents.restype = C.c_int
        lib.seq_tree_attention_workspace_bytes.argtypes = [C.POINTER(AttentionParams)]
        lib.seq_tree_attention_workspace_bytes.restype = C.c_size_t
        lib.seq_tree_attention.argtypes = [C.POINTER(AttentionParams), C.c_void_p]
        lib.seq_tree_attention.restype = C.c_int
        lib.seq_tree_attention_noalloc.argtypes = [C.POINTER(AttentionParams), C.c_void_p]
        lib.seq_tree_attention_noalloc.restype = C.c_int
        lib.seq_tree_draft_sample_workspace_bytes.argtypes = [C.POINTER(DraftSampleParams)]
        lib.seq_tree_draft_sample_workspace_bytes.restype = C.c_size_t
        lib.seq_tree_draft_sample.argtypes = [C.POINTER(DraftSampleParams), C.c_void_p]
        lib.seq_tree_draft_sample.restype = C.c_int
        lib.seq_tree_verify_workspace_bytes.argtypes = [C.POINTER(VerifyParams)]
        lib.seq_tree_verify_workspace_bytes.restype = C.c_size_t
        lib.seq_tree_verify.argtypes = [C.POINTER(VerifyParams), C.c_void_p]
        lib.seq_tree_verify.restype = C.c_int
        lib.seq_tree_verify_batch.argtypes = [C.POINTER(VerifyBatchParams), C.c_void_p]
        lib.seq_tree_verify_batch.restype = C.c_int
        lib.seq_tree_kv_commit.argtypes = [C.POINTER(KvCommitParams), C.c_void_p]
        lib.seq_tree_kv_commit.restype = C.c_int
        lib.seq_tree_top_p_filter.argtypes = [C.POINTER(TopPParams), C.c_void_p]
        lib.seq_tree_top_p_filter.restype = C.c_int
        lib.seq_tree_build.argtypes = [C.POINTER(TreeBuildParams)]
        lib.seq_tree_build.restype = C.c_int
        lib.seq_tree_speedup_search.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_double, C.POINTER(C.c_int32),
                                                C.POINTER(C.c_int32), C.POINTER(C.c_double)]
        lib.seq_tree_speedup_search.restype = C.c_int
        lib.seq_tree_version.restype = C.c_char_p
        lib.seq_tree_probe_stream_read.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p]
        lib.seq_tree_probe_stream_read.restype = C.c_int
        lib.seq_tree_probe_dependent_load.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        lib.seq_tree_probe_dependent_load.restype = C.c_int
        _lib = lib
    return _lib


def _dev(t: torch.Tensor | None, name: str, dtype=None) -> int | None:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must live on a CUDA device (there is no CPU path)")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream if hasattr(s, "cuda_stream") else int(s)


def _check(fn: str, code: int) -> None:
    if code != SEQ_OK:
        raise SeqTreeError(fn, code)


def seq_tree_version() -> str:
    return load().seq_tree_version().decode()


def seq_tree_mask_from_parents(parent: torch.Tensor, *, words_per_row: int | None = None,
                               mask_bits: torch.Tensor | None = None, depth: torch.Tensor | None = None,
                               dev_status: torch.Tensor | None = None, stream=None):
    """parent int32 [n] (device) -> (mask_bits int32-typed uint32 words [n, words_per_row], depth int32 [n])."""
    n = parent.shape[0]
    wpr = words_per_row or (n + 31) // 32
    if mask_bits is None:
        mask_bits = torch.empty((n, wpr), dtype=torch.int32, device=parent.device)
    if depth is None:
        depth = torch.empty(n, dtype=torch.int32, device=parent.device)
    rc = load().seq_tree_mask_from_parents(_dev(parent, "parent", torch.int32), n, _dev(mask_bits, "mask_bits", torch.int32),
                                           wpr, _dev(depth, "depth", torch.int32), _dev(dev_status, "dev_status", torch.int32),
                                           _stream(stream))
    _check("seq_tree_mask_from_parents", rc)
    return mask_bits, depth


class DraftSampleParams(C.Structure):
    _fields_ = [
        ("n_rows", C.c_int32), ("vocab", C.c_int32), ("k", C.c_int32),
        ("draft_logits", C.c_void_p), ("logits_row_stride", C.c_int64),
        ("uniforms", C.c_void_p), ("uniforms_row_stride", C.c_int64),
        ("temperature", C.c_float), ("tokens_out", C.c_void_p), ("dev_status", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
    ]


class KvCommitParams(C.Structure):
    _fields_ = [
        ("num_planes", C.c_int32), ("row_bytes", C.c_int32), ("prefix_len", C.c_int32), ("n_tree", C.c_int32),
        ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
        ("plane_stride_bytes", C.c_int64), ("row_stride_bytes", C.c_int64),
        ("path", C.c_void_p), ("path_len", C.c_void_p), ("new_prefix_len", C.c_void_p), ("dev_status", C.c_void_p),
        ("prefix_len_dev", C.c_void_p),
    ]


def seq_tree_draft_sample(draft_logits, temperature: float, uniforms, k: int, *, tokens_out=None, dev_status=None,
                          workspace=None, stream=None):
    """k tokens per row drawn without replacement from softmax(draft_logits / temperature) by exponential
    sort with the supplied uniforms; returns int32 [rows, k] (device), -1 where nothing was left to draw."""
    rows, V = draft_logits.shape
    if uniforms.shape != draft_logits.shape or draft_logits.stride(1) != 1 or uniforms.stride(1) != 1:
        raise ValueError("draft_logits and uniforms must be [rows, vocab] with contiguous rows")
    if tokens_out is None:
        tokens_out = torch.empty((rows, k), dtype=torch.int32, device=draft_logits.device)
    p = DraftSampleParams()
    p.n_rows, p.vocab, p.k = rows, V, k
    p.draft_logits, p.logits_row_stride = _dev(draft_logits, "draft_logits", torch.float32), (draft_logits.stride(0) if rows > 1 else V)
    p.uniforms, p.uniforms_row_stride = _dev(uniforms, "uniforms", torch.float32), (uniforms.stride(0) if rows > 1 else V)
    p.temperature = temperature
    p.tokens_out = _dev(tokens_out, "tokens_out", torch.int32)
    p.dev_status = _dev(dev_status, "dev_status", torch.int32)
    need = load().seq_tree_draft_sample_workspace_bytes(C.byref(p))
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=draft_logits.device)
    p.workspace = _dev(workspace, "workspace") if workspace is not None else None
    p.workspace_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check("seq_tree_draft_sample", load().seq_tree_draft_sample(C.byref(p), _stream(stream)))
    return tokens_out


class AttentionCall:
    """A prepared seq_tree_attention call: the parameter struct is filled once and can be launched many times."""

    def __init__(self, q, k_cache, v_cache, mask_bits, prefix_len: int, *, out=None, lse=None,
                 softmax_scale: float = 0.0, workspace=None, dev_status=None, kernel: int = KERNEL_AUTO,
                 noalloc: bool = False, parent=None, prefix_len_dev=None):
        """``noalloc=True`` prepares a call of ``seq_tree_attention_noalloc``: no workspace tensor is
        created or passed; the library's built-in scratch array is used (CUDA-core kernel).
        ``mask_bits=None`` with ``parent`` (int32 [n], device) lets the tensor-core kernel derive the
        ancestor mask from the parent array itself."""
        if q.dtype not in _DTYPES or k_cache.dtype != q.dtype or v_cache.dtype != q.dtype:
            raise ValueError("q, k_cache, v_cache must share one of float16/bfloat16/float32")
        n, Hq, d = q.shape
        Hkv, cap, dk = k_cache.shape
        if v_cache.shape != k_cache.shape or dk != d:
            raise ValueError("k_cache and v_cache must be [Hkv, capacity, head_dim]")
        for t, nm in ((q, "q"), (k_cache, "k_cache"), (v_cache, "v_cache")):
            if t.stride(-1) != 1:
                raise ValueError(f"{nm}: head_dim must be contiguous")
        if k_cache.stride() != v_cache.stride():
            raise ValueError("k_cache and v_cache must share strides")
        if out is None:
            out = torch.empty_like(q)
        p = AttentionParams()
        p.n_tree, p.prefix_len, p.num_q_heads, p.num_kv_heads, p.head_dim = n, prefix_len, Hq, Hkv, d
        p.dtype, p.softmax_scale = _DTYPES[q.dtype], softmax_scale
        p.q, p.q_stride_tok, p.q_stride_head = _dev(q, "q"), q.stride(0), q.stride(1)
        p.k_cache, p.v_cache = _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache")
        p.kv_stride_tok, p.kv_stride_head, p.kv_capacity = k_cache.stride(1), k_cache.stride(0), cap
        if mask_bits is not None:
            p.mask_bits, p.mask_words_per_row = _dev(mask_bits, "mask_bits", torch.int32), mask_bits.shape[1]
        else:
            if parent is None:
                raise ValueError("mask_bits or parent is required")
            p.mask_bits, p.mask_words_per_row = None, 0
        p.parent = _dev(parent, "parent", torch.int32)
        p.prefix_len_dev = _dev(prefix_len_dev, "prefix_len_dev", torch.int32)  # prefix_len is then its upper bound
        # more than one element: one length per request of a batch stacked as heads
        p.prefix_len_dev_count = 0 if prefix_len_dev is None else prefix_len_dev.numel()
        p.out, p.o_stride_tok, p.o_stride_head = _dev(out, "out", q.dtype), out.stride(0), out.stride(1)
        p.lse = _dev(lse, "lse", torch.float32)
        p.dev_status = _dev(dev_status, "dev_status", torch.int32)
        p.kernel = kernel
        self.noalloc = noalloc
        need = 0 if noalloc else load().seq_tree_attention_workspace_bytes(C.byref(p))
        if workspace is None and need:
            workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
        p.workspace = _dev(workspace, "workspace") if workspace is not None else None
        p.workspace_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
        self.params, self.out, self.lse, self.workspace_bytes_needed = p, out, lse, need
        self.workspace = workspace
        self._keep = (q, k_cache, v_cache, mask_bits, parent, out, lse, workspace, dev_status, prefix_len_dev)

    def run(self, stream=None):
        if self.noalloc:
            _check("seq_tree_attention_noalloc", load().seq_tree_attention_noalloc(C.byref(self.params), _stream(stream)))
        else:
            _check("seq_tree_attention", load().seq_tree_attention(C.byref(self.params), _stream(stream)))
        return self.out


def seq_tree_attention(q, k_cache, v_cache, mask_bits, prefix_len: int, **kw):
    """Tree-masked attention of the n tree tokens; returns out [n, Hq, d] (same dtype as q)."""
    stream = kw.pop("stream", None)
    return AttentionCall(q, k_cache, v_cache, mask_bits, prefix_len, **kw).run(stream)


def seq_tree_attention_noalloc(q, k_cache, v_cache, mask_bits, prefix_len: int, **kw):
    """seq_tree_attention for callers that cannot provide scratch memory: same result as the CUDA-core
    kernel, split-KV partials in the library's built-in array (see ``include/seq_tree.h``)."""
    stream = kw.pop("stream", None)
    return AttentionCall(q, k_cache, v_cache, mask_bits, prefix_len, noalloc=True, **kw).run(stream)


class VerifyCall:
    """A prepared seq_tree_verify call."""

    def __init__(self, parent, tokens, target_logits, draft_logits, temperature: float, uniforms, *,
                 path=None, path_len=None, bonus_token=None, residual_out=None, next_child_out=None,
                 all_nodes: bool = False, dev_status=None, specinfer: bool = False, target_sample: bool = False,
                 schedule: str = "auto", workspace=None):
        """schedule: "auto" (node-parallel where it applies), "walk" or "nodes" (forced)."""
        n, V = target_logits.shape
        dev = target_logits.device
        if path is None:
            path = torch.empty(n, dtype=torch.int32, device=dev)
        if path_len is None:
            path_len = torch.zeros(1, dtype=torch.int32, device=dev)
        if bonus_token is None:
            bonus_token = torch.full((1,), -1, dtype=torch.int32, device=dev)
        if all_nodes and next_child_out is None:
            next_child_out = torch.empty(n, dtype=torch.int32, device=dev)
        for t, nm in ((target_logits, "target_logits"), (draft_logits, "draft_logits")):
            if t is not None and t.stride(-1) != 1:
                raise ValueError(f"{nm}: vocabulary dimension must be contiguous")
        p = VerifyParams()
        p.n_tree, p.vocab = n, V
        p.parent, p.tokens = _dev(parent, "parent", torch.int32), _dev(tokens, "tokens", torch.int32)
        ldt = target_logits.dtype  # fp32, or bfloat16 (then the draft's too)
        if ldt not in (torch.float32, torch.bfloat16):
            raise ValueError("target_logits must be float32 or bfloat16")
        p.target_logits, p.target_row_stride = _dev(target_logits, "target_logits", ldt), target_logits.stride(0)
        p.draft_logits = _dev(draft_logits, "draft_logits", ldt)
        p.draft_row_stride = draft_logits.stride(0) if draft_logits is not None else 0
        p.temperature = temperature
        p.uniforms = _dev(uniforms, "uniforms", torch.float32)
        p.path, p.path_len = _dev(path, "path", torch.int32), _dev(path_len, "path_len", torch.int32)
        p.bonus_token = _dev(bonus_token, "bonus_token", torch.int32)
        p.residual_out = _dev(residual_out, "residual_out", torch.float32)
        p.next_child_out = _dev(next_child_out, "next_child_out", torch.int32)
        p.workspace, p.workspace_bytes = None, 0
        p.dev_status = _dev(dev_status, "dev_status", torch.int32)
        p.flags = ((SEQ_VERIFY_ALL_NODES if all_nodes else 0) | (SEQ_VERIFY_SPECINFER if specinfer else 0) |
                   (SEQ_VERIFY_TARGET_SAMPLE if target_sample else 0) | (SEQ_VERIFY_LOGITS_BF16 if ldt == torch.bfloat16 else 0) |
                   {"auto": 0, "walk": SEQ_VERIFY_SCHED_WALK, "nodes": SEQ_VERIFY_SCHED_NODES}[schedule])
        need = load().seq_tree_verify_workspace_bytes(C.byref(p))
        if workspace is None and need:
            workspace = torch.empty(need, dtype=torch.uint8, device=dev)
        if workspace is not None:
            p.workspace, p.workspace_bytes = _dev(workspace, "workspace"), workspace.numel() * workspace.element_size()
        self.workspace, self.workspace_bytes_needed = workspace, need
        self.params = p
        self.path, self.path_len, self.bonus_token = path, path_len, bonus_token
        self.residual_out, self.next_child_out = residual_out, next_child_out
        self._keep = (parent, tokens, target_logits, draft_logits, uniforms, dev_status)

    def run(self, stream=None):
        _check("seq_tree_verify", load().seq_tree_verify(C.byref(self.params), _stream(stream)))
        return self.path, self.path_len, self.bonus_token

    def rows_read(self):
        """Logit rows the last call read (synchronises); None for the walk, which reads the visited nodes' rows only."""
        if self.workspace is None or not self.workspace_bytes_needed:
            return None
        return int(self.workspace[:4].view(torch.int32).item())


class VerifyBatchParams(C.Structure):
    _fields_ = [
        ("request0", VerifyParams), ("batch", C.c_int32),
        ("tree_stride", C.c_int64), ("logits_stride", C.c_int64), ("uniforms_stride", C.c_int64),
        ("residual_stride", C.c_int64),
    ]


def seq_tree_verify_batch(parent, tokens, target_logits, draft_logits, temperature: float, uniforms, *, residual_out=None,
                          next_child_out=None, dev_status=None, specinfer: bool = False, target_sample: bool = False,
                          stream=None):
    """R requests in one launch.  parent, tokens [R, n]; target_logits, draft_logits [R, n, V]; uniforms [R, n+1];
    residual_out [R, V] and next_child_out [R, n] optional.  Returns path [R, n], path_len [R], bonus_token [R]."""
    R, n, V = target_logits.shape
    dev = target_logits.device
    path = torch.empty((R, n), dtype=torch.int32, device=dev)
    path_len = torch.zeros(R, dtype=torch.int32, device=dev)
    bonus = torch.full((R,), -1, dtype=torch.int32, device=dev)
    for t, nm in ((parent, "parent"), (tokens, "tokens"), (uniforms, "uniforms"), (target_logits, "target_logits"),
                  (draft_logits, "draft_logits"), (residual_out, "residual_out"), (next_child_out, "next_child_out")):
        if t is not None and (t.shape[0] != R or t.stride(-1) != 1):
            raise ValueError(f"{nm}: one entry per request, innermost dimension contiguous")
    if draft_logits is not None and draft_logits.stride(0) != target_logits.stride(0):
        raise ValueError("target_logits and draft_logits must have the same stride between requests")
    if parent.stride(0) != tokens.stride(0) or parent.stride(0) != n or (next_child_out is not None and next_child_out.stride(0) != n):
        raise ValueError("parent, tokens and next_child_out must be [R, n] contiguous")
    one = VerifyCall(parent[0], tokens[0], target_logits[0], None if draft_logits is None else draft_logits[0], temperature,
                     uniforms[0], path=path[0], path_len=path_len, bonus_token=bonus,
                     residual_out=None if residual_out is None else residual_out[0],
                     next_child_out=None if next_child_out is None else next_child_out[0], dev_status=dev_status,
                     specinfer=specinfer, target_sample=target_sample)
    p = VerifyBatchParams()
    p.request0 = one.params
    p.batch = R
    p.tree_stride, p.logits_stride = n, target_logits.stride(0)
    p.uniforms_stride = uniforms.stride(0)
    p.residual_stride = residual_out.stride(0) if residual_out is not None else 0
    _check("seq_tree_verify_batch", load().seq_tree_verify_batch(C.byref(p), _stream(stream)))
    return path, path_len, bonus


def seq_tree_verify(parent, tokens, target_logits, draft_logits, temperature: float, uniforms, **kw):
    """Algorithm 2 walked from the root; returns device tensors (path [n], path_len [1], bonus_token [1])."""
    stream = kw.pop("stream", None)
    return VerifyCall(parent, tokens, target_logits, draft_logits, temperature, uniforms, **kw).run(stream)


class TopPParams(C.Structure):
    _fields_ = [
        ("n_rows", C.c_int32), ("vocab", C.c_int32),
        ("logits", C.c_void_p), ("logits_row_stride", C.c_int64),
        ("out", C.c_void_p), ("out_row_stride", C.c_int64),
        ("temperature", C.c_float), ("top_p", C.c_float),
        ("kept_out", C.c_void_p), ("dev_status", C.c_void_p),
    ]


def seq_tree_top_p_filter(logits, temperature: float, top_p: float, *, out=None, kept_out=None, dev_status=None,
                          stream=None):
    """Nucleus truncation of softmax(logits / temperature) per row: returns logits with -inf outside the nucleus
    (``out=logits`` works in place)."""
    rows, V = logits.shape
    if out is None:
        out = torch.empty_like(logits)
    for t, nm in ((logits, "logits"), (out, "out")):
        if t.shape != logits.shape or t.stride(1) != 1:
            raise ValueError(f"{nm} must be [rows, vocab] with contiguous rows")
    p = TopPParams()
    p.n_rows, p.vocab = rows, V
    p.logits, p.logits_row_stride = _dev(logits, "logits", torch.float32), (logits.stride(0) if rows > 1 else (V + 3) // 4 * 4)
    p.out, p.out_row_stride = _dev(out, "out", torch.float32), (out.stride(0) if rows > 1 else (V + 3) // 4 * 4)
    p.temperature, p.top_p = temperature, top_p
    p.kept_out = _dev(kept_out, "kept_out", torch.int32)
    p.dev_status = _dev(dev_status, "dev_status", torch.int32)
    _check("seq_tree_top_p_filter", load().seq_tree_top_p_filter(C.byref(p), _stream(stream)))
    return out


class TreeBuildParams(C.Structure):
    _fields_ = [
        ("max_size", C.c_int32), ("max_depth", C.c_int32), ("max_branch", C.c_int32), ("acc_rows", C.c_int32),
        ("acc_rates", C.c_void_p), ("parent_out", C.c_void_p), ("size_out", C.c_void_p), ("expected_out", C.c_void_p),
        ("table_out", C.c_void_p),
    ]


def seq_tree_build(acc_rates, max_size: int, max_depth: int, max_branch: int | None = None, *, want_table: bool = False):
    """Host call: Sequoia's dynamic program.  acc_rates: [B] or [rows][B] array-like of acceptance probabilities.
    Returns (parent int32 numpy array in level order, F) or (parent, F, table [max_size+1][max_depth+1])."""
    import numpy as np

    rates = np.ascontiguousarray(np.atleast_2d(np.asarray(acc_rates, dtype=np.float64)))
    B = max_branch if max_branch is not None else rates.shape[1]
    if B > rates.shape[1]:
        raise ValueError("max_branch exceeds the number of acceptance rates per row")
    rates = np.ascontiguousarray(rates[:, :B])
    parent = np.empty(max(max_size, 1), dtype=np.int32)
    size, F = C.c_int32(0), C.c_double(0.0)
    table = np.empty((max_size + 1, max_depth + 1), dtype=np.float64) if want_table else None
    p = TreeBuildParams()
    p.max_size, p.max_depth, p.max_branch, p.acc_rows = max_size, max_depth, B, rates.shape[0]
    p.acc_rates, p.parent_out = rates.ctypes.data, parent.ctypes.data
    p.size_out, p.expected_out = C.addressof(size), C.addressof(F)
    p.table_out = table.ctypes.data if want_table else None
    _check("seq_tree_build", load().seq_tree_build(C.byref(p)))
    out = (parent[: size.value].copy(), float(F.value))
    return out + (table,) if want_table else out


def seq_tree_speedup_search(table, t_of_n, c: float):
    """Host call: (n, d, speedup) maximising G(n, d) / (t(n) + d c)."""
    import numpy as np

    table = np.ascontiguousarray(table, dtype=np.float64)
    t = np.ascontiguousarray(t_of_n, dtype=np.float64)
    if t.shape[0] != table.shape[0]:
        raise ValueError("t_of_n needs one entry per row of the table (entry 0 unused)")
    n, d, s = C.c_int32(0), C.c_int32(0), C.c_double(0.0)
    _check("seq_tree_speedup_search",
           load().seq_tree_speedup_search(table.ctypes.data, table.shape[0] - 1, table.shape[1] - 1, t.ctypes.data, float(c),
                                          C.byref(n), C.byref(d), C.byref(s)))
    return int(n.value), int(d.value), float(s.value)


def seq_tree_kv_commit(k_cache, v_cache, prefix_len: int, n_tree: int, path, path_len, *, new_prefix_len=None,
                       dev_status=None, stream=None, prefix_len_dev=None):
    """In place: row prefix_len+i of every plane <- row prefix_len+path[i], i < path_len (device tensors as
    seq_tree_verify wrote them).  k_cache / v_cache: [planes, rows, head_dim] (v_cache may be None), rows
    contiguous."""
    planes, rows, d = k_cache.shape
    for t in (k_cache, v_cache):
        if t is not None and (t.shape != k_cache.shape or t.stride() != k_cache.stride() or t.stride(2) != 1):
            raise ValueError("k_cache and v_cache must be [planes, rows, head_dim] with the same strides, rows contiguous")
    e = k_cache.element_size()
    p = KvCommitParams()
    p.num_planes, p.row_bytes, p.prefix_len, p.n_tree = planes, d * e, prefix_len, n_tree
    p.k_cache, p.v_cache = _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache")
    p.plane_stride_bytes = (k_cache.stride(0) if planes > 1 else rows * k_cache.stride(1)) * e
    p.row_stride_bytes = k_cache.stride(1) * e
    p.path, p.path_len = _dev(path, "path", torch.int32), _dev(path_len, "path_len", torch.int32)
    p.new_prefix_len = _dev(new_prefix_len, "new_prefix_len", torch.int32)
    p.prefix_len_dev = _dev(prefix_len_dev, "prefix_len_dev", torch.int32)
    p.dev_status = _dev(dev_status, "dev_status", torch.int32)
    _check("seq_tree_kv_commit", load().seq_tree_kv_commit(C.byref(p), _stream(stream)))


class HostStep:
    """One whole verify step fed from pinned HOST buffers: per call it copies the step's inputs to
    the device, builds the ancestor mask (inside the attention kernel with ``fused_mask``, else by a
    launch of its own), runs attention and verification, and copies the results (attention output,
    path, bonus token) back.  Device staging buffers are allocated once here.

    ``resident_cache``: the prefix rows of the key/value cache are copied once, here, and a step copies only what a
    step changes: the tree's rows ``[prefix_len, prefix_len + n)`` of every head, the queries, the tree, the logits
    and the uniforms.  ``two_streams``: the logits, tokens and uniforms travel on a second stream while the first
    copies q/k/v and runs the attention; the verification waits for them, and the attention output returns on the
    second stream while the verification runs."""

    def __init__(self, q, k_cache, v_cache, parent, prefix_len, tokens, target_logits, draft_logits, temperature,
                 uniforms, device="cuda", fused_mask: bool = False, kernel: int = KERNEL_AUTO,
                 resident_cache: bool = False, two_streams: bool = False):
        self.host_in = [t if t.is_pinned() else t.pin_memory()
                        for t in (q, k_cache, v_cache, parent, tokens, target_logits, draft_logits, uniforms)]
        self.dev_in = [torch.empty_like(t, device=device) for t in self.host_in]
        dq, dk, dv, dparent, dtok, dtl, ddl, du = self.dev_in
        n = parent.shape[0]
        self.mask = torch.empty((n, (n + 31) // 32), dtype=torch.int32, device=device)
        self.depth = torch.empty(n, dtype=torch.int32, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.fused_mask = fused_mask
        self.attn = AttentionCall(dq, dk, dv, None if fused_mask else self.mask, prefix_len, parent=dparent,
                                  dev_status=self.status, kernel=kernel)
        self.verify = VerifyCall(dparent, dtok, dtl, ddl, temperature, du, dev_status=self.status)
        self.host_out = [torch.empty_like(self.attn.out, device="cpu").pin_memory(),
                         torch.empty(n, dtype=torch.int32).pin_memory(),
                         torch.empty(1, dtype=torch.int32).pin_memory(),
                         torch.empty(1, dtype=torch.int32).pin_memory()]
        # (host, device) pairs per group: what the attention needs, what only the verification needs
        hq, hk, hv, hparent, htok, htl, hdl, hu = self.host_in
        if resident_cache:
            dk.copy_(hk)
            dv.copy_(hv)
            rows = slice(prefix_len, prefix_len + n)
            kv_pairs = [(hk[:, rows], dk[:, rows]), (hv[:, rows], dv[:, rows])]
        else:
            kv_pairs = [(hk, dk), (hv, dv)]
        self.copies_attention = [(hq, dq)] + kv_pairs + [(hparent, dparent)]
        self.copies_verify = [(htok, dtok), (htl, dtl), (hdl, ddl), (hu, du)]
        self.h2d_bytes = sum(h.numel() * h.element_size() for h, _ in self.copies_attention + self.copies_verify)
        self.d2h_bytes = sum(t.numel() * t.element_size() for t in self.host_out)
        self.side = torch.cuda.Stream(device=device) if two_streams else None
        self.ev_inputs = torch.cuda.Event() if two_streams else None
        self.ev_attention = torch.cuda.Event() if two_streams else None
        self.ev_side_done = torch.cuda.Event() if two_streams else None
        self.ev_start = torch.cuda.Event() if two_streams else None

    def run(self, stream=None):
        main = stream if stream is not None else torch.cuda.current_stream()
        with torch.cuda.stream(main):
            if self.side is not None:
                self.ev_start.record(main)
                with torch.cuda.stream(self.side):
                    self.side.wait_event(self.ev_start)  # not before the previous step has finished with the buffers
                    for h, d in self.copies_verify:
                        d.copy_(h, non_blocking=True)
                    self.ev_inputs.record(self.side)
            for h, d in self.copies_attention:
                d.copy_(h, non_blocking=True)
            if self.side is None:
                for h, d in self.copies_verify:
                    d.copy_(h, non_blocking=True)
            if not self.fused_mask:
                seq_tree_mask_from_parents(self.dev_in[3], mask_bits=self.mask, depth=self.depth, dev_status=self.status,
                                           stream=main)
            self.attn.run(main)
            if self.side is not None:
                self.ev_attention.record(main)
                main.wait_event(self.ev_inputs)
            self.verify.run(main)
            if self.side is not None:
                with torch.cuda.stream(self.side):
                    self.side.wait_event(self.ev_attention)
                    self.host_out[0].copy_(self.attn.out, non_blocking=True)
                    self.ev_side_done.record(self.side)
            else:
                self.host_out[0].copy_(self.attn.out, non_blocking=True)
            for h, d in zip(self.host_out[1:], (self.verify.path, self.verify.path_len, self.verify.bonus_token)):
                h.copy_(d, non_blocking=True)
            if self.side is not None:
                main.wait_event(self.ev_side_done)  # a caller that waits for `stream` has everything
        return self.host_out


def seq_tree_probe_stream_read(buf: torch.Tensor, sink: torch.Tensor, stream=None) -> None:
    """Measurement aid: one read-only pass over ``buf`` (device, contiguous); ``sink`` int64 device scratch of at
    least 4 x SM count words."""
    nbytes = buf.numel() * buf.element_size()
    _check("seq_tree_probe_stream_read",
           load().seq_tree_probe_stream_read(_dev(buf, "buf"), nbytes, _dev(sink, "sink", torch.int64), sink.numel(), _stream(stream)))


def seq_tree_probe_dependent_load(src: torch.Tensor, dst: torch.Tensor, stream=None) -> None:
    """Measurement aid: a one-warp kernel that loads src[0] and stores it, plus one, to dst[0]."""
    _check("seq_tree_probe_dependent_load",
           load().seq_tree_probe_dependent_load(_dev(src, "src", torch.int32), _dev(dst, "dst", torch.int32), _stream(stream)))
