"""ctypes front end of the fp64 CPU oracle (``seq_oracle.c``).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only tests, the smoke check and the
benchmark's ``cpu_baseline`` / ``--impl reference`` legs may import this
module.  It shares nothing with the CUDA library; arrays cross the boundary as
plain numpy buffers.  All arithmetic lives in the C file; this module only
builds it, converts inputs to the exact fp64 value of what the caller holds,
and shapes the outputs.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "seq_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None

VARIANT_SEQUOIA = 0
VARIANT_SPECINFER = 1

BAD_PARENT, BAD_TOKEN, NONFINITE, DEGENERATE = 1, 2, 4, 8
BAD_PATH = 32


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2 -fopenmp) if the library is missing or stale."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.run(
                ["gcc", "-O2", "-fopenmp", "-std=c99", "-shared", "-fPIC", _SRC, "-o", tmp, "-lm"],
                check=True,
            )
            os.replace(tmp, _LIB)
    return _LIB


def _p(arr, typ):
    return arr.ctypes.data_as(C.POINTER(typ)) if arr is not None else None


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        i32, i64, f64 = C.c_int32, C.c_int64, C.c_double
        pi32, pu32, pf32, pf64 = (C.POINTER(t) for t in (C.c_int32, C.c_uint32, C.c_float, C.c_double))
        L.orc_num_threads.restype = C.c_int
        L.orc_mask_from_parents.argtypes = [pi32, i32, pu32, i32, pi32]
        L.orc_tree_attention.argtypes = [pf64, pf64, pf64, pi32, i32, i32, i32, i32, i32, i32, f64, pf64, pf64]
        L.orc_softmax_T.argtypes = [pf32, i32, f64, pf64]
        L.orc_softmax_T.restype = None
        L.orc_alg2_node.argtypes = [pf64, pf64, i32, pi32, pf64, i32, i32, pi32, pf64, pf64, pf64, pf64]
        L.orc_draft_sample.argtypes = [pf32, i32, f64, pf32, i32, pi32, pf64, pf64]
        L.orc_sample_inverse_cdf.argtypes = [pf64, i32, f64]
        L.orc_sample_inverse_cdf.restype = i32
        L.orc_tree_verify.argtypes = [i32, i32, pi32, pi32, pf32, i64, pf32, i64, f64, pf32, i32,
                                      pi32, pi32, pi32, pf64, pi32, pf64, pf64]
        L.orc_tree_verify_target_sample.argtypes = [i32, i32, pi32, pi32, pf32, i64, f64, pf32, pi32, pi32, pi32, pf64, pi32, pf64]
        L.orc_top_p.argtypes = [pf32, i32, f64, f64, C.c_void_p, pf64, pi32]
        L.orc_top_p.restype = i32
        L.orc_kv_commit.argtypes = [C.c_void_p, C.c_void_p, i64, i64, i64, i32, i32, pi32, i32]
        L.orc_alg3_chain.argtypes = [pf64, pf64, i32, i32, pi32, pf64, f64, pi32]
        L.orc_alg3_chain.restype = i32
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _f64(x) -> np.ndarray:
    """Exact fp64 value of a numpy array or a torch tensor of any float type."""
    if hasattr(x, "detach"):
        x = x.detach().cpu().double().numpy()
    return np.ascontiguousarray(x, dtype=np.float64)


def _i32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(x, dtype=np.int32)


def _f32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(x, dtype=np.float32)


def mask_from_parents(parent, words_per_row: int | None = None):
    parent = _i32(parent)
    n = parent.shape[0]
    wpr = words_per_row or (n + 31) // 32
    mask = np.empty((n, wpr), dtype=np.uint32)
    depth = np.empty(n, dtype=np.int32)
    flags = lib().orc_mask_from_parents(_p(parent, C.c_int32), n, _p(mask, C.c_uint32), wpr, _p(depth, C.c_int32))
    return mask, depth, int(flags)


def tree_attention(q, k, v, parent, prefix_len: int, scale: float | None = None):
    """q [n,Hq,d]; k,v [Hkv,rows,d] with tree rows at [prefix_len, prefix_len+n). Returns out, lse, flags."""
    q, k, v, parent = _f64(q), _f64(k), _f64(v), _i32(parent)
    n, Hq, d = q.shape
    Hkv, rows, _ = k.shape
    assert v.shape == k.shape and rows >= prefix_len + n and Hq % Hkv == 0
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.empty_like(q)
    lse = np.empty((Hq, n), dtype=np.float64)
    flags = lib().orc_tree_attention(_p(q, C.c_double), _p(k, C.c_double), _p(v, C.c_double),
                                     _p(parent, C.c_int32), n, prefix_len, Hq, Hkv, d, rows, float(scale),
                                     _p(out, C.c_double), _p(lse, C.c_double))
    return out, lse, int(flags)


def softmax_T(logits, T: float) -> np.ndarray:
    logits = _f32(logits)
    out = np.empty(logits.shape[0], dtype=np.float64)
    lib().orc_softmax_T(_p(logits, C.c_float), logits.shape[0], float(T), _p(out, C.c_double))
    return out


def draft_sample(logits, T: float, u, k: int) -> dict:
    """k tokens drawn without replacement from softmax(logits/T) by exponential sort with the uniforms u."""
    logits, u = _f32(logits), _f32(u)
    V = logits.shape[0]
    assert u.shape[0] == V and k >= 0
    out = np.full(max(k, 1), -1, dtype=np.int32)
    keys = np.empty(V, dtype=np.float64)
    gap = C.c_double(0.0)
    lib().orc_draft_sample(_p(logits, C.c_float), V, float(T), _p(u, C.c_float), k, _p(out, C.c_int32),
                           _p(keys, C.c_double), C.byref(gap))
    return dict(tokens=out[:k].copy(), keys=keys, min_rel_gap=float(gap.value))


def alg2_node(P, Q, child_tok, child_u, variant: int = VARIANT_SEQUOIA) -> dict:
    """Algorithm 2 at one node given distributions P, Q, the drawn children and their uniforms."""
    R, D = _f64(P).copy(), _f64(Q).copy()
    tok, u = _i32(child_tok), _f64(child_u)
    k = tok.shape[0]
    acc = C.c_int32(-1)
    ratio, rnum, dden = (np.empty(max(k, 1), dtype=np.float64) for _ in range(3))
    gap = C.c_double(0.0)
    flags = lib().orc_alg2_node(_p(R, C.c_double), _p(D, C.c_double), R.shape[0], _p(tok, C.c_int32),
                                _p(u, C.c_double), k, variant, C.byref(acc), _p(ratio, C.c_double),
                                _p(rnum, C.c_double), _p(dden, C.c_double), C.byref(gap))
    return dict(accepted=int(acc.value), R=R, D=D, ratio=ratio[:k], rnum=rnum[:k], dden=dden[:k],
                min_gap=float(gap.value), flags=int(flags))


def sample_inverse_cdf(R, u: float) -> int:
    R = _f64(R)
    return int(lib().orc_sample_inverse_cdf(_p(R, C.c_double), R.shape[0], float(u)))


def tree_verify(parent, tokens, target_logits, draft_logits, T: float, uniforms,
                variant: int = VARIANT_SEQUOIA) -> dict:
    parent, tokens = _i32(parent), _i32(tokens)
    tl, dl, un = _f32(target_logits), _f32(draft_logits), _f32(uniforms)
    n, V = tl.shape
    assert dl.shape == tl.shape and un.shape[0] == n + 1 and parent.shape[0] == n
    path = np.empty(n, dtype=np.int32)
    plen, bonus = C.c_int32(0), C.c_int32(-1)
    residual = np.empty(V, dtype=np.float64)
    next_child = np.empty(n, dtype=np.int32)
    ratio = np.empty(n, dtype=np.float64)
    gap = C.c_double(0.0)
    flags = lib().orc_tree_verify(n, V, _p(parent, C.c_int32), _p(tokens, C.c_int32), _p(tl, C.c_float), V,
                                  _p(dl, C.c_float), V, float(T), _p(un, C.c_float), variant,
                                  _p(path, C.c_int32), C.byref(plen), C.byref(bonus), _p(residual, C.c_double),
                                  _p(next_child, C.c_int32), _p(ratio, C.c_double), C.byref(gap))
    return dict(path=path[: plen.value].copy(), path_len=int(plen.value), bonus=int(bonus.value),
                residual=residual, next_child=next_child, ratio=ratio, min_gap=float(gap.value),
                flags=int(flags))


def tree_verify_target_sample(parent, tokens, target_logits, T: float, uniforms) -> dict:
    """Verification by sampling from the target at every visited node ("naive" / "top-k sampling")."""
    parent, tokens = _i32(parent), _i32(tokens)
    tl, un = _f32(target_logits), _f32(uniforms)
    n, V = tl.shape
    assert un.shape[0] == n + 1 and parent.shape[0] == n
    path = np.empty(n, dtype=np.int32)
    plen, bonus = C.c_int32(0), C.c_int32(-1)
    residual = np.empty(V, dtype=np.float64)
    next_child = np.empty(n, dtype=np.int32)
    gap = C.c_double(0.0)
    flags = lib().orc_tree_verify_target_sample(n, V, _p(parent, C.c_int32), _p(tokens, C.c_int32), _p(tl, C.c_float), V,
                                                float(T), _p(un, C.c_float), _p(path, C.c_int32), C.byref(plen),
                                                C.byref(bonus), _p(residual, C.c_double), _p(next_child, C.c_int32),
                                                C.byref(gap))
    return dict(path=path[: plen.value].copy(), path_len=int(plen.value), bonus=int(bonus.value), residual=residual,
                next_child=next_child, min_gap=float(gap.value), flags=int(flags))


def alg3_chain(p, q, x, r, u_final: float):
    p, q, x, r = _f64(p), _f64(q), _i32(x), _f64(r)
    gamma, V = q.shape
    assert p.shape == (gamma + 1, V)
    t = C.c_int32(-1)
    s = lib().orc_alg3_chain(_p(p, C.c_double), _p(q, C.c_double), V, gamma, _p(x, C.c_int32),
                             _p(r, C.c_double), float(u_final), C.byref(t))
    return int(s), int(t.value)


def kv_commit(cache, prefix_len: int, n_tree: int, path):
    """cache: numpy array [..., rows, d] of any item size (leading dimensions = planes).  Returns the committed
    copy (row L+i <- row L+path[i]) and the flags."""
    cache = np.ascontiguousarray(cache)
    path = _i32(path)
    rows, d = cache.shape[-2], cache.shape[-1]
    assert rows >= prefix_len + n_tree
    planes = int(np.prod(cache.shape[:-2], dtype=np.int64))
    out = np.empty_like(cache)
    flags = lib().orc_kv_commit(cache.ctypes.data, out.ctypes.data, planes, rows, d * cache.itemsize, prefix_len,
                                n_tree, _p(path, C.c_int32), path.shape[0])
    return out, int(flags)


def top_p(logits, T: float, top_p: float) -> dict:
    """Nucleus truncation of softmax(logits/T): keep mask [V] (bool), the filtered logits (-inf outside), the two
    margins of the decision (mass above top_p with the last kept token, mass below it without) and the flags."""
    logits = _f32(logits)
    V = logits.shape[0]
    keep = np.zeros(V, dtype=np.uint8)
    margins, flags = (C.c_double * 2)(), C.c_int32(0)
    kept = lib().orc_top_p(_p(logits, C.c_float), V, float(T), float(top_p), keep.ctypes.data, margins, C.byref(flags))
    keep = keep.astype(bool)
    return dict(keep=keep, kept=int(kept), filtered=np.where(keep, logits, np.float32(-np.inf)), over=float(margins[0]),
                under=float(margins[1]), min_gap=float(min(margins[0], margins[1])), flags=int(flags.value))
