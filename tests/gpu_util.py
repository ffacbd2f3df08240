"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI and the fp64 oracle
on the same seeded inputs and compare under the stated tolerances."""
from __future__ import annotations

import numpy as np
import torch

from oracle import oracle as O
from paper_2402_12374_b200 import binding as B
from paper_2402_12374_b200 import workloads as W

ATTN_TOL = {torch.float16: 2e-2, torch.bfloat16: 2e-2, torch.float32: 1e-5}  # max abs error of the output
RESID_TOL = 1e-5   # max abs error of residual probabilities
GAP = 1e-5         # |u - ratio| below this: the accept decision is within rounding, outcome excluded
SCHEDULE = "auto"  # schedule of seq_tree_verify in run_verify: set per test by the `verify_schedule` fixture


def dev():
    return torch.device("cuda:0")


def gpu_mask(parent_np):
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    mask, depth = B.seq_tree_mask_from_parents(torch.as_tensor(parent_np, dtype=torch.int32).to(dev()), dev_status=st)
    return mask, depth, st


def run_attention(ai: W.AttentionInputs, kernel=B.KERNEL_AUTO, want_lse=True, scale=0.0):
    d = dev()
    mask, _, st = gpu_mask(ai.parent.numpy())
    n, Hq, _ = ai.q.shape
    lse = torch.empty((Hq, n), dtype=torch.float32, device=d) if want_lse else None
    out = B.seq_tree_attention(ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d), mask, ai.prefix_len, lse=lse,
                               dev_status=st, kernel=kernel, softmax_scale=scale)
    torch.cuda.synchronize()
    return out, lse, int(st.item())


def check_attention(ai: W.AttentionInputs, kernel=B.KERNEL_AUTO, scale=0.0, rows=None):
    """Element-by-element comparison with the oracle (all rows, or the sampled `rows` of nodes)."""
    out, lse, status = run_attention(ai, kernel, scale=scale)
    assert status == 0
    rows_used = ai.k_cache.shape[1]
    if rows is None:
        ref, rlse, _ = O.tree_attention(ai.q, ai.k_cache[:, :rows_used], ai.v_cache[:, :rows_used], ai.parent,
                                        ai.prefix_len, scale=scale or None)
        got, glse = out.double().cpu().numpy(), lse.double().cpu().numpy()
    else:
        # the oracle computes a node's row from that node's path alone, so any subset of nodes that is
        # closed under "parent" can be checked on its own
        keep = sorted(set(int(a) for r in rows for a in _path(ai.parent.numpy(), r)))
        idx = {a: j for j, a in enumerate(keep)}
        parent_sub = np.array([-1 if ai.parent[a] < 0 else idx[int(ai.parent[a])] for a in keep], np.int32)
        L = ai.prefix_len
        sel = torch.tensor(list(range(L)) + [L + a for a in keep])
        ref, rlse, _ = O.tree_attention(ai.q[keep], ai.k_cache[:, sel], ai.v_cache[:, sel], parent_sub, L,
                                        scale=scale or None)
        got, glse = out[keep].double().cpu().numpy(), lse[:, keep].double().cpu().numpy()
    tol = ATTN_TOL[ai.q.dtype]
    err = np.abs(got - ref).max()
    assert err < tol, f"attention max abs err {err} (tol {tol})"
    lerr = np.abs(glse - rlse).max()
    assert lerr < (1e-4 if ai.q.dtype == torch.float32 else 2e-2), f"lse err {lerr}"
    return err


def _path(parent, i):
    out = []
    while i >= 0:
        out.append(i)
        i = int(parent[i])
    return out


def run_verify(vi: W.VerifyInputs, all_nodes=False, want_residual=True, specinfer=False, target_sample=False, bf16_logits=False):
    d = dev()
    n, V = vi.target_logits.shape
    st = torch.zeros(1, dtype=torch.int32, device=d)
    residual = torch.full((V,), float("nan"), dtype=torch.float32, device=d) if want_residual else None
    nxt = torch.full((n,), -9, dtype=torch.int32, device=d)
    # rows padded to a multiple of 4 floats (NaN in the padding) so every row stays 16-byte aligned
    Vp = (V + 3) // 4 * 4
    tl = torch.full((n, Vp), float("nan"), dtype=torch.float32, device=d)
    tl[:, :V] = vi.target_logits.to(d)
    dl = None
    if vi.draft_logits is not None:
        dl = torch.full((n, Vp), float("nan"), dtype=torch.float32, device=d)
        dl[:, :V] = vi.draft_logits.to(d)
        dl = dl[:, :V]
    if bf16_logits:  # (the caller made sure the values are exact in bfloat16; the padded row stride is kept)
        tl = tl.to(torch.bfloat16)
        if dl is not None:
            dl_full = torch.full((n, Vp), float("nan"), dtype=torch.bfloat16, device=d)
            dl_full[:, :V] = dl.to(torch.bfloat16)
            dl = dl_full[:, :V]
    call = B.VerifyCall(vi.parent.to(d), vi.tokens.to(d), tl[:, :V], dl,
                        vi.temperature, vi.uniforms.to(d), residual_out=residual, next_child_out=nxt,
                        all_nodes=all_nodes, dev_status=st, specinfer=specinfer, target_sample=target_sample,
                        schedule="auto" if all_nodes else SCHEDULE)
    call.run()
    torch.cuda.synchronize()
    plen = int(call.path_len.item())
    return dict(rows_read=call.rows_read(), path=call.path[:plen].cpu().numpy(), path_len=plen, bonus=int(call.bonus_token.item()),
                residual=None if residual is None else residual.double().cpu().numpy(),
                next_child=nxt.cpu().numpy(), status=int(st.item()))


def check_verify(vi: W.VerifyInputs, specinfer=False, bf16_logits=False):
    """Path and bonus identical to the oracle's (outside the rounding band), residual within 1e-5.
    Returns 'ok' or 'excluded'."""
    got = run_verify(vi, specinfer=specinfer, bf16_logits=bf16_logits)
    ref = O.tree_verify(vi.parent, vi.tokens, vi.target_logits, vi.draft_logits, vi.temperature, vi.uniforms,
                        variant=O.VARIANT_SPECINFER if specinfer else O.VARIANT_SEQUOIA)
    assert got["status"] == ref["flags"] == 0
    if ref["min_gap"] < GAP:
        return "excluded"
    assert got["path"].tolist() == ref["path"].tolist(), (got["path"], ref["path"])
    visited = ref["next_child"] != -2
    assert np.array_equal(got["next_child"], ref["next_child"]), "per-node decisions differ"
    assert visited.sum() == got["path_len"]
    rerr = np.abs(got["residual"] - ref["residual"]).max()
    assert rerr < RESID_TOL, f"residual max abs err {rerr}"
    assert abs(got["residual"].sum() - 1.0) < 1e-5 and (got["residual"] >= 0).all()
    # bonus: identical, or inside the rounding band of the oracle's CDF at the supplied uniform
    if got["bonus"] != ref["bonus"]:
        cdf = np.cumsum(ref["residual"])
        u = float(vi.uniforms[-1])
        t = got["bonus"]
        lo = cdf[t - 1] if t > 0 else 0.0
        assert lo - GAP <= u < cdf[t] + GAP and ref["residual"][t] > 0, (t, ref["bonus"], u, lo, cdf[t])
        return "excluded"
    return "ok"


def check_verify_target_sample(vi: W.VerifyInputs, with_draft=False):
    """SEQ_VERIFY_TARGET_SAMPLE: path, per-node decisions and bonus identical to the oracle's walk that samples
    from the target at every node (outside the rounding band of its inverse CDFs); residual_out = the target
    distribution at the last node, within 1e-5.  Returns 'ok' or 'excluded'."""
    if not with_draft:
        vi = W.VerifyInputs(vi.parent, vi.tokens, vi.target_logits, None, vi.uniforms, vi.temperature)
    got = run_verify(vi, target_sample=True)
    ref = O.tree_verify_target_sample(vi.parent, vi.tokens, vi.target_logits, vi.temperature, vi.uniforms)
    assert got["status"] == ref["flags"] == 0
    if ref["min_gap"] < GAP:
        return "excluded"
    assert got["path"].tolist() == ref["path"].tolist(), (got["path"], ref["path"])
    assert np.array_equal(got["next_child"], ref["next_child"]), "per-node decisions differ"
    assert got["bonus"] == ref["bonus"]
    rerr = np.abs(got["residual"] - ref["residual"]).max()
    assert rerr < RESID_TOL, f"residual max abs err {rerr}"
    assert abs(got["residual"].sum() - 1.0) < 1e-5 and (got["residual"] >= 0).all()
    return "ok"


def steer_tokens_to_samples(vi, every=1):
    """Rewrites the first child's token of every `every`-th internal node to the token the oracle's inverse CDF
    draws there, so that the walk goes deep; returns the number of nodes steered."""
    kids = W.children_lists(vi.parent.numpy())
    steered = 0
    for v, ch in enumerate(kids):
        if ch and v % every == 0:
            P = O.softmax_T(vi.target_logits[v], vi.temperature)
            vi.tokens[ch[0]] = O.sample_inverse_cdf(P, float(vi.uniforms[v]))
            steered += 1
    return steered


def check_verify_all_nodes(vi: W.VerifyInputs):
    """SEQ_VERIFY_ALL_NODES: every internal node's accept/reject loop against Algorithm 2 run by the
    oracle on that node's two distributions."""
    got = run_verify(vi, all_nodes=True, want_residual=False)
    parent = vi.parent.numpy()
    kids = W.children_lists(parent)
    n_checked = n_excluded = 0
    for v in range(len(parent)):
        if not kids[v]:
            assert got["next_child"][v] == -1
            continue
        tok = vi.tokens.numpy()[kids[v]]
        if vi.temperature == 0:
            a = int(np.argmax(vi.target_logits[v].numpy()))
            hit = [c for c in kids[v] if vi.tokens[c] == a]
            expect = hit[0] if hit else -1
        else:
            P = O.softmax_T(vi.target_logits[v], vi.temperature)
            Q = O.softmax_T(vi.draft_logits[v], vi.temperature)
            r = O.alg2_node(P, Q, tok, vi.uniforms.numpy()[kids[v]].astype(np.float64))
            if r["min_gap"] < GAP:
                n_excluded += 1
                continue
            expect = kids[v][r["accepted"]] if r["accepted"] >= 0 else -1
        assert got["next_child"][v] == expect, (v, got["next_child"][v], expect)
        n_checked += 1
    return n_checked, n_excluded
