"""GPU parity at the full workload sizes and in the corners the smaller cases leave open: every row of every
configuration's attention in the launch configuration the benchmark times, the largest configuration's
verification on its own tree, low temperature, the output law of the verification measured on GPU outputs, the
inverse CDF's fallback branch, and the stream schedule with fewer blocks than CTAs."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2402_12374_b200 import binding as B
from paper_2402_12374_b200 import workloads as W
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _cfg(name, **kw):
    return dataclasses.replace(W.CONFIGS[name], **kw)


# ---------------------------------------------------------------- attention, all rows, bench configuration ----
@pytest.mark.parametrize("name", ["tiny", "llama2-7b", "llama2-13b", "vicuna-33b", "llama3-70b"])
def test_attention_every_row_of_every_config_as_the_benchmark_launches_it(name):
    """Every node x every head against the oracle (no sampling of rows), launched as bench.py launches it: mask
    derived from the parent array inside the kernel, kernel and schedule chosen by the library (the 768-node
    configuration runs the stream schedule, its cut tiles completed from workspace pieces)."""
    cfg = W.CONFIGS[name]
    ai = W.make_attention_inputs(cfg, 0)
    d = G.dev()
    n, Hq = cfg.n_tree, cfg.num_q_heads
    st = torch.zeros(1, dtype=torch.int32, device=d)
    lse = torch.empty((Hq, n), dtype=torch.float32, device=d)
    call = B.AttentionCall(ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d), None, cfg.prefix_len, parent=ai.parent.to(d),
                           lse=lse, dev_status=st)
    if name == "llama3-70b":
        assert call.workspace_bytes_needed > 0, "the largest configuration is expected to take the stream schedule"
    out = call.run()
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    ref, rlse, _ = O.tree_attention(ai.q, ai.k_cache, ai.v_cache, ai.parent, cfg.prefix_len)
    err = np.abs(out.double().cpu().numpy() - ref)
    assert err.max() < G.ATTN_TOL[ai.q.dtype], f"max abs err {err.max()} at {np.unravel_index(err.argmax(), err.shape)}"
    assert np.abs(lse.double().cpu().numpy() - rlse).max() < 2e-2
    # the mean error tells rounding (about 1e-3) from a wrong block, which a 2e-2 bound on N(0,1) values could hide
    assert err.mean() < 2e-3


def test_tensor_core_attention_stream_schedule_with_fewer_blocks_than_ctas():
    """Stream schedule forced on a problem whose flattened block space (26 positions) is shorter than the number of
    CTAs a GPU offers: ranges must not be empty, and a tile cut over several CTAs must still be completed."""
    for (n, L, Hq, Hkv) in [(16, 300, 2, 2), (40, 700, 1, 1), (130, 1000, 4, 4)]:
        cfg = _cfg("tiny", num_q_heads=Hq, num_kv_heads=Hkv, prefix_len=L, n_tree=n, max_depth=12)
        ai = W.make_attention_inputs(cfg, 31, dtype="bf16")
        d = G.dev()
        st = torch.zeros(1, dtype=torch.int32, device=d)
        out = torch.full((n, Hq, 128), float("nan"), dtype=torch.bfloat16, device=d)
        call = B.AttentionCall(ai.q.to(d), ai.k_cache.to(d), ai.v_cache.to(d), None, L, parent=ai.parent.to(d), out=out,
                               dev_status=st, kernel=B.KERNEL_TENSOR_CORE_STREAM)
        assert call.workspace_bytes_needed > 0
        call.run()
        torch.cuda.synchronize()
        assert int(st.item()) == 0 and torch.isfinite(out).all(), "some tile was never completed"
        ref, _, _ = O.tree_attention(ai.q, ai.k_cache, ai.v_cache, ai.parent, L)
        assert np.abs(out.double().cpu().numpy() - ref).max() < 2e-2


# ---------------------------------------------------------------- verification -----------------------------
@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_verify_llama3_70b_config_on_its_own_tree(seed):
    """The largest configuration in the default (Sequoia) mode: 768 nodes drawn with fan-out <= 16 and depth <= 20,
    128256 logits per row, T = 0.6."""
    cfg = W.CONFIGS["llama3-70b"]
    vi = W.make_verify_inputs(cfg, 0.6, seed)
    assert G.check_verify(vi) in ("ok", "excluded")


@pytest.mark.parametrize("name,T", [("llama2-13b", 1.0), ("vicuna-33b", 0.6)])
def test_verify_mid_size_configs_more_seeds(name, T):
    cfg = W.CONFIGS[name]
    outcomes = [G.check_verify(W.make_verify_inputs(cfg, T, seed)) for seed in range(2, 8)]
    assert outcomes.count("ok") >= 3, outcomes


@pytest.mark.parametrize("name,seeds", [("tiny", range(6)), ("llama2-7b", range(4))])
def test_verify_low_temperature(name, seeds):
    """T = 0.2, the lowest temperature of the paper's figures: distributions are peaked, rejections leave little
    residual mass, which is where single precision is thinnest."""
    cfg = W.CONFIGS[name]
    outcomes = [G.check_verify(W.make_verify_inputs(cfg, 0.2, seed)) for seed in seeds]
    assert outcomes.count("ok") >= len(outcomes) - 1, outcomes
    outcomes = [G.check_verify(W.make_verify_inputs(cfg, 0.2, seed), specinfer=True) for seed in list(seeds)[:2]]
    assert outcomes.count("ok") >= 1, outcomes


def _chi2_ok(counts, probs, trials):
    exp = probs * trials
    keep = exp >= 5
    stat = ((counts[keep] - exp[keep]) ** 2 / exp[keep]).sum()
    dof = keep.sum() - 1
    if dof < 2:  # a distribution this peaked leaves too few cells for a chi-square: every token within 6 binomial sigmas
        return bool((np.abs(counts - exp) <= 6 * np.sqrt(exp * (1 - probs)) + 1).all()), stat, dof
    return stat < dof + 6 * np.sqrt(2 * dof), stat, dof


@pytest.mark.parametrize("T", [1.0, 0.6, 0.2])
@pytest.mark.parametrize("V,k", [(24, 1), (24, 4), (24, 24), (64, 4), (64, 64)])
def test_monte_carlo_on_gpu_outputs_follows_the_target(T, V, k):
    """The property Algorithm 2 exists for (appendix, proof of correctness): whatever the draft, the emitted token
    is distributed as softmax(target / T).  Root + k children drawn without replacement from the draft (numpy's
    Gumbel arg-sort, on the host), fresh uniforms per trial, 24000 trials through seq_tree_verify_batch; the
    first emitted token (the accepted child's, else the bonus) against the target by chi-square, and against the
    draft, which must fail."""
    trials, chunk = 24000, 6000
    rng = np.random.default_rng(4000 + 10 * V + k)
    tl = (2.0 * rng.standard_normal(V)).astype(np.float32)
    dl = (tl + 1.5 * rng.standard_normal(V)).astype(np.float32)
    n = k + 1
    d = G.dev()
    parent = torch.from_numpy(W.star_tree(n)).to(d).unsqueeze(0).repeat(chunk, 1).contiguous()
    TL = torch.from_numpy(tl).to(d).expand(chunk, n, V).contiguous()
    DL = torch.from_numpy(dl).to(d).expand(chunk, n, V).contiguous()
    counts = np.zeros(V)
    accepted = 0
    st = torch.zeros(1, dtype=torch.int32, device=d)
    for c in range(trials // chunk):
        keys = dl.astype(np.float64) / T + rng.gumbel(size=(chunk, V))
        kids = np.argsort(-keys, axis=1)[:, :k].astype(np.int32)
        tokens = np.zeros((chunk, n), np.int32)
        tokens[:, 1:] = kids
        U = rng.random((chunk, n + 1), dtype=np.float32)
        path, plen, bonus = B.seq_tree_verify_batch(parent, torch.from_numpy(tokens).to(d), TL, DL, T,
                                                    torch.from_numpy(U).to(d), dev_status=st)
        torch.cuda.synchronize()
        plen, bonus, path = plen.cpu().numpy(), bonus.cpu().numpy(), path.cpu().numpy()
        acc = plen >= 2
        first = np.where(acc, tokens[np.arange(chunk), path[:, 1].clip(0, n - 1)], bonus)
        counts += np.bincount(first, minlength=V)
        accepted += int(acc.sum())
    assert int(st.item()) == 0
    p = np.exp((tl.astype(np.float64) - tl.max()) / T)
    q = np.exp((dl.astype(np.float64) - dl.max()) / T)
    ok, stat, dof = _chi2_ok(counts, p / p.sum(), trials)
    assert ok, (stat, dof)
    if k == V:
        assert accepted == trials  # k = vocabulary size: some child is always accepted
    if np.abs(p / p.sum() - q / q.sum()).sum() > 0.1:  # (at T = 0.2 the two can share one dominant token)
        assert not _chi2_ok(counts, q / q.sum(), trials)[0], "the check cannot tell the target from the draft"


def test_monte_carlo_on_gpu_outputs_single_launch_kernel():
    """The same law through seq_tree_verify itself (the single-request kernel and schedule), fewer trials."""
    V, k, T, trials = 40, 3, 0.7, 1500
    rng = np.random.default_rng(77)
    tl = (2.0 * rng.standard_normal(V)).astype(np.float32)
    dl = (tl + 1.5 * rng.standard_normal(V)).astype(np.float32)
    n = k + 1
    d = G.dev()
    parent = torch.from_numpy(W.star_tree(n)).to(d)
    TL = torch.from_numpy(tl).to(d).expand(n, V).contiguous()
    DL = torch.from_numpy(dl).to(d).expand(n, V).contiguous()
    keys = dl.astype(np.float64) / T + rng.gumbel(size=(trials, V))
    kids = np.argsort(-keys, axis=1)[:, :k].astype(np.int32)
    tokens = np.zeros((trials, n), np.int32)
    tokens[:, 1:] = kids
    tok_d = torch.from_numpy(tokens).to(d)
    U = torch.from_numpy(rng.random((trials, n + 1), dtype=np.float32)).to(d)
    st = torch.zeros(1, dtype=torch.int32, device=d)
    paths = torch.zeros((trials, n), dtype=torch.int32, device=d)
    plens = torch.zeros(trials, dtype=torch.int32, device=d)
    bonuses = torch.zeros(trials, dtype=torch.int32, device=d)
    for t in range(trials):
        B.VerifyCall(parent, tok_d[t], TL, DL, T, U[t], path=paths[t], path_len=plens[t:t + 1],
                     bonus_token=bonuses[t:t + 1], dev_status=st).run()
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    plen, bonus, path = plens.cpu().numpy(), bonuses.cpu().numpy(), paths.cpu().numpy()
    first = np.where(plen >= 2, tokens[np.arange(trials), path[:, 1].clip(0, n - 1)], bonus)
    p = np.exp((tl.astype(np.float64) - tl.max()) / T)
    ok, stat, dof = _chi2_ok(np.bincount(first, minlength=V).astype(float), p / p.sum(), trials)
    assert ok, (stat, dof)


def test_verify_bonus_draw_falls_back_to_the_last_token_with_mass():
    """The inverse CDF's second branch (the cumulative sum never exceeds the uniform): the last token with R > 0,
    not the last token of the vocabulary.  Reached with a uniform of 1 (outside [0, 1), defined all the same);
    the largest uniform below 1 must stay within the rounding band of the oracle's CDF."""
    rng = np.random.default_rng(5)
    V = 1000
    for trial, (n, tail) in enumerate([(1, 300), (1, 1), (6, 77), (6, 513)]):
        parent = W.star_tree(n)
        tl = (1.5 * rng.standard_normal((n, V))).astype(np.float32)
        tl[:, V - tail:] = -np.inf                      # trailing tokens without mass
        dl = (tl + rng.standard_normal((n, V)).astype(np.float32)).astype(np.float32)
        dl[:, V - tail:] = -np.inf
        tokens = W.draw_children_tokens(parent, dl, 0.8, rng)
        u = np.full(n + 1, 0.9999, np.float32)          # children are rejected: the draw is from a residual
        for last in (np.float32(1.0), np.nextafter(np.float32(1.0), np.float32(0.0))):
            u[-1] = last
            vi = W.VerifyInputs(torch.from_numpy(parent), torch.from_numpy(tokens), torch.from_numpy(tl),
                                torch.from_numpy(dl), torch.from_numpy(u.copy()), 0.8)
            got = G.run_verify(vi)
            ref = O.tree_verify(parent, tokens, tl, dl, 0.8, u)
            assert got["status"] == ref["flags"] == 0
            if ref["min_gap"] < G.GAP:
                continue
            assert got["path"].tolist() == ref["path"].tolist()
            if last == 1.0:
                want = int(np.flatnonzero(ref["residual"] > 0)[-1])
                assert ref["bonus"] == want < V - tail   # the oracle's own branch, pinned on the CPU side as well
                # single precision may flush a vanishing probability that fp64 keeps: the token must carry mass in
                # the GPU's own residual and nothing after it may
                g = got["residual"]
                assert g[got["bonus"]] > 0 and not (g[got["bonus"] + 1:] > 0).any()
                assert got["bonus"] <= want and ref["residual"][got["bonus"] + 1:].sum() < 1e-30
            else:
                cdf = np.cumsum(ref["residual"])
                t = got["bonus"]
                lo = cdf[t - 1] if t > 0 else 0.0
                assert lo - G.GAP <= float(last) < cdf[t] + G.GAP and ref["residual"][t] > 0


@pytest.mark.parametrize("name,T,seeds", [("tiny", 0.6, range(4)), ("llama2-7b", 0.6, range(4)), ("llama2-7b", 1.0, range(2)),
                                          ("llama3-70b", 0.6, range(1))])
def test_bf16_logits_are_widened_exactly(name, T, seeds):
    """SEQ_VERIFY_LOGITS_BF16: both logit matrices in bfloat16 (half the bytes per visited node).  The oracle is given
    the same values as fp32 (the widening is exact), so the parity rule is the usual one; also with a ragged
    vocabulary (rows that end inside an 8-byte load) and for the variant without the draft update."""
    cfg = W.CONFIGS[name]
    outcomes = []
    for seed in seeds:
        vi = W.make_verify_inputs(cfg, T, seed, vocab=None if seed % 2 == 0 or cfg.vocab > 100000 else 30001)
        vi.target_logits = vi.target_logits.to(torch.bfloat16).float()
        vi.draft_logits = vi.draft_logits.to(torch.bfloat16).float()
        outcomes.append(G.check_verify(vi, bf16_logits=True))
        if seed == 0:
            outcomes.append(G.check_verify(vi, bf16_logits=True, specinfer=True))
    assert outcomes.count("ok") >= len(outcomes) - 1, outcomes
