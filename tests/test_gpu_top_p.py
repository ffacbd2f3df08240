"""GPU parity of seq_tree_top_p_filter against the oracle: the kept set of every row whose decision is not within
rounding of the boundary (bit-exact logits inside, -inf outside), equal logits at the cut, in place, strides, flags,
and the chain filter -> verification against the oracle's verification of the oracle's filtered logits."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2402_12374_b200 import binding as B, workloads as W
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

# The order of the tokens is that of the fp32 logits' bits on both sides: exact.  Only the cumulative mass is computed
# in lower precision on the GPU (fp32 exponent arguments and ex2.approx: about 1e-6 of the total mass), so the cut can
# sit one token away from the oracle's when the oracle's own margin on that side is below this band.
BAND = 3e-6


def _run(logits_np, T, tp, *, in_place=False, pad=0):
    d = G.dev()
    rows, V = logits_np.shape
    Vp = (V + 3) // 4 * 4 + pad
    buf = torch.full((rows, Vp), float("nan"), dtype=torch.float32, device=d)
    buf[:, :V] = torch.from_numpy(logits_np).to(d)
    src = buf[:, :V]
    out = src if in_place else torch.full((rows, Vp), 7.0, dtype=torch.float32, device=d)[:, :V]
    kept = torch.full((rows,), -1, dtype=torch.int32, device=d)
    st = torch.zeros(1, dtype=torch.int32, device=d)
    res = B.seq_tree_top_p_filter(src, T, tp, out=out, kept_out=kept, dev_status=st)
    torch.cuda.synchronize()
    if not in_place and (pad or Vp != V):
        assert torch.isnan(buf[:, V:]).all()  # the padding behind a row is not written
    return res.cpu().numpy(), kept.cpu().numpy(), int(st.item())


def _check(logits_np, T, tp, **kw):
    """Every row: the kept set is a prefix of the exact order (descending logit, equal logits by token id), bits
    inside untouched, -inf outside; its length is the oracle's, or one off on the side whose margin is inside the
    band.  Returns (rows identical to the oracle, status)."""
    got, kept, st = _run(logits_np, T, tp, **kw)
    n_same = 0
    for r in range(logits_np.shape[0]):
        x = logits_np[r]
        ref = O.top_p(x, T, tp)
        k = int(kept[r])
        order = np.lexsort((np.arange(x.size), -x.astype(np.float64)))
        mask = np.zeros(x.size, bool)
        mask[order[:k]] = True
        want = np.where(mask, x, np.float32(-np.inf))
        assert np.array_equal(got[r].view(np.uint32), want.view(np.uint32)), f"row {r}: not a prefix of the exact order"
        if k == ref["kept"]:
            n_same += 1
        elif k == ref["kept"] + 1:
            assert ref["over"] < BAND, (r, k, ref["kept"], ref["over"])
        elif k == ref["kept"] - 1:
            assert ref["under"] < BAND, (r, k, ref["kept"], ref["under"])
        else:
            raise AssertionError((r, k, ref["kept"]))
    return n_same, st


@pytest.mark.parametrize("name,T,tp", [("tiny", 0.6, 0.9), ("llama2-7b", 0.6, 0.8), ("llama2-7b", 1.0, 0.9),
                                       ("llama2-7b", 1.0, 0.99), ("llama2-13b", 1.0, 0.9)])
def test_top_p_on_config_logits(name, T, tp):
    cfg = W.CONFIGS[name]
    vi = W.make_verify_inputs(cfg, T, 0)
    rows = vi.target_logits.numpy()[: min(cfg.n_tree, 48)]
    n_ok, st = _check(rows, T, tp)
    assert st == 0 and n_ok >= rows.shape[0] // 2


def test_top_p_large_vocabulary_and_flat_rows():
    rng = np.random.default_rng(0)
    # 128256 tokens, and a flat-ish distribution (sigma 0.5) whose nucleus holds tens of thousands of tokens
    rows = np.concatenate([(3.0 * rng.standard_normal((3, 128256))), (0.5 * rng.standard_normal((3, 128256)))]).astype(np.float32)
    n_ok, st = _check(rows, 0.6, 0.9)
    assert st == 0 and n_ok >= 5
    _, kept, _ = _run(rows, 0.6, 0.9)
    assert kept[:3].max() < 2000 and kept[3:].min() > 20000


@pytest.mark.parametrize("V", [1, 2, 3, 7, 33, 1023, 1024, 1025, 4099, 5003])
def test_top_p_ragged_vocabularies_strides_and_in_place(V):
    rng = np.random.default_rng(V)
    rows = (2.0 * rng.standard_normal((5, V))).astype(np.float32)
    for tp in (0.3, 0.9):
        n_ok, st = _check(rows, 0.8, tp, pad=8)
        assert st == 0 and n_ok >= 4
        n_ok, st = _check(rows, 0.8, tp, in_place=True)
        assert st == 0 and n_ok >= 4


def test_top_p_equal_logits_at_the_cut_go_in_token_order():
    # all equal: the first ceil(top_p V) tokens
    for V, tp in ((10, 0.35), (10, 0.31), (1000, 0.9005), (4099, 0.5)):  # (off the exact multiples of 1/V)
        got, kept, st = _run(np.zeros((2, V), np.float32), 1.0, tp)
        ref = O.top_p(np.zeros(V, np.float32), 1.0, tp)
        assert st == 0 and kept.tolist() == [ref["kept"]] * 2
        assert np.array_equal(np.isfinite(got[0]), ref["keep"]) and np.array_equal(got[0], got[1])
    # a run of equal logits straddling the cut inside an otherwise random row
    rng = np.random.default_rng(1)
    V = 3000
    x = (rng.standard_normal(V)).astype(np.float32)
    top = np.argsort(-x)
    x[top[:3]] = 6.0                      # three clear leaders
    dup = rng.choice(top[3:], 40, replace=False)
    x[dup] = 2.5                          # then forty equal ones, more than the rest of the nucleus needs
    prob = O.softmax_T(x, 1.0)
    tp = float(prob[x > 2.5].sum() + 0.49 * prob[dup].sum())  # 19.6 of the 40 equal tokens are needed: 20
    ref = O.top_p(x, 1.0, tp)
    inside = ref["keep"][dup]
    assert 0 < inside.sum() < 40          # the cut really falls inside the run
    got, kept, st = _run(x[None], 1.0, tp)
    assert st == 0 and kept[0] == ref["kept"]
    assert np.array_equal(np.isfinite(got[0]), ref["keep"])
    kept_dup = np.sort(dup[np.isfinite(got[0][dup])])
    assert np.array_equal(kept_dup, np.sort(dup)[: inside.sum()])   # the lowest token ids of the run


def test_top_p_one_keeps_everything_and_tiny_keeps_the_argmax():
    rng = np.random.default_rng(2)
    rows = (3 * rng.standard_normal((4, 777))).astype(np.float32)
    got, kept, st = _run(rows, 0.7, 1.0)
    assert st == 0 and np.array_equal(got, rows) and kept.tolist() == [777] * 4
    got, kept, st = _run(rows, 0.7, 1e-6)
    assert st == 0 and kept.tolist() == [1] * 4
    assert np.array_equal(np.argmax(rows, axis=1), np.argmax(got, axis=1)) and np.isfinite(got).sum() == 4


def test_top_p_nonfinite_and_empty_rows_are_flagged():
    rng = np.random.default_rng(3)
    rows = (2 * rng.standard_normal((3, 500))).astype(np.float32)
    rows[0, 7], rows[0, 9], rows[0, 11] = np.nan, np.inf, -np.inf
    got, kept, st = _run(rows, 1.0, 0.95)
    ref = O.top_p(rows[0], 1.0, 0.95)
    assert st == B.SEQ_DEV_NONFINITE and ref["flags"] == O.NONFINITE
    assert np.array_equal(np.isfinite(got[0]), ref["keep"]) and np.isneginf(got[0, [7, 9, 11]]).all()
    rows[:] = -np.inf
    got, kept, st = _run(rows, 1.0, 0.9)
    assert st == B.SEQ_DEV_DEGENERATE and kept.tolist() == [0, 0, 0] and np.isneginf(got).all()


def test_top_p_is_repeatable_bit_for_bit():
    rng = np.random.default_rng(4)
    rows = (0.7 * rng.standard_normal((16, 32000))).astype(np.float32)
    first, k1, _ = _run(rows, 1.0, 0.9)
    for _ in range(3):
        again, k2, _ = _run(rows, 1.0, 0.9)
        assert np.array_equal(first.view(np.uint32), again.view(np.uint32)) and np.array_equal(k1, k2)


@pytest.mark.parametrize("tp", [0.8, 0.9])
def test_filter_then_verify_matches_the_oracle_chain(tp):
    """Target rows truncated on the GPU, then Algorithm 2 on the GPU, against the oracle's Algorithm 2 on the oracle's
    truncated rows: the output law is the truncated target distribution."""
    cfg = W.CONFIGS["llama2-7b"]
    checked = 0
    for seed in range(3):
        vi = W.make_verify_inputs(cfg, 0.6, seed)
        refs = [O.top_p(vi.target_logits[v].numpy(), 0.6, tp) for v in range(cfg.n_tree)]
        if min(r["min_gap"] for r in refs) < BAND:
            continue
        d = G.dev()
        filt = B.seq_tree_top_p_filter(vi.target_logits.to(d), 0.6, tp)
        torch.cuda.synchronize()
        want = np.stack([r["filtered"] for r in refs])
        assert np.array_equal(filt.cpu().numpy().view(np.uint32), want.view(np.uint32))
        vi2 = W.VerifyInputs(vi.parent, vi.tokens, filt.cpu(), vi.draft_logits, vi.uniforms, vi.temperature)
        checked += G.check_verify(vi2) == "ok"
    assert checked >= 1


def test_top_p_cut_with_a_clear_margin_is_the_oracles_on_every_row():
    """Rows whose probabilities fall off geometrically (each token 0.6 of the one before, in a shuffled order): the
    cumulative mass passes top_p with a margin of percents, far outside the rounding band, so every row's kept set must
    be exactly the oracle's — an off-by-one at the cut could not hide here."""
    rng = np.random.default_rng(5)
    rows, V, T = 48, 5000, 0.7
    logits = np.full((rows, V), -60.0, np.float32)
    for r in range(rows):
        perm = rng.permutation(V)[:40]
        logits[r, perm] = (T * np.log(0.6) * np.arange(40)).astype(np.float32) + np.float32(rng.normal())
    for tp in (0.5, 0.8, 0.95, 0.999):
        same, st = _check(logits, T, tp)
        assert st == 0 and same == rows, (tp, same)
