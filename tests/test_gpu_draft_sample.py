"""GPU parity of seq_tree_draft_sample (exponential sort) against the oracle: the drawn tokens, in order,
for every row whose keys are further apart than fp32 resolves; edge cases."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2402_12374_b200 import binding as B, workloads as W

pytestmark = pytest.mark.gpu

GAP = 1e-4  # relative distance between neighbouring keys below which fp32 may order them differently


def _dev():
    return torch.device("cuda:0")


def _check_rows(logits, u, T, k):
    d = _dev()
    st = torch.zeros(1, dtype=torch.int32, device=d)
    got = B.seq_tree_draft_sample(torch.from_numpy(logits).to(d), T, torch.from_numpy(u).to(d), k, dev_status=st)
    torch.cuda.synchronize()
    got = got.cpu().numpy()
    n_ok = n_excl = 0
    for r in range(logits.shape[0]):
        ref = O.draft_sample(logits[r], T, u[r], k)
        if ref["min_rel_gap"] < GAP:
            # two keys too close for fp32: the same set is still required up to the close pair, so only count it
            n_excl += 1
            continue
        assert got[r].tolist() == ref["tokens"].tolist(), (r, got[r], ref["tokens"])
        n_ok += 1
    return n_ok, n_excl, int(st.item())


@pytest.mark.parametrize("name,rows,k", [("tiny", 16, 4), ("llama2-7b", 24, 8), ("llama3-70b", 6, 16)])
def test_draft_sample_config_shapes(name, rows, k):
    """Vocabulary sizes and draft-logit statistics of the workloads (32000: scores in shared memory;
    128256: recomputed), uniforms from the seeded generator."""
    cfg = W.CONFIGS[name]
    vi = W.make_verify_inputs(cfg, 0.6, 5)
    logits = vi.draft_logits.numpy()[:rows].copy()
    rng = np.random.default_rng(17)
    u = rng.random(logits.shape).astype(np.float32)
    ok, excl, st = _check_rows(logits, u, 0.6, k)
    assert st == 0 and ok >= rows - 2, (ok, excl)


@pytest.mark.parametrize("V", [1, 2, 3, 5, 31, 257, 1000, 4099, 50257])
def test_draft_sample_ragged_vocab_and_unaligned_rows(V):
    rng = np.random.default_rng(V)
    rows, k = 5, min(7, 64)
    logits = (2 * rng.standard_normal((rows, V))).astype(np.float32)
    u = rng.random((rows, V)).astype(np.float32)
    ok, excl, st = _check_rows(logits, u, 0.9, k)   # rows of V floats: 16-byte aligned only if V % 4 == 0
    assert st == 0 and ok + excl == rows and ok >= rows - 1


def test_draft_sample_support_smaller_than_k_and_bad_values():
    d = _dev()
    rng = np.random.default_rng(9)
    V, k = 200, 12
    logits = np.full((3, V), -np.inf, np.float32)
    keep = rng.choice(V, 5, replace=False)
    logits[0, keep] = rng.standard_normal(5)
    logits[1] = rng.standard_normal(V)
    logits[2] = rng.standard_normal(V)
    u = rng.random((3, V)).astype(np.float32)
    u[1, :10] = 0.0      # no chance
    u[1, 10:20] = 1.0    # no chance
    logits[2, 7] = np.nan
    logits[2, 8] = np.inf
    st = torch.zeros(1, dtype=torch.int32, device=d)
    got = B.seq_tree_draft_sample(torch.from_numpy(logits).to(d), 1.0, torch.from_numpy(u).to(d), k, dev_status=st).cpu().numpy()
    assert sorted(got[0][:5].tolist()) == sorted(keep.tolist()) and (got[0][5:] == -1).all()
    assert got[0].tolist() == O.draft_sample(logits[0], 1.0, u[0], k)["tokens"].tolist()
    assert got[1].tolist() == O.draft_sample(logits[1], 1.0, u[1], k)["tokens"].tolist()
    assert not set(got[1].tolist()) & set(range(20))
    assert int(st.item()) == B.SEQ_DEV_NONFINITE and 7 not in got[2] and 8 not in got[2]
    clean = logits[2].copy()
    clean[[7, 8]] = -np.inf   # flagged entries are never drawn: same draws as with probability 0
    assert got[2].tolist() == O.draft_sample(clean, 1.0, u[2], k)["tokens"].tolist()


def test_draft_sample_strided_rows_and_argument_checks():
    d = _dev()
    rng = np.random.default_rng(4)
    V, rows, k = 1000, 4, 6
    big_l = torch.from_numpy(rng.standard_normal((rows, V + 24)).astype(np.float32)).to(d)
    big_u = torch.from_numpy(rng.random((rows, V + 8)).astype(np.float32)).to(d)
    got = B.seq_tree_draft_sample(big_l[:, :V], 0.8, big_u[:, :V], k).cpu().numpy()
    for r in range(rows):
        ref = O.draft_sample(big_l[r, :V].cpu().numpy(), 0.8, big_u[r, :V].cpu().numpy(), k)
        if ref["min_rel_gap"] >= GAP:
            assert got[r].tolist() == ref["tokens"].tolist()
    for bad in (dict(k=0), dict(k=65), dict(T=0.0), dict(T=float("inf"))):
        with pytest.raises(B.SeqTreeError) as e:
            B.seq_tree_draft_sample(big_l[:, :V], bad.get("T", 0.8), big_u[:, :V], bad.get("k", k))
        assert e.value.code == B.SEQ_ERR_INVALID_ARG


def test_draft_sample_first_draw_frequencies_follow_the_softmax():
    """A property that holds at any size: over many rows with independent uniforms the first draw is a sample
    of the row's softmax (same logits in every row)."""
    d = _dev()
    rng = np.random.default_rng(21)
    V, rows = 50, 20000
    base = (1.5 * rng.standard_normal(V)).astype(np.float32)
    logits = torch.from_numpy(np.tile(base, (rows, 1))).to(d)
    u = torch.from_numpy(rng.random((rows, V)).astype(np.float32)).to(d)
    first = B.seq_tree_draft_sample(logits, 0.7, u, 2)[:, 0].cpu().numpy()
    q = O.softmax_T(base, 0.7)
    cnt = np.bincount(first, minlength=V)
    assert (np.abs(cnt - rows * q) <= 5 * np.sqrt(rows * q * (1 - q)) + 1).all()
