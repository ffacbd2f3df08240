"""Pins of the oracle's nucleus truncation (``orc_top_p``): the three properties that characterise the kept set,
a library implementation (torch.sort + cumsum), closed forms (uniform, geometric), limits and invariances."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as O


def test_kept_set_is_characterised_by_three_properties():
    """(1) its mass reaches top_p; (2) without its least probable member it does not; (3) nothing outside is more
    probable than anything inside.  Together they fix the set (up to equal probabilities)."""
    rng = np.random.default_rng(0)
    for trial in range(40):
        V = int(rng.integers(2, 400))
        T = float(rng.choice([0.3, 0.6, 1.0, 1.7]))
        tp = float(rng.choice([0.05, 0.5, 0.8, 0.9, 0.99]))
        logits = (rng.standard_normal(V) * rng.choice([0.5, 3.0])).astype(np.float32)
        r = O.top_p(logits, T, tp)
        p = O.softmax_T(logits, T)
        inside, outside = p[r["keep"]], p[~r["keep"]]
        assert r["kept"] == inside.size >= 1
        assert inside.sum() >= tp - 1e-15
        assert inside.sum() - inside.min() < tp
        assert outside.size == 0 or outside.max() <= inside.min()
        assert np.array_equal(r["filtered"][r["keep"]], logits[r["keep"]]) and np.all(np.isneginf(r["filtered"][~r["keep"]]))


def test_against_a_library_sort_and_cumsum():
    g = torch.Generator().manual_seed(1)
    for V, T, tp in ((1000, 0.6, 0.9), (32000, 1.0, 0.8), (5003, 0.3, 0.95), (64, 1.0, 0.5)):
        logits = 3.0 * torch.randn(V, generator=g)
        r = O.top_p(logits, T, tp)
        if r["min_gap"] < 1e-9:
            continue
        p = torch.softmax(logits.double() / T, dim=0)
        sp, idx = torch.sort(p, descending=True, stable=True)
        cum = torch.cumsum(sp, dim=0)
        k = int(torch.searchsorted(cum, torch.tensor(tp, dtype=torch.float64)).item()) + 1  # first position reaching top_p
        keep = torch.zeros(V, dtype=torch.bool)
        keep[idx[:k]] = True
        assert np.array_equal(keep.numpy(), r["keep"])


def test_closed_forms_uniform_and_geometric():
    # equal logits: the first ceil(top_p * V) tokens (equal probabilities go in token order)
    for V, tp in ((10, 0.35), (10, 0.3), (7, 0.5), (1000, 0.9)):
        r = O.top_p(np.zeros(V, np.float32), 1.0, tp)
        k = math.ceil(tp * V - 1e-12)
        assert r["keep"].tolist() == [True] * k + [False] * (V - k)
    # p_i proportional to r^i (logits = i * ln r): kept = the smallest k with 1 - r^k >= top_p (1 - r^V)
    V, ratio = 60, 0.8
    logits = (np.arange(V) * math.log(ratio)).astype(np.float64)
    for tp in (0.2, 0.5, 0.9, 0.999):
        res = O.top_p(logits.astype(np.float32), 1.0, tp)
        k = next(k for k in range(1, V + 1) if 1 - ratio ** k >= tp * (1 - ratio ** V) - 1e-9)
        assert res["kept"] == k and res["keep"][:k].all() and not res["keep"][k:].any()
    # temperature: a geometric ratio r at T = 1 is r^(1/T) at T
    res = O.top_p(logits.astype(np.float32), 0.5, 0.9)
    r2 = ratio ** 2
    k = next(k for k in range(1, V + 1) if 1 - r2 ** k >= 0.9 * (1 - r2 ** V) - 1e-9)
    assert res["kept"] == k


def test_limits_and_invariances():
    rng = np.random.default_rng(2)
    logits = (2 * rng.standard_normal(300)).astype(np.float32)
    assert O.top_p(logits, 1.0, 1.0)["kept"] == 300 and O.top_p(logits, 1.0, 1.5)["kept"] == 300
    tiny = O.top_p(logits, 1.0, 1e-9)
    assert tiny["kept"] == 1 and tiny["keep"][int(np.argmax(logits))]
    a = O.top_p(logits, 0.7, 0.85)
    b = O.top_p(logits * 2, 1.4, 0.85)          # only logits / T matters
    assert np.array_equal(a["keep"], b["keep"])
    perm = rng.permutation(300)
    c = O.top_p(logits[perm], 0.7, 0.85)      # relabelling tokens relabels the set (no equal logits here)
    assert np.array_equal(c["keep"], a["keep"][perm])
    # growing top_p only adds tokens
    prev = np.zeros(300, bool)
    for tp in (0.1, 0.3, 0.6, 0.9, 0.99):
        k = O.top_p(logits, 1.0, tp)["keep"]
        assert not (prev & ~k).any()
        prev = k
    # -inf logits are never kept; a NaN or +inf logit is flagged and never kept
    x = logits.copy()
    x[5], x[9] = -np.inf, np.nan
    r = O.top_p(x, 1.0, 0.999999)
    assert not r["keep"][5] and not r["keep"][9] and r["flags"] == O.NONFINITE


def test_min_gap_reports_the_margin():
    # p = [.5, .3, .2]: top_p = .79 keeps two, 0.01 below their mass and 0.29 above the first alone
    logits = np.log(np.array([0.5, 0.3, 0.2])).astype(np.float32)
    r = O.top_p(logits, 1.0, 0.79)
    assert r["keep"].tolist() == [True, True, False] and r["min_gap"] == pytest.approx(0.01, abs=1e-6)
    r = O.top_p(logits, 1.0, 0.51)
    assert r["keep"].tolist() == [True, True, False] and r["min_gap"] == pytest.approx(0.01, abs=1e-6)
    assert r["over"] == pytest.approx(0.29, abs=1e-6) and r["under"] == pytest.approx(0.01, abs=1e-6)
    r = O.top_p(logits, 1.0, 0.4)
    assert r["keep"].tolist() == [True, False, False] and r["min_gap"] == pytest.approx(0.1, abs=1e-6)
    assert r["over"] == pytest.approx(0.1, abs=1e-6) and r["under"] == pytest.approx(0.4, abs=1e-6)
