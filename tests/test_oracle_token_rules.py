"""Pins for the oracle's two token-level comparison rules (Top-P count, skipping relative to the top-1 score):
hand-worked fixtures, closed forms, the defining inequalities, a library cross-check on exactly representable
values, monotonicity -- and the host-side threshold calibration run on the oracle."""
import os

import numpy as np
import pytest

from oracle import alloc_moe_oracle as orc
from paper_2604_08133_b200 import synth
from paper_2604_08133_b200 import token_baselines as TB

HERE = os.path.dirname(os.path.abspath(__file__))


def _golden():
    out = []
    with open(os.path.join(HERE, "golden", "token_rule_worked_examples.txt")) as f:
        for ln in f:
            if ln.startswith("#") or not ln.strip():
                continue
            rule, row, thr, n = [c.strip() for c in ln.split("|")]
            out.append((rule, np.array([[float(v) for v in row.split()]], np.float32), float(thr), int(n)))
    return out


@pytest.mark.parametrize("rule,row,thr,n", _golden())
def test_worked_examples(rule, row, thr, n):
    got = orc.top_p_count(row, thr) if rule == "top_p" else orc.rel_threshold_count(row, thr)
    assert got.tolist() == [n]


def _dyadic_rows(T, K, key):
    """Descending rows whose entries are multiples of 2^-12 below 1/K: every partial sum is exact in fp32."""
    idx = np.array(synth.permutation(T * K * 7, key)[:T * K], np.int64).reshape(T, K)
    v = ((idx % 400) + 1).astype(np.float32) / np.float32(4096.0)
    return -np.sort(-v, axis=1)


def test_top_p_uniform_rows_closed_form():
    s = np.full((1, 8), 0.125, np.float32)
    for P, want in [(0.125, 1), (0.126, 2), (0.5, 4), (0.51, 5), (1.0, 8), (1.1, 8), (-1.0, 1)]:
        assert orc.top_p_count(s, P).tolist() == [want]


def test_top_p_defining_inequalities_and_library_crosscheck():
    s = _dyadic_rows(200, 6, 11)
    for P in (0.01, 0.05, 0.1, 0.2, 0.33, 0.5):
        n = orc.top_p_count(s, P)
        cum = np.cumsum(s.astype(np.float64), axis=1)          # exact for these values, in any order
        thr = float(np.float32(P))
        for t in range(s.shape[0]):
            k = n[t]
            assert 1 <= k <= 6
            if k > 1:
                assert cum[t, k - 2] < thr                      # one expert fewer would not have reached P
            assert cum[t, k - 1] >= thr or k == 6               # reached, or the row ran out
        lib = np.minimum(np.array([np.searchsorted(cum[t], thr, side="left") for t in range(s.shape[0])]) + 1, 6)
        assert np.array_equal(n, lib)


def test_top_p_is_monotone_in_P():
    s = synth.score_rows(300, 6, 5).numpy()
    prev = orc.top_p_count(s, 0.0)
    assert (prev == 1).all()
    for P in np.linspace(0.05, 3.0, 30):
        cur = orc.top_p_count(s, float(P))
        assert (cur >= prev).all()
        prev = cur
    assert (orc.top_p_count(s, 1e9) == 6).all()


def test_rel_threshold_limits_ties_and_library_crosscheck():
    s = _dyadic_rows(200, 6, 12)
    assert (orc.rel_threshold_count(s, 0.0) == 6).all()
    ties = (s == s[:, :1]).sum(axis=1)
    assert np.array_equal(orc.rel_threshold_count(s, 1.0), ties)         # only scores equal to the top-1 survive beta = 1
    assert (orc.rel_threshold_count(s, 1.0009765625) == 1).all()
    for beta in (0.5, 0.25, 0.125, 0.75):                                # dyadic: the product is exact
        want = (s >= np.float32(beta) * s[:, :1]).sum(axis=1)            # rows are sorted, so the count is the prefix
        assert np.array_equal(orc.rel_threshold_count(s, beta), want)
    prev = orc.rel_threshold_count(s, 0.0)
    for beta in np.linspace(0.0, 1.2, 25):
        cur = orc.rel_threshold_count(s, float(beta))
        assert (cur <= prev).all()
        prev = cur


def _oracle_top_p(scores, thr):
    n = orc.top_p_count(scores, thr)
    return n, int(n.sum())


def _oracle_rel(scores, thr):
    n = orc.rel_threshold_count(scores, thr)
    return n, int(n.sum())


def test_threshold_calibration_meets_the_budget_without_exceeding_it():
    s = synth.score_rows(500, 6, 21).numpy()
    s = s / s.sum(axis=1, keepdims=True).astype(np.float32)
    for budget in (500, 1000, 1500, 2400, 3000):
        P, tot = TB.calibrate(_oracle_top_p, s, budget, increasing=True, lo=0.0, hi=2.0)
        assert tot <= budget and tot == int(orc.top_p_count(s, P).sum())
        # the next representable step up would overshoot (or everything is already kept)
        assert tot == 3000 or int(orc.top_p_count(s, np.nextafter(np.float32(P), np.float32(4.0))).sum()) > budget
        beta, tot = TB.calibrate(_oracle_rel, s, budget, increasing=False, lo=0.0, hi=1.5)
        assert tot <= budget and tot == int(orc.rel_threshold_count(s, beta).sum())
