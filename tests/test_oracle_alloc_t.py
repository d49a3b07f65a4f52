"""Pins for the oracle's Alloc-T (Sec. 3.3): the 0/1 programme by brute force, the
invariants the paper fixes, its degenerate cases, hand-worked examples."""
import itertools
import os

import numpy as np
import pytest

from oracle import alloc_moe_oracle as orc
from paper_2604_08133_b200 import synth

HERE = os.path.dirname(os.path.abspath(__file__))


def _rows(T, K, key, ties=False):
    return synth.score_rows(T, K, synth.stream_key(99, key), ties=ties).numpy()


def _golden_cases():
    cases, scores = [], None
    with open(os.path.join(HERE, "golden", "alloc_t_worked_examples.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line or line.startswith("case"):
                continue
            if line.startswith("scores:"):
                scores = np.array([[float(v) for v in r.split()] for r in line[7:].split(";")], np.float32)
            else:
                lhs, rhs = line.split("->")
                kb, b = (int(v) for v in lhs.split())
                cases.append((scores, kb, b, [int(v) for v in rhs.split()]))
    return cases


@pytest.mark.parametrize("scores,K_base,budget,want", _golden_cases())
def test_hand_worked_examples(scores, K_base, budget, want):
    for fn in (orc.alloc_t_select, orc.alloc_t_select_threshold):
        z = fn(scores, K_base, budget)
        assert orc.n_sel_from_mask(z).tolist() == want


@pytest.mark.parametrize("T,K", [(2, 2), (3, 3), (4, 3), (2, 4), (4, 4), (5, 3)])
def test_procedure_is_the_unique_ilp_optimum(T, K):
    """Eq. 8-10 enumerated: with distinct scores the arg-max is unique and is the procedure's z."""
    for trial in range(3):
        s = _rows(T, K, 1000 * T + 10 * K + trial)
        assert len(np.unique(s)) == s.size
        for K_base in range(0, K + 1):
            for budget in range(K_base * T, K * T + 1):
                best, arg = orc.alloc_t_bruteforce(s, K_base, budget)
                z = orc.alloc_t_select(s, K_base, budget)
                assert len(arg) == 1
                assert np.array_equal(arg[0], z), (K_base, budget)
                assert abs(orc.alloc_t_objective(s, z) - best) < 1e-12
                assert np.array_equal(z, orc.alloc_t_select_threshold(s, K_base, budget))


def test_with_ties_objective_is_optimal_and_selection_is_one_of_the_optima():
    for trial in range(4):
        s = _rows(4, 3, 50 + trial, ties=True)
        for K_base in range(0, 3):
            for budget in range(K_base * 4, 13):
                best, arg = orc.alloc_t_bruteforce(s, K_base, budget)
                for fn in (orc.alloc_t_select, orc.alloc_t_select_threshold):
                    z = fn(s, K_base, budget)
                    assert abs(orc.alloc_t_objective(s, z) - best) < 1e-12
                    assert any(np.array_equal(z, a) for a in arg)
                    orc.n_sel_from_mask(z)          # prefix property holds under ties


@pytest.mark.parametrize("ties", [False, True])
def test_invariants_and_two_forms_at_workload_sizes(ties):
    T, K = 512, 6
    s = _rows(T, K, 7, ties)
    for K_base in (0, 1, 2):
        for budget in (K_base * T, K_base * T + 1, 2 * T, 3 * T, int(4.5 * T), K * T - 1, K * T):
            if budget < K_base * T:
                continue
            z = orc.alloc_t_select(s, K_base, budget)
            assert np.array_equal(z, orc.alloc_t_select_threshold(s, K_base, budget))
            n = orc.n_sel_from_mask(z)
            assert int(n.sum()) == budget                       # total activations = layer budget
            assert n.min() >= K_base and n.max() <= K           # per-token bounds (Eq. 10, candidate set)
            resid = s[:, K_base:]
            zk = z[:, K_base:].astype(bool)
            if zk.any() and (~zk).any():
                assert resid[zk].min() >= resid[~zk].max()      # every kept residual >= every dropped one


def test_degenerate_cases():
    T, K = 64, 6
    s = _rows(T, K, 3)
    for kb in range(K + 1):
        n = orc.n_sel_from_mask(orc.alloc_t_select(s, kb, kb * T))   # K_base = K_l: plain Top-K
        assert (n == kb).all()
    n = orc.n_sel_from_mask(orc.alloc_t_select(s, 1, K * T))         # full budget: plain Top-K_orig
    assert (n == K).all()


def test_nesting_in_the_budget():
    T, K = 32, 4
    s = _rows(T, K, 11, ties=True)
    prev = orc.alloc_t_select(s, 1, T)
    for budget in range(T + 1, K * T + 1):
        z = orc.alloc_t_select(s, 1, budget)
        assert ((z - prev) >= 0).all() and int((z - prev).sum()) == 1
        prev = z


def test_objective_beats_uniform_topk():
    T, K = 256, 6
    s = _rows(T, K, 21)
    for k_l in range(1, K + 1):
        uniform = float(s[:, :k_l].astype(np.float64).sum())
        for kb in range(0, k_l + 1):
            z = orc.alloc_t_select(s, kb, k_l * T)
            assert orc.alloc_t_objective(s, z) >= uniform - 1e-12


def test_budget_is_shifted_to_flat_rows():
    """Sec. 3.3: computation moves toward tokens with less concentrated routing."""
    s = np.array([[0.90, 0.05, 0.03], [0.40, 0.35, 0.20]], np.float32)
    assert orc.n_sel_from_mask(orc.alloc_t_select(s, 1, 4)).tolist() == [1, 3]


def test_rejects_infeasible_budgets():
    s = _rows(4, 3, 1)
    for kb, b in [(1, 3), (1, 13), (4, 12), (-1, 4)]:
        with pytest.raises(ValueError):
            orc.alloc_t_select(s, kb, b)
        with pytest.raises(ValueError):
            orc.alloc_t_select_threshold(s, kb, b)


def test_prefix_check_detects_a_non_prefix_mask():
    z = np.array([[1, 0, 1]], np.int8)
    with pytest.raises(AssertionError):
        orc.n_sel_from_mask(z)
