"""alloc_l_solve (the library's host-side Alloc-L solver, Sec. 3.2) against the oracle's dynamic programme, brute
force over all K_orig^L allocations, and the properties Eq. 3-5 fix.  No GPU needed."""
import numpy as np
import pytest

from oracle import alloc_moe_oracle as orc
from paper_2604_08133_b200 import binding as B


def _profile(rng, L, K, noise=0.05):
    # decreasing-in-k costs like a perplexity profile, plus noise so the rows are not convex
    return np.sort(rng.random((L, K)), axis=1)[:, ::-1] + noise * rng.random((L, K))


@pytest.mark.parametrize("L,K", [(1, 1), (1, 6), (3, 4), (5, 3), (6, 3), (4, 6)])
def test_equals_bruteforce_and_oracle_dp(L, K):
    rng = np.random.default_rng(100 * L + K)
    for _ in range(3):
        S = _profile(rng, L, K)
        for budget in range(L, L * K + 3):
            ks, cost = B.alloc_l_solve(S, budget)
            assert len(ks) == L and all(1 <= k <= K for k in ks) and sum(ks) <= budget       # Eq. 4, 5
            assert abs(cost - sum(S[i, ks[i] - 1] for i in range(L))) < 1e-12                   # Eq. 3
            assert abs(cost - orc.alloc_l_bruteforce(S, budget)) < 1e-12
            oks, ocost = orc.alloc_l_dp(S, budget)
            assert ks == oks and abs(cost - ocost) < 1e-12                                      # same tie rule


def test_degenerate_budgets():
    rng = np.random.default_rng(7)
    S = _profile(rng, 26, 6, noise=0.0)                 # strictly decreasing rows
    ks, _ = B.alloc_l_solve(S, 26)
    assert ks == [1] * 26                               # one expert per layer is all the budget allows
    ks, cost = B.alloc_l_solve(S, 26 * 6)
    assert ks == [6] * 26                               # enough for every layer's best setting
    ks2, cost2 = B.alloc_l_solve(S, 10 ** 6)            # more budget than can be used changes nothing
    assert ks2 == ks and cost2 == cost


def test_more_budget_never_costs_more_and_stack_sized_problem():
    rng = np.random.default_rng(3)
    S = _profile(rng, 26, 6)                            # the DeepSeek-V2-Lite-shaped stack: 26 layers, K_orig 6
    prev = np.inf
    for budget in range(26, 26 * 6 + 1):
        ks, cost = B.alloc_l_solve(S, budget)
        assert cost <= prev + 1e-15
        prev = cost
        oks, ocost = orc.alloc_l_dp(S, budget)
        assert ks == oks and abs(cost - ocost) < 1e-12


def test_ties_take_the_smaller_k():
    S = np.array([[1.0, 1.0, 1.0], [2.0, 1.0, 1.0]])
    assert B.alloc_l_solve(S, 6)[0] == [1, 2]


def test_errors():
    S = np.ones((4, 3))
    with pytest.raises(B.MoeError) as ei:
        B.alloc_l_solve(S, 3)                           # below one expert per layer
    assert ei.value.status == B.MOE_ERR_BUDGET
    with pytest.raises(B.MoeError) as ei:
        B.alloc_l_solve(np.full((2, 2), np.inf), 4)
    assert ei.value.status == B.MOE_ERR_NONFINITE


def test_stack_budgets_from_the_synthetic_sensitivity_matrix():
    """What `bench.py --stack-budgets alloc-l` runs: a decreasing, seeded S for the 26-layer stack, solved at the
    same total (78) as the Dirichlet split; earlier layers are the more sensitive ones and get more on average."""
    from paper_2604_08133_b200 import synth
    cfg = synth.CONFIGS["c4"]
    S = np.array(synth.sensitivity_matrix(cfg))
    assert S.shape == (26, 6) and np.array_equal(S, np.array(synth.sensitivity_matrix(cfg)))
    assert (np.diff(S, axis=1) <= 0).all() and (S[:, -1] == 0).all() and (S[:, 0] > 0).all()
    ks, cost = B.alloc_l_solve(S, 78)
    assert sum(ks) == 78 and all(1 <= k <= 6 for k in ks)
    assert ks == orc.alloc_l_dp(S, 78)[0]
    assert sum(ks[:13]) > sum(ks[13:])

