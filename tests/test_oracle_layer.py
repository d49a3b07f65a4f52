"""Pins for the oracle's permutation, expert math, Eq. 2 combine, stack and Alloc-L DP."""
import numpy as np
import pytest
import torch

from oracle import alloc_moe_oracle as orc
from paper_2604_08133_b200 import synth


def _np_layer(cfg):
    d = synth.make_layer(cfg)
    return {k: (None if v is None else v.float().numpy()) for k, v in d.items()}


SMALL = synth.CONFIGS["c2"].with_(T=24, H=64, N=8, I=32, S=2, K_orig=3, K_base=1, budget=40)


def test_expert_ffn_against_torch_fp64():
    d = _np_layer(SMALL)
    x = torch.from_numpy(d["x"]).double()
    W13 = torch.from_numpy(d["W13"][3]).double()
    W2 = torch.from_numpy(d["W2"][3]).double()
    I = SMALL.I
    want = (torch.nn.functional.silu(x @ W13[:I].T) * (x @ W13[I:].T)) @ W2.T
    got = orc.expert_ffn(d["x"], d["W13"][3], d["W2"][3])
    assert np.allclose(got, want.numpy(), rtol=1e-12, atol=1e-15)
    # gate and up halves are not interchangeable
    swapped = np.concatenate([d["W13"][3][I:], d["W13"][3][:I]])
    assert not np.allclose(orc.expert_ffn(d["x"], swapped, d["W2"][3]), got, rtol=1e-3)


def test_silu_closed_forms():
    assert orc.silu(np.array([0.0]))[0] == 0.0
    a = np.array([-3.0, 0.5, 4.0])
    assert np.allclose(orc.silu(a) - orc.silu(-a), a)          # silu(a) - silu(-a) = a
    assert abs(orc.silu(np.array([1.0]))[0] - 1 / (1 + np.e ** -1)) < 1e-15


def test_permute_invariants():
    d = _np_layer(SMALL)
    r = orc.route(d["x"], d["W_gate"], d["gate_bias"], SMALL.K_orig, SMALL.K_base, SMALL.budget)
    p = orc.permute(r["topk_idx"], r["topk_score"], r["n_sel"], SMALL.N)
    off, tok, w, pos = p["expert_offsets"], p["perm_token"], p["perm_weight"], p["pair_pos"]
    assert off[0] == 0 and off[-1] == SMALL.budget and (np.diff(off) >= 0).all()
    kept_e = [r["topk_idx"][t, j] for t in range(SMALL.T) for j in range(r["n_sel"][t])]
    assert np.array_equal(np.diff(off), np.bincount(kept_e, minlength=SMALL.N))
    for e in range(SMALL.N):
        seg = tok[off[e]:off[e + 1]]
        assert (np.diff(seg) > 0).all()                          # token-ascending, no duplicates
    kept_pos = sorted(pos[pos >= 0].tolist())
    assert kept_pos == list(range(SMALL.budget))                  # bijection kept pairs <-> [0,B)
    for t in range(SMALL.T):
        for j in range(SMALL.K_orig):
            if j < r["n_sel"][t]:
                q = pos[t, j]
                assert tok[q] == t and w[q] == r["topk_score"][t, j]
                assert off[r["topk_idx"][t, j]] <= q < off[r["topk_idx"][t, j] + 1]
            else:
                assert pos[t, j] == -1


def test_permute_hand_case():
    idx = np.array([[2, 0], [0, 1], [2, 1]], np.int32)
    sc = np.array([[.6, .3], [.5, .4], [.7, .2]], np.float32)
    p = orc.permute(idx, sc, np.array([2, 1, 2]), 3)
    # kept: (t0,e2) (t0,e0) (t1,e0) (t2,e2) (t2,e1) -> e0:[t0,t1] e1:[t2] e2:[t0,t2]
    assert p["expert_offsets"].tolist() == [0, 2, 3, 5]
    assert p["perm_token"].tolist() == [0, 1, 2, 0, 2]
    assert np.allclose(p["perm_weight"], [.3, .5, .2, .6, .7])
    assert p["pair_pos"].tolist() == [[3, 0], [1, -1], [4, 2]]


def test_sparse_form_equals_literal_eq2():
    d = _np_layer(SMALL)
    a = (d["x"], d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"], d["Wsh2"],
         SMALL.K_orig, SMALL.K_base, SMALL.budget)
    sparse = orc.layer_forward(*a)["out"]
    dense = orc.layer_forward_dense(*a)
    assert np.allclose(sparse, dense, rtol=1e-11, atol=1e-14)
    rows = [3, 17, 5]
    assert np.allclose(orc.layer_forward(*a, rows=rows)["out"], dense[rows], rtol=1e-11, atol=1e-14)


def test_identical_experts_collapse_to_sum_of_kept_scores():
    cfg = SMALL.with_(S=0)
    d = _np_layer(cfg)
    W13 = np.repeat(d["W13"][:1], cfg.N, axis=0)
    W2 = np.repeat(d["W2"][:1], cfg.N, axis=0)
    r = orc.layer_forward(d["x"], d["W_gate"], d["gate_bias"], W13, W2, None, None,
                          cfg.K_orig, cfg.K_base, cfg.budget)
    mass = np.array([r["topk_score"][t, :r["n_sel"][t]].astype(np.float64).sum() for t in range(cfg.T)])
    want = mass[:, None] * orc.expert_ffn(d["x"], W13[0], W2[0])
    assert np.allclose(r["out"], want, rtol=1e-11, atol=1e-14)


def test_full_budget_is_a_standard_topk_moe_layer():
    """budget = K_orig*T: Eq. 1-2 with plain Top-K, written independently with torch."""
    cfg = SMALL
    d = _np_layer(cfg)
    got = orc.layer_forward(d["x"], d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"], d["Wsh2"],
                            cfg.K_orig, cfg.K_base, cfg.K_orig * cfg.T)["out"]
    x = torch.from_numpy(d["x"]).double()
    p = torch.softmax(x @ torch.from_numpy(d["W_gate"]).double() + torch.from_numpy(d["gate_bias"]).double(), 1).float()
    v, i = torch.topk(p, cfg.K_orig, dim=1)
    w = torch.zeros_like(p).scatter_(1, i, v).double()

    def ffn(W13, W2):
        W13, W2 = torch.from_numpy(W13).double(), torch.from_numpy(W2).double()
        return (torch.nn.functional.silu(x @ W13[:cfg.I].T) * (x @ W13[cfg.I:].T)) @ W2.T
    want = sum(w[:, e:e + 1] * ffn(d["W13"][e], d["W2"][e]) for e in range(cfg.N))
    want = want + sum(ffn(d["Wsh13"][s], d["Wsh2"][s]) for s in range(cfg.S))
    assert np.allclose(got, want.numpy(), rtol=1e-9, atol=1e-12)


def test_zero_budget_token_gets_shared_only():
    cfg = SMALL.with_(K_base=0, budget=5)
    d = _np_layer(cfg)
    r = orc.layer_forward(d["x"], d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"], d["Wsh2"],
                          cfg.K_orig, 0, 5)
    empty = np.flatnonzero(r["n_sel"] == 0)
    assert len(empty) > 0
    sh = orc.shared_experts(d["x"], d["Wsh13"], d["Wsh2"])
    assert np.allclose(r["out"][empty], sh[empty], rtol=1e-12, atol=1e-15)


def test_bf16_round_against_torch():
    a = np.concatenate([np.random.default_rng(0).standard_normal(4096).astype(np.float32),
                        np.array([1.00390625, 1.01171875, -1.00390625, 0.0], np.float32)])   # exact ties
    want = torch.from_numpy(a).to(torch.bfloat16).float().numpy()
    assert np.array_equal(orc.bf16_round(a), want)


def test_stack_is_the_residual_recurrence():
    cfg = SMALL.with_(n_layers=3, T=8)
    layers = [_np_layer(cfg.with_()) if l == 0 else
              {k: (None if v is None else v.float().numpy()) for k, v in synth.make_layer(cfg, l, with_x=False).items()}
              for l in range(3)]
    budgets = [8, 16, 24]
    xs = orc.stack_forward(layers[0]["x"], layers, cfg.K_orig, cfg.K_base, budgets)
    xs_literal = orc.stack_forward(layers[0]["x"], layers, cfg.K_orig, cfg.K_base, budgets, prenorm=False)
    x = layers[0]["x"]
    for l in range(3):
        lw = layers[l]
        xd = torch.from_numpy(x).double()
        xn = (xd * torch.rsqrt(xd.pow(2).mean(dim=1, keepdim=True) + 1e-6)).to(torch.bfloat16).float().numpy()
        o = orc.layer_forward(xn, lw["W_gate"], lw["gate_bias"], lw["W13"], lw["W2"], lw["Wsh13"], lw["Wsh2"],
                              cfg.K_orig, cfg.K_base, budgets[l])["out"]
        x = torch.from_numpy((x.astype(np.float64) + o).astype(np.float32)).to(torch.bfloat16).float().numpy()
        assert np.array_equal(xs[l], x)
    assert not np.array_equal(xs[0], xs_literal[0])


def test_rmsnorm_against_torch_and_unit_rms():
    x = np.random.default_rng(1).standard_normal((5, 64)) * 7.0
    xt = torch.from_numpy(x)
    want = xt * torch.rsqrt(xt.pow(2).mean(dim=1, keepdim=True) + 1e-6)
    got = orc.rmsnorm(x)
    assert np.allclose(got, want.numpy(), rtol=1e-13)
    assert np.allclose(np.sqrt((got ** 2).mean(axis=1)), 1.0, atol=1e-6)


@pytest.mark.parametrize("L,K", [(3, 4), (5, 3), (6, 3), (4, 6)])
def test_alloc_l_dp_equals_bruteforce(L, K):
    rng = np.random.default_rng(L * 10 + K)
    for trial in range(3):
        # decreasing-in-k costs like a perplexity profile, plus noise so it is not convex
        S = np.sort(rng.random((L, K)), axis=1)[:, ::-1] + 0.05 * rng.random((L, K))
        for B in range(L, L * K + 2):
            ks, cost = orc.alloc_l_dp(S, B)
            assert sum(ks) <= B and all(1 <= k <= K for k in ks)
            assert abs(cost - sum(S[i, ks[i] - 1] for i in range(L))) < 1e-12
            assert abs(cost - orc.alloc_l_bruteforce(S, B)) < 1e-12
    with pytest.raises(ValueError):
        orc.alloc_l_dp(S, L - 1)
