"""Pins for the oracle's Eq. 1 steps: library routines, closed forms, tie order."""
import numpy as np
import torch

from oracle import alloc_moe_oracle as orc
from paper_2604_08133_b200 import synth


def _layer(name="c1", **kw):
    cfg = synth.CONFIGS[name].with_(**kw)
    d = synth.make_layer(cfg)
    return cfg, {k: (None if v is None else v.float().numpy()) for k, v in d.items()}


def test_logits_and_softmax_against_torch_fp64():
    cfg, d = _layer("c2", T=16, I=64)
    z = orc.gate_logits(d["x"], d["W_gate"], d["gate_bias"])
    zt = torch.from_numpy(d["x"]).double() @ torch.from_numpy(d["W_gate"]).double() + torch.from_numpy(d["gate_bias"]).double()
    assert np.allclose(z, zt.numpy(), rtol=0, atol=1e-12)
    p = orc.softmax_scores(z)
    pt = torch.softmax(zt, dim=1).float().numpy()
    assert p.dtype == np.float32
    assert np.max(np.abs(p - pt)) <= 2 ** -24
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-6)


def test_bias_shifts_logits_not_omitted():
    cfg, d = _layer("c2", T=4, I=64)
    z0 = orc.gate_logits(d["x"], d["W_gate"], None)
    z1 = orc.gate_logits(d["x"], d["W_gate"], d["gate_bias"])
    assert np.allclose(z1 - z0, d["gate_bias"][None, :].astype(np.float64), atol=1e-12)


def test_softmax_closed_forms():
    # equal logits -> uniform; a shift does not change the result; two-expert case is a logistic
    assert np.allclose(orc.softmax_scores(np.zeros((2, 8))), 1 / 8)
    z = np.array([[0.3, -1.2, 2.0]])
    assert np.array_equal(orc.softmax_scores(z), orc.softmax_scores(z + 1000.0))
    a = 0.7
    p = orc.softmax_scores(np.array([[a, 0.0]]))
    assert abs(p[0, 0] - 1 / (1 + np.exp(-a))) < 1e-7


def test_topk_against_torch_topk():
    cfg, d = _layer("c2", T=64, I=64)
    p = orc.softmax_scores(orc.gate_logits(d["x"], d["W_gate"], d["gate_bias"]))
    idx, val = orc.topk_sorted(p, 6)
    tv, ti = torch.topk(torch.from_numpy(p), 6, dim=1)
    assert np.array_equal(val, tv.numpy())
    distinct = np.array([len(set(r)) == len(r) for r in p])
    assert distinct.any()
    assert np.array_equal(idx[distinct], ti.numpy()[distinct])
    assert (val[:, :-1] >= val[:, 1:]).all()
    assert np.array_equal(np.take_along_axis(p, idx.astype(np.int64), axis=1), val)


def test_topk_ties_prefer_lower_expert():
    p = np.array([[0.2, 0.3, 0.3, 0.2]], np.float32)
    idx, val = orc.topk_sorted(p, 3)
    assert idx.tolist() == [[1, 2, 0]]
    assert val.tolist() == [[np.float32(0.3), np.float32(0.3), np.float32(0.2)]]


def test_c5_gate_scale_gives_mean_top1_of_0p6():
    cfg = synth.CONFIGS["c5"].with_(T=1024)
    x = synth.normal_bf16((cfg.T, cfg.H), 1.0, synth.stream_key(cfg.seed, 0, 0)).float().numpy()
    Wg = synth.normal_bf16((cfg.H, cfg.N), 0.02 * cfg.gate_scale, synth.stream_key(cfg.seed, 0, 1)).float().numpy()
    p = orc.softmax_scores(orc.gate_logits(x, Wg))
    assert abs(float(p.max(axis=1).mean()) - 0.60) < 0.01
