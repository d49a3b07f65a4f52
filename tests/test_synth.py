"""The seeded generator: integer-exact, chunk-independent, right moments, right shapes."""
import math

import numpy as np
import torch

from paper_2604_08133_b200 import synth


def test_torch_hash_equals_python_ints():
    key = synth.stream_key(7, 3, 1)
    idx = torch.tensor([0, 1, 2, 12345, (1 << 24) - 1, 1 << 24, 553_648_127], dtype=torch.int64)
    got = synth._irwin_hall_int(key, idx).tolist()
    want = [synth.irwin_hall_int_ref(key, int(i)) for i in idx]
    assert got == want


def test_chunk_independent_and_deterministic():
    key = synth.stream_key(0, 0, 2)
    old = synth._CHUNK
    a = synth.normal_bf16((1000, 37), 0.02, key)
    try:
        synth._CHUNK = 4099
        b = synth.normal_bf16((1000, 37), 0.02, key)
    finally:
        synth._CHUNK = old
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    c = synth.normal_bf16((1000, 37), 0.02, synth.stream_key(0, 0, 3))
    assert not torch.equal(a, c)


def test_moments():
    z = synth.normal_bf16((1 << 20,), 1.0, synth.stream_key(1, 2)).float()
    assert abs(z.mean().item()) < 5e-3
    assert abs(z.std().item() - 1.0) < 5e-3
    assert z.abs().max().item() <= 6.0
    w = synth.normal_bf16((1 << 18,), 0.02, synth.stream_key(1, 3)).float()
    assert abs(w.std().item() - 0.02) < 2e-4


def test_layer_shapes_and_bias():
    cfg = synth.CONFIGS["c2"].with_(T=8, H=64, I=128)
    d = synth.make_layer(cfg)
    assert d["x"].shape == (8, 64) and d["x"].dtype == torch.bfloat16
    assert d["W_gate"].shape == (64, 64)
    assert d["W13"].shape == (64, 256, 64) and d["W2"].shape == (64, 64, 128)
    assert d["Wsh13"].shape == (2, 256, 64) and d["Wsh2"].shape == (2, 64, 128)
    b = d["gate_bias"].numpy()
    assert b.shape == (64,) and abs(b.max() - 0.5) < 1e-7
    ranks = np.sort((b / 0.5) ** (-1 / 1.1))
    assert np.allclose(ranks, np.arange(1, 65), rtol=1e-4)
    assert synth.make_layer(synth.CONFIGS["c1"])["gate_bias"] is None


def test_stack_budgets():
    cfg = synth.CONFIGS["c4"]
    k = synth.stack_budgets(cfg)
    assert len(k) == 26 and sum(k) == 78
    assert all(1 <= v <= 6 for v in k)
    assert len(set(k)) > 1
    assert k == synth.stack_budgets(cfg)
    for tot in (26, 60, 156):
        kk = synth.stack_budgets(cfg, tot)
        assert sum(kk) == tot and all(1 <= v <= 6 for v in kk)


def test_score_rows_sorted_positive():
    s = synth.score_rows(100, 6, 5)
    assert (s[:, :-1] >= s[:, 1:]).all() and (s > 0).all()
    st = synth.score_rows(100, 6, 5, ties=True)
    assert len(torch.unique(st)) <= 12
