"""Whole-layer parity of moe_layer_forward against the CPU oracle on the five workloads.

Two comparisons (the GPU's fp32 scores differ from the oracle's in the last bits, so a pair whose
score sits within an ulp or two of the selection threshold may flip):
  fed   the oracle's Alloc-T, permutation, experts and Eq. 2 run on the GPU's own Top-K scores:
        selection, offsets and permutation must be bit-exact, outputs within TOL_OUT;
  free  the oracle runs end to end from x: flipped pairs are counted and must be rare and
        near-ties; outputs are compared on tokens whose selection is identical.
"""
import numpy as np
import pytest
import torch

from oracle import alloc_moe_oracle as orc
from paper_2604_08133_b200 import binding as B
from paper_2604_08133_b200 import synth
from helpers import TOL_OUT, check_routing_fed, dev_layer, forward_gpu, max_rel, np32

pytestmark = pytest.mark.gpu


def _cpu(d):
    return {k: np32(v) for k, v in d.items()}


def _full_check(cfg, budget=None):
    budget = cfg.budget if budget is None else budget
    d = dev_layer(cfg)
    out, inter, status = forward_gpu(cfg, d, budget)
    assert status == 0
    idx, sc, n_ref = check_routing_fed(cfg, inter, budget)
    dn = _cpu(d)
    got = out.float().cpu().numpy()
    # fed: Eq. 2 on the GPU's routing
    fed = orc.combine(dn["x"], idx, sc, n_ref, dn["W13"], dn["W2"], dn["Wsh13"], dn["Wsh2"])
    assert max_rel(got, fed) <= TOL_OUT
    # free: oracle end to end
    free = orc.layer_forward(dn["x"], dn["W_gate"], dn["gate_bias"], dn["W13"], dn["W2"], dn["Wsh13"], dn["Wsh2"],
                             cfg.K_orig, cfg.K_base, budget)
    same = (free["n_sel"] == n_ref) & (free["topk_idx"] == idx).all(axis=1)
    flips = int((~same).sum())
    assert flips <= max(1, cfg.T // 100), f"{flips} tokens with a different selection"
    assert max_rel(got[same], free["out"][same]) <= TOL_OUT
    return flips


def test_c1_degenerate_top1():
    cfg = synth.CONFIGS["c1"]
    _full_check(cfg)
    # K_base = K_l: plain Top-1 routing
    _, inter, _ = forward_gpu(cfg, dev_layer(cfg))
    assert (inter["n_sel"] == 1).all()


def test_c1_kbase0_redistributes():
    cfg = synth.CONFIGS["c1k0"]
    _full_check(cfg)
    _, inter, _ = forward_gpu(cfg, dev_layer(cfg))
    n = inter["n_sel"].cpu().numpy()
    assert n.sum() == 64 and n.min() == 0 and n.max() == 2      # budget moved between tokens


def test_c2_decode():
    cfg = synth.CONFIGS["c2"]
    _full_check(cfg)
    _full_check(cfg, budget=6 * cfg.T)       # full Top-K_orig, the unbudgeted layer


def test_ragged_multi_tile_layer():
    # several 128-row tiles per expert with ragged ends, a partial column tile (I=192), S=1
    cfg = synth.CONFIGS["c2"].with_(T=700, H=256, N=8, I=192, S=1, K_orig=3, K_base=1, budget=1500)
    _full_check(cfg)
    cfg = cfg.with_(K_base=0, budget=701)
    _full_check(cfg)


def test_residual_flag_adds_the_input():
    cfg = synth.CONFIGS["c1k0"]
    d = dev_layer(cfg)
    out0, _, _ = forward_gpu(cfg, d)
    out1, inter, _ = forward_gpu(cfg, d, residual=d["x"])
    dn = _cpu(d)
    ref = orc.combine(dn["x"], inter["topk_idx"].cpu().numpy(), inter["topk_score"].cpu().numpy(),
                      inter["n_sel"].cpu().numpy(), dn["W13"], dn["W2"]) + dn["x"].astype(np.float64)
    assert max_rel(out1.float().cpu().numpy(), ref) <= 4e-3
    assert not torch.equal(out0, out1)


def test_forward_is_deterministic():
    cfg = synth.CONFIGS["c2"]
    d = dev_layer(cfg)
    a, ia, _ = forward_gpu(cfg, d)
    for _ in range(5):
        b, ib, _ = forward_gpu(cfg, d)
        assert torch.equal(a, b)
        assert torch.equal(ia["perm_token"], ib["perm_token"])


@pytest.mark.parametrize("name", ["c2", "c4l"])
def test_layer_forward_replays_from_a_cuda_graph(name):
    """The call only enqueues work on the caller's stream (kernels as programmatic dependents, cluster launches, one
    memset), so it can be captured once and replayed: same bits as the direct call, also after x changed in place."""
    cfg = synth.CONFIGS[name]
    if name == "c4l":
        cfg = cfg.with_(T=1500, budget=3 * 1500)          # cluster routing kernel, ragged last segment
    d = dev_layer(cfg)
    shape = B.shape_of(cfg)
    ws = B.new_workspace(shape, cfg.budget)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    x = d["x"].clone()
    args = (shape, x, d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"], d["Wsh2"], cfg.budget)
    want0 = torch.empty_like(x)
    B.moe_layer_forward(*args, want0, status, ws)            # also the first call: one-time attribute set-up
    out = torch.empty_like(x)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            B.moe_layer_forward(*args, out, status, ws)
    torch.cuda.current_stream().wait_stream(side)
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert status.item() == 0
    assert torch.equal(out, want0)
    x.copy_(torch.roll(d["x"], 7, dims=0))
    want1 = torch.empty_like(x)
    graph.replay()
    B.moe_layer_forward(*args, want1, status, ws)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert torch.equal(out, want1)
    assert not torch.equal(out, want0)


def test_host_checked_errors_launch_nothing():
    cfg = synth.CONFIGS["c1"]
    d = dev_layer(cfg)
    shape = B.shape_of(cfg)
    ws = B.new_workspace(shape, cfg.K_orig * cfg.T)
    out = torch.full_like(d["x"], 7.0)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = (d["x"], d["W_gate"], None, d["W13"], d["W2"], None, None)
    for budget, want in ((cfg.T - 1, B.MOE_ERR_BUDGET), (cfg.K_orig * cfg.T + 1, B.MOE_ERR_BUDGET)):
        with pytest.raises(B.MoeError) as ei:
            B.moe_layer_forward(shape, *args, budget, out, st, ws)
        assert ei.value.status == want
    with pytest.raises(B.MoeError) as ei:
        B.moe_layer_forward(shape, *args, cfg.budget, out, st, ws[:1024])
    assert ei.value.status == B.MOE_ERR_WORKSPACE
    bad = B.make_shape(cfg.T, cfg.H + 1, cfg.N, cfg.I, 0, 2, 1)
    with pytest.raises(B.MoeError) as ei:
        B.moe_layer_forward(bad, *args, cfg.budget, out, st, ws)
    assert ei.value.status == B.MOE_ERR_ARG
    with pytest.raises(B.MoeError) as ei:
        B.moe_layer_forward(shape, d["x"].view(-1)[1:], *args[1:], cfg.budget, out, st, ws)   # misaligned x
    assert ei.value.status == B.MOE_ERR_ARG
    torch.cuda.synchronize()
    assert (out == 7.0).all() and st.item() == 0


# ----------------------------------------------------------------------------- full sizes, sampled rows
def _sampled_check(cfg, d, budget, rows, x=None, residual=None):
    out, inter, status = forward_gpu(cfg, d, budget, residual=residual, x=x)
    assert status == 0
    idx, sc, n_ref = check_routing_fed(cfg, inter, budget)
    xin = d["x"] if x is None else x
    xn = np32(xin)
    ref = orc.combine(xn, idx, sc, n_ref, np32(d["W13"]), np32(d["W2"]), np32(d["Wsh13"]), np32(d["Wsh2"]), rows=rows)
    if residual is not None:
        ref = ref + np32(residual)[rows].astype(np.float64)
    got = out.float().cpu().numpy()[rows]
    assert bool(torch.isfinite(out.float()).all())
    assert max_rel(got, ref) <= TOL_OUT
    return out, inter


def _sample_rows(T, n, key):
    return sorted(set(synth.permutation(T, synth.stream_key(123, key))[:n]))


def test_c3_prefill_full_size_budget_sweep():
    cfg = synth.CONFIGS["c3"]
    d = dev_layer(cfg)
    rows = _sample_rows(cfg.T, 48, 3)
    touched = []
    for mult in synth.C3_BUDGET_MULTS:
        budget = int(mult * cfg.T)
        _, inter = _sampled_check(cfg, d, budget, rows if mult == 3.0 else rows[:8])
        off = inter["expert_offsets"].cpu().numpy()
        assert off[-1] == budget
        touched.append(int((np.diff(off) > 0).sum()))
    # free-running comparison of the routing at the paper's half budget
    dn = {k: np32(d[k]) for k in ("x", "W_gate", "gate_bias")}
    r = orc.route(dn["x"], dn["W_gate"], dn["gate_bias"], cfg.K_orig, cfg.K_base, 3 * cfg.T)
    _, inter, _ = forward_gpu(cfg, d, 3 * cfg.T)
    same = (r["n_sel"] == inter["n_sel"].cpu().numpy()) & (r["topk_idx"] == inter["topk_idx"].cpu().numpy()).all(axis=1)
    assert (~same).sum() <= cfg.T // 100


def test_c5_large_experts_full_size():
    cfg = synth.CONFIGS["c5"]
    d = dev_layer(cfg)
    _sampled_check(cfg, d, cfg.budget, _sample_rows(cfg.T, 12, 5))


def test_rmsnorm_against_oracle():
    cfg = synth.CONFIGS["c4"].with_(T=300)
    x = (synth.normal_bf16((cfg.T, cfg.H), 3.0, 11).cuda())
    out = torch.empty_like(x)
    B.moe_rmsnorm(B.shape_of(cfg), x, out)
    torch.cuda.synchronize()
    want = orc.rmsnorm(np32(x))
    got = out.float().cpu().numpy()
    assert np.abs(got - want).max() <= 2 ** -8 * np.abs(want).max() * 1.01


def test_c4_stack_teacher_forced():
    """26 layers, per-layer budgets, pre-norm residual stream in bf16:
    x_{l+1} = x_l + MoE_l(rmsnorm(x_l)).  Every layer's routing is checked in full; outputs of
    three layers are checked on sampled rows, each against the oracle run on the GPU's own input to
    that layer (teacher forcing, so errors do not compound)."""
    cfg = synth.CONFIGS["c4"]
    ks = synth.stack_budgets(cfg)
    shape = B.shape_of(cfg)
    x = synth.make_layer(cfg.with_(N=8, I=64, S=0), 0, device="cuda")["x"]
    xn = torch.empty_like(x)
    rows = _sample_rows(cfg.T, 16, 4)
    for l in range(cfg.n_layers):
        d = dev_layer(cfg, l, with_x=False)
        budget = ks[l] * cfg.T
        B.moe_rmsnorm(shape, x, xn)
        if l in (0, 12, 25):
            out, _ = _sampled_check(cfg, d, budget, rows, x=xn, residual=x)
        else:
            out, inter, status = forward_gpu(cfg, d, budget, residual=x, x=xn)
            assert status == 0
            check_routing_fed(cfg, inter, budget)
        assert bool(torch.isfinite(out.float()).all())
        assert 0.5 < float(out.float().std()) < 50.0          # the pre-norm stream grows slowly
        x = out
        del d


def test_global_selection_path_equals_the_fused_call_on_one_rank():
    """With one rank the batch-wide selection is the local one: the step-by-step path of dist.py (gate, selection,
    permute, experts, combine as separate C-ABI calls) must give the fused call's output bit for bit."""
    from paper_2604_08133_b200 import dist as D
    cfg = synth.CONFIGS["c2"]
    d = dev_layer(cfg)
    out_fused, inter, status = forward_gpu(cfg, d)
    assert status == 0
    shape = B.shape_of(cfg)
    out = torch.empty_like(d["x"])
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    b_local = D.moe_layer_forward_global(shape, d["x"], d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"],
                                         d["Wsh2"], cfg.budget, out, st)
    torch.cuda.synchronize()
    assert st.item() == 0 and b_local == cfg.budget
    assert torch.equal(out, out_fused)


@pytest.mark.parametrize("name,T,mult", [("qwen", 320, 2.5), ("qwen", 320, 3.5), ("olmoe", 256, 5.0), ("olmoe", 256, 7.0)])
def test_other_model_shapes(name, T, mult):
    """Qwen1.5-MoE-shaped (60 experts: not a multiple of 8, Top-4) and OLMoE-shaped (Top-8: a residual pool seven
    columns wide) layers at a size the oracle finishes in seconds."""
    cfg = synth.CONFIGS[name].with_(T=T, budget=int(mult * T))
    _full_check(cfg)


@pytest.mark.parametrize("T,H,N,I,S,K,kb,budget", [
    (1, 64, 8, 64, 0, 2, 1, 1),            # one token, the smallest sizes the ABI accepts
    (33, 192, 12, 128, 1, 3, 0, 40),        # N a multiple of 4 only, K_base 0, ragged everything
    (130, 128, 128, 192, 0, 16, 2, 1000),   # the largest N and K_orig
    (257, 256, 8, 64, 3, 4, 4, 1028),       # K_base = K_orig: nothing to redistribute, three shared experts
    (300, 128, 8, 128, 2, 4, 1, 1200),      # budget = K_orig*T: plain Top-K_orig
    (700, 128, 4 * 2, 256, 1, 2, 1, 1390),  # ~174 rows per expert: the CTA-pair tiles, with a shared expert
    (1030, 64, 16, 64, 0, 4, 1, 2000),      # just past 1024 tokens: routing cluster whose second CTA holds 6 tokens
    (2100, 128, 128, 64, 1, 16, 3, 9000),   # routing cluster of 3 CTAs at the largest N and K_orig; row-indexed A loads
    (1500, 64, 8, 128, 3, 2, 0, 1600),      # three shared sub-experts (GEMM-2 tiles of triple length), K_base 0
    (40, 320, 20, 448, 2, 5, 1, 41),        # budget one above K_base*T: a single redistributed pair
])
def test_odd_shapes(T, H, N, I, S, K, kb, budget):
    cfg = synth.MoEConfig("odd", T=T, H=H, N=N, I=I, S=S, K_orig=K, K_base=kb, budget=budget, zipf_bias=(N >= 12), seed=T)
    _full_check(cfg)

