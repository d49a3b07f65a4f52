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
from helpers import (TOL_OUT, assert_close, check_routing_fed, dev_layer, forward_gpu, max_rel, np32,
                     tile_covering_tokens)

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
    assert_close(got, fed, cfg.name)
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


@pytest.mark.parametrize("S,T", [(1, 70), (0, 70), (2, 1500)])
def test_zero_budget_keeps_only_the_shared_experts(S, T):
    """K_base = 0 and budget = 0: no routed pair is kept (Sec. 4's K_base ablation allows tokens without a routed
    expert); the output is the shared experts' alone, or zero.  The same through the routed entry with n_sel = 0."""
    cfg = synth.MoEConfig("zero", T=T, H=128, N=8, I=128, S=S, K_orig=2, K_base=0, budget=0, seed=5)
    d = dev_layer(cfg)
    out, inter, status = forward_gpu(cfg, d, 0)
    assert status == 0
    assert int(inter["n_sel"].sum()) == 0 and int(inter["expert_offsets"][-1]) == 0
    assert (inter["pair_pos"] == -1).all()
    want = orc.shared_experts(np32(d["x"]), np32(d["Wsh13"]), np32(d["Wsh2"])) if S else np.zeros((T, cfg.H))
    got = out.float().cpu().numpy()
    if S:
        assert max_rel(got, want) <= TOL_OUT
    else:
        assert (got == 0).all()
    shape = B.shape_of(cfg)
    for bmax in (0, 10):
        ws = B.new_workspace(shape, bmax)
        out2 = torch.full_like(d["x"], 9.0)
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.moe_layer_forward_routed(shape, d["x"], inter["topk_idx"], inter["topk_score"], inter["n_sel"], bmax, 0, d["W13"],
                                   d["W2"], d["Wsh13"], d["Wsh2"], out2, st, ws)
        torch.cuda.synchronize()
        assert st.item() == 0 and torch.equal(out2, out)


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
    for _ in range(20):
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


# ----------------------------------------------------------------------------- full sizes, tile-covering rows
class _OnDemand:
    """Per-expert weights converted to fp32 numpy only when the oracle asks for expert e."""

    def __init__(self, t):
        self.t = t

    def __getitem__(self, e):
        return np32(self.t[e])


def _sampled_check(cfg, d, budget, x=None, residual=None, min_tokens=256, block=128, key=0):
    """One forward call at full size.  Routing is compared in full (bit-exact, oracle fed the GPU's scores).
    Outputs are compared on a token sample that reaches every tile of both expert GEMMs (block=128) or, with
    block=None, on min_tokens seeded random tokens."""
    out, inter, status = forward_gpu(cfg, d, budget, residual=residual, x=x)
    assert status == 0
    idx, sc, n_ref = check_routing_fed(cfg, inter, budget)
    rows = tile_covering_tokens(inter, cfg.T, cfg.S, min_tokens, block if block else 1 << 30, key)
    if block:      # the sample does reach every 128-row block of every expert's run
        off = inter["expert_offsets"].cpu().numpy()
        tok = inter["perm_token"].cpu().numpy()
        hit = np.zeros(cfg.T, bool)
        hit[rows] = True
        for e in range(cfg.N):
            for b0 in range(int(off[e]), int(off[e + 1]), block):
                assert hit[tok[b0:min(int(off[e + 1]), b0 + block)]].any()
        assert len(rows) >= min(min_tokens, cfg.T)
    xin = d["x"] if x is None else x
    ref = orc.combine(np32(xin), idx, sc, n_ref, _OnDemand(d["W13"]), _OnDemand(d["W2"]), np32(d["Wsh13"]),
                      np32(d["Wsh2"]), rows=rows)
    if residual is not None:
        ref = ref + np32(residual)[rows].astype(np.float64)
    assert bool(torch.isfinite(out.float()).all())
    m = assert_close(out.float().cpu().numpy()[rows], ref, f"{cfg.name} budget {budget}")
    return out, inter, m


def test_c3_prefill_full_size_budget_sweep():
    cfg = synth.CONFIGS["c3"]
    d = dev_layer(cfg)
    for mult in synth.C3_BUDGET_MULTS:
        budget = int(mult * cfg.T)
        _, inter, _ = _sampled_check(cfg, d, budget, key=int(mult * 10))
        off = inter["expert_offsets"].cpu().numpy()
        assert off[-1] == budget
    # free-running comparison of the routing at the paper's half budget
    dn = {k: np32(d[k]) for k in ("x", "W_gate", "gate_bias")}
    r = orc.route(dn["x"], dn["W_gate"], dn["gate_bias"], cfg.K_orig, cfg.K_base, 3 * cfg.T)
    _, inter, _ = forward_gpu(cfg, d, 3 * cfg.T)
    same = (r["n_sel"] == inter["n_sel"].cpu().numpy()) & (r["topk_idx"] == inter["topk_idx"].cpu().numpy()).all(axis=1)
    assert (~same).sum() <= cfg.T // 100


def test_c5_large_experts_full_size():
    cfg = synth.CONFIGS["c5"]
    d = dev_layer(cfg)
    _sampled_check(cfg, d, cfg.budget, key=5)


@pytest.mark.parametrize("name", ["qwen", "olmoe"])
def test_other_model_shapes_full_size(name):
    """The Qwen1.5-MoE-shaped (60 experts, Top-4, one shared expert) and OLMoE-shaped (64 experts, Top-8) prefill
    layers at their benchmark size: routing in full, outputs on a tile-covering token sample."""
    cfg = synth.CONFIGS[name]
    d = dev_layer(cfg)
    _, inter, _ = _sampled_check(cfg, d, cfg.budget, key=60 if name == "qwen" else 64)
    assert int(inter["expert_offsets"][-1]) == cfg.budget


def test_layer_beyond_8192_tokens_takes_the_unfused_routing_path():
    """Above 8192 tokens moe_layer_forward runs alloc_t_select and moe_permute's kernels one after the other instead
    of the one-launch routing step; small H and I keep the oracle's whole-layer run short."""
    cfg = synth.MoEConfig("t8200", T=8200, H=128, N=16, I=128, S=1, K_orig=4, K_base=1, budget=int(2.5 * 8200),
                          zipf_bias=True, seed=8200)
    _full_check(cfg)
    _full_check(cfg.with_(K_base=0, budget=8200 + 77))


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
    x_{l+1} = x_l + MoE_l(rmsnorm(x_l)).  Every layer's routing is checked in full; every layer's output is
    checked against the oracle run on the GPU's own input to that layer (teacher forcing, so errors do not
    compound): on a tile-covering token sample for layers 0, 12 and 25, on 32 random tokens for the others."""
    cfg = synth.CONFIGS["c4"]
    ks = synth.stack_budgets(cfg)
    shape = B.shape_of(cfg)
    x = synth.make_layer(cfg.with_(N=8, I=64, S=0), 0, device="cuda")["x"]
    xn = torch.empty_like(x)
    for l in range(cfg.n_layers):
        d = dev_layer(cfg, l, with_x=False)
        budget = ks[l] * cfg.T
        B.moe_rmsnorm(shape, x, xn)
        if l in (0, 12, 25):
            out, _, _ = _sampled_check(cfg, d, budget, x=xn, residual=x, key=100 + l)
        else:
            out, _, _ = _sampled_check(cfg, d, budget, x=xn, residual=x, min_tokens=32, block=None, key=100 + l)
        assert 0.5 < float(out.float().std()) < 50.0          # the pre-norm stream grows slowly
        x = out
        del d


def test_c4_literal_recurrence_first_layers():
    """The stack as the workload list writes it, x_{l+1} = x_l + MoE_l(x_l) with no normalisation, over the first
    four layers, where the stream is still finite (its scale roughly squares from layer to layer)."""
    cfg = synth.CONFIGS["c4"]
    ks = synth.stack_budgets(cfg)
    x = synth.make_layer(cfg.with_(N=8, I=64, S=0), 0, device="cuda")["x"]
    for l in range(4):
        d = dev_layer(cfg, l, with_x=False)
        out, _, _ = _sampled_check(cfg, d, ks[l] * cfg.T, x=x, residual=x, min_tokens=64, key=200 + l)
        assert bool(torch.isfinite(out.float()).all())
        x = out
        del d


@pytest.mark.parametrize("name,T,budget", [("c2", 64, 192), ("c4l", 1500, 4500), ("c2", 9000, 20000)])
def test_global_selection_path_equals_the_fused_call_on_one_rank(name, T, budget):
    """With one rank the batch-wide selection is the local one: gate, selection over the (one-rank) pool and
    moe_layer_forward_routed -- the path of dist.py -- must give the fused call's output bit for bit: by-index
    rows (c2), the cluster routing kernel with the row gather (c4l), the unfused routing kernels (9000 tokens)."""
    from paper_2604_08133_b200 import dist as D
    cfg = synth.CONFIGS[name].with_(T=T, budget=budget)
    if T == 9000:
        cfg = cfg.with_(H=128, I=128, N=16)
    d = dev_layer(cfg)
    out_fused, inter, status = forward_gpu(cfg, d)
    assert status == 0
    shape = B.shape_of(cfg)
    out = torch.empty_like(d["x"])
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    layer = D.GlobalAllocTLayer(shape, "cuda")
    for _ in range(2):
        out.zero_()
        layer.forward(d["x"], d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"], d["Wsh2"], cfg.budget, out, st)
        torch.cuda.synchronize()
        assert st.item() == 0
        assert torch.equal(out, out_fused)
    # an upper bound that is too small is reported, and nothing is written out of bounds
    n_sel = inter["n_sel"]
    ws = B.new_workspace(shape, cfg.budget - 1)
    guard = torch.full((cfg.T + 4, cfg.H), 3.0, dtype=torch.bfloat16, device="cuda")
    B.moe_layer_forward_routed(shape, d["x"], inter["topk_idx"], inter["topk_score"], n_sel, cfg.budget - 1, 0, d["W13"],
                               d["W2"], d["Wsh13"], d["Wsh2"], guard[:cfg.T], st, ws)
    torch.cuda.synchronize()
    assert st.item() & (1 << B.MOE_ERR_BUDGET)
    assert (guard[cfg.T:] == 3.0).all()


def test_global_selection_over_nccl_at_world_size_one():
    """The exchange itself on the GPU: a one-rank NCCL group, the all-gather forced to run, the library's selection
    on the gathered pool, then the routed layer call; bit-identical to the fused call."""
    import os
    import torch.distributed as dist
    from paper_2604_08133_b200 import dist as D
    cfg = synth.CONFIGS["c4l"].with_(T=1024, budget=3 * 1024)
    d = dev_layer(cfg)
    out_fused, _, status = forward_gpu(cfg, d)
    assert status == 0
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", str(29400 + os.getpid() % 500))
    os.environ.setdefault("NCCL_NVLS_ENABLE", "0")
    own = not dist.is_initialized()
    if own:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        shape = B.shape_of(cfg)
        layer = D.GlobalAllocTLayer(shape, "cuda", always_collective=True)
        out = torch.empty_like(d["x"])
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        layer.forward(d["x"], d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"], d["Wsh2"], cfg.budget, out, st)
        torch.cuda.synchronize()
        assert layer.pool.data_ptr() != layer.topk_score.data_ptr() and torch.equal(layer.pool, layer.topk_score)
        assert st.item() == 0
        assert torch.equal(out, out_fused)
    finally:
        if own:
            dist.destroy_process_group()


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

