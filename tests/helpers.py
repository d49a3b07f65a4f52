"""Shared helpers of the GPU parity tests (input marshalling and error measures only)."""
import numpy as np
import torch

from oracle import alloc_moe_oracle as orc
from paper_2604_08133_b200 import binding as B
from paper_2604_08133_b200 import synth

TOL_OUT = 2e-2     # max |gpu - ref| / max |ref| per tensor (bf16 path vs fp64 oracle)


def np32(t):
    return None if t is None else t.detach().float().cpu().numpy()


def max_rel(gpu, ref):
    gpu = np.asarray(gpu, np.float64)
    ref = np.asarray(ref, np.float64)
    return float(np.abs(gpu - ref).max() / max(np.abs(ref).max(), 1e-30))


def dev_layer(cfg, layer=0, with_x=True):
    return synth.make_layer(cfg, layer, device="cuda", with_x=with_x)


def forward_gpu(cfg, d, budget=None, residual=None, x=None):
    """One moe_layer_forward call; returns (out bf16 [T,H], intermediates dict, dev_status int)."""
    budget = cfg.budget if budget is None else budget
    shape = B.shape_of(cfg)
    ws = B.new_workspace(shape, budget)
    x = d["x"] if x is None else x
    out = torch.empty_like(x)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.moe_layer_forward(shape, x, d["W_gate"], d["gate_bias"], d["W13"], d["W2"], d["Wsh13"], d["Wsh2"],
                        budget, out, status, ws, residual=residual)
    torch.cuda.synchronize()
    inter = B.moe_layer_intermediates(shape, budget, ws)
    return out, inter, int(status.item())


def check_routing_fed(cfg, inter, budget):
    """Selection, offsets and permutation must be bit-exact when the oracle is fed the GPU's scores."""
    idx = inter["topk_idx"].cpu().numpy()
    sc = inter["topk_score"].cpu().numpy()
    z = orc.alloc_t_select_threshold(sc, cfg.K_base, budget)
    n_ref = orc.n_sel_from_mask(z)
    assert np.array_equal(inter["n_sel"].cpu().numpy(), n_ref)
    p = orc.permute(idx, sc, n_ref, cfg.N)
    assert np.array_equal(inter["expert_offsets"].cpu().numpy(), p["expert_offsets"])
    assert np.array_equal(inter["perm_token"].cpu().numpy(), p["perm_token"])
    assert np.array_equal(inter["pair_pos"].cpu().numpy(), p["pair_pos"])
    return idx, sc, n_ref
