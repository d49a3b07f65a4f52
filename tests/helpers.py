"""Shared helpers of the GPU parity tests (input marshalling and error measures only)."""
import numpy as np
import torch

from oracle import alloc_moe_oracle as orc
from paper_2604_08133_b200 import binding as B
from paper_2604_08133_b200 import synth

TOL_OUT = 2e-2     # max |gpu - ref| / max |ref| per tensor (bf16 path vs fp64 oracle)
# Two further measures of the same comparison, both free of the blow-up of a pure element-wise relative
# error at zero crossings.  h, y_perm and the output are each rounded to bf16 once (relative step 2^-9 per
# rounding, about 2e-3), so an output element's error has a standard deviation of about 2.5e-3 of the
# tensor's RMS; over the 1e5..1e7 compared elements its maximum reaches five to six of those.
TOL_ELEMENTWISE = 2e-2   # max over elements of |gpu - ref| / (|ref| + rms(ref))
TOL_RMS = 5e-3           # rms(gpu - ref) / rms(ref)


def np32(t):
    return None if t is None else t.detach().float().cpu().numpy()


def max_rel(gpu, ref):
    gpu = np.asarray(gpu, np.float64)
    ref = np.asarray(ref, np.float64)
    return float(np.abs(gpu - ref).max() / max(np.abs(ref).max(), 1e-30))


def err_measures(gpu, ref):
    """(max |d| / max |ref|,  max |d| / (|ref| + rms(ref)),  rms(d) / rms(ref))."""
    gpu = np.asarray(gpu, np.float64)
    ref = np.asarray(ref, np.float64)
    d = np.abs(gpu - ref)
    rms = max(float(np.sqrt((ref * ref).mean())), 1e-30)
    return (float(d.max() / max(np.abs(ref).max(), 1e-30)), float((d / (np.abs(ref) + rms)).max()),
            float(np.sqrt((d * d).mean()) / rms))


def assert_close(gpu, ref, what=""):
    """The three output measures against their bounds; returns them for reporting."""
    m = err_measures(gpu, ref)
    assert m[0] <= TOL_OUT, f"{what}: max|d|/max|ref| = {m[0]:.3e}"
    assert m[1] <= TOL_ELEMENTWISE, f"{what}: element-wise measure = {m[1]:.3e}"
    assert m[2] <= TOL_RMS, f"{what}: rms relative error = {m[2]:.3e}"
    return m


def tile_covering_tokens(inter, T, S, min_tokens=256, block=128, key=0):
    """Tokens whose output rows together touch every tile of the expert GEMMs of one forward call: for every
    routed expert the first and the last row of its run and one row in every `block`-row piece of it (128 rows:
    a one-CTA tile, half of a CTA-pair tile), one token in every `block` tokens for the shared experts' tiles,
    filled up with seeded random tokens to at least min_tokens.  Built from the GPU's own expert_offsets and
    perm_token, which the caller has already checked against the oracle."""
    off = inter["expert_offsets"].cpu().numpy()
    tok = inter["perm_token"].cpu().numpy()
    pick = set()
    for e in range(len(off) - 1):
        lo, hi = int(off[e]), int(off[e + 1])
        if hi <= lo:
            continue
        rows = {lo, hi - 1}
        for b0 in range(lo, hi, block):
            b1 = min(hi, b0 + block)
            rows.add(b0 + (synth.mix64_int(key * 1000003 + b0) % (b1 - b0)))
        pick.update(int(tok[r]) for r in rows)
    if S > 0:
        for b0 in range(0, T, block):
            b1 = min(T, b0 + block)
            pick.add(b0 + (synth.mix64_int(key * 7919 + b0 + 17) % (b1 - b0)))
    for t in synth.permutation(T, synth.stream_key(123, key)):
        if len(pick) >= min(min_tokens, T):
            break
        pick.add(int(t))
    return sorted(pick)


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
