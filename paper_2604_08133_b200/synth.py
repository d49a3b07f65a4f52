"""Seeded synthetic inputs for the budgeted MoE layer (workload shapes of the
paper's Table 1 DeepSeek-V2-Lite row: 26 MoE layers, 6 of 64 routed experts;
hidden / intermediate sizes, shared experts and the gate bias are workload
parameters the paper does not give).

This module holds NO arithmetic of the method (no softmax, no routing, no
selection, no expert math).  It only draws numbers: every element of every
tensor is a pure function of (seed, tensor id, element index), computed with
wrapping 64-bit integer arithmetic, so the same bits come out on the CPU and
on a CUDA device and in any chunking.  Both the CPU oracle's tests and the
CUDA path's tests draw their inputs from here.

Normal deviates are an Irwin-Hall sum of twelve 16-bit uniforms (exactly
representable in fp32), scaled by one fp32 multiply and rounded to bf16 with
round-to-nearest-even.  Tails end at +-6 sigma and the excess kurtosis is -0.1;
that is irrelevant for the workloads here and keeps the generator free of
transcendental functions (which differ between CPU and GPU libraries).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import torch

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB


def _signed(v: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant (torch has no uint64 math)."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def mix64_int(v: int) -> int:
    """splitmix64 finaliser on a Python int (reference form of `_mix64_t`)."""
    v &= _MASK64
    v = ((v ^ (v >> 30)) * _M1) & _MASK64
    v = ((v ^ (v >> 27)) * _M2) & _MASK64
    return v ^ (v >> 31)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64_t(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _signed(_M1)
    x = (x ^ _lsr(x, 27)) * _signed(_M2)
    return x ^ _lsr(x, 31)


def stream_key(seed: int, *ids: int) -> int:
    """Key of one tensor's random stream: a hash chain over (seed, ids...)."""
    k = mix64_int(seed + _GOLDEN)
    for i in ids:
        k = mix64_int(k ^ mix64_int((int(i) + 1) * _GOLDEN))
    return k


def _irwin_hall_int(key: int, idx: torch.Tensor) -> torch.Tensor:
    """Sum of twelve 16-bit uniforms per element index (int64, 0 .. 12*65535)."""
    h = _mix64_t(idx * _signed(_GOLDEN) + _signed(key))
    total = torch.zeros_like(idx)
    for r in range(3):
        if r:
            h = _mix64_t(h + _signed((_GOLDEN * (r + 1)) & _MASK64))
        total += (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)
    return total


def irwin_hall_int_ref(key: int, i: int) -> int:
    """Pure-Python form of `_irwin_hall_int` for one element (used by tests)."""
    h = mix64_int((i * _GOLDEN + key) & _MASK64)
    total = 0
    for r in range(3):
        if r:
            h = mix64_int((h + _GOLDEN * (r + 1)) & _MASK64)
        total += (h & 0xFFFF) + ((h >> 16) & 0xFFFF) + ((h >> 32) & 0xFFFF) + (h >> 48)
    return total


_CHUNK = 1 << 24


def normal_bf16(shape, std: float, key: int, device="cpu") -> torch.Tensor:
    """bf16 tensor of ~N(0, std^2) deviates; element i depends only on (key, i)."""
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    scale = torch.tensor(float(std) / 131072.0, dtype=torch.float32, device=device)
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        s = _irwin_hall_int(key, idx)
        # 2*sum - 12*65535 is an integer below 2^21: exact in fp32.
        z = (2 * s - 12 * 65535).to(torch.float32)
        out[lo:hi] = (z * scale).to(torch.bfloat16)
    return out.reshape(*shape)


def uniform01(n: int, key: int) -> List[float]:
    """n host-side uniforms in (0,1) (53-bit), for the small host-drawn profiles."""
    out = []
    for i in range(n):
        h = mix64_int((i * _GOLDEN + key) & _MASK64)
        out.append(((h >> 11) + 0.5) / float(1 << 53))
    return out


def permutation(n: int, key: int) -> List[int]:
    """Seeded permutation of 0..n-1 (argsort of n hashes)."""
    hs = [mix64_int((i * _GOLDEN + key) & _MASK64) for i in range(n)]
    return sorted(range(n), key=lambda i: (hs[i], i))


@dataclasses.dataclass(frozen=True)
class MoEConfig:
    """One synthetic workload.  `budget` is the layer's TOTAL activation count."""
    name: str
    T: int
    H: int
    N: int
    I: int
    S: int
    K_orig: int
    K_base: int
    budget: int
    zipf_bias: bool = False      # per-expert gate bias 0.5 * rank^-1.1
    gate_scale: float = 1.0      # scalar folded into W_gate before bf16 rounding
    n_layers: int = 1
    seed: int = 0

    def with_(self, **kw) -> "MoEConfig":
        return dataclasses.replace(self, **kw)


# gate_scale of c5: bisection on mean top-1 softmax probability = 0.60 over the
# seeded inputs (found with the CPU oracle; a CPU test re-checks the 0.60).
C5_GATE_SCALE = 1.75

CONFIGS: Dict[str, MoEConfig] = {
    # tiny layer; K_orig=2 at half budget.  With K_base=1 this is the degenerate
    # pure Top-1 case, "c1k0" runs the same tensors with K_base=0.
    "c1": MoEConfig("c1", T=64, H=256, N=8, I=512, S=0, K_orig=2, K_base=1, budget=64),
    "c1k0": MoEConfig("c1k0", T=64, H=256, N=8, I=512, S=0, K_orig=2, K_base=0, budget=64),
    # DeepSeek-V2-Lite-shaped layer, decode: one token per sequence.
    "c2": MoEConfig("c2", T=64, H=2048, N=64, I=1408, S=2, K_orig=6, K_base=1, budget=192,
                    zipf_bias=True),
    # the same layer in prefill; budgets swept at {6, 4.5, 3, 2} x T.
    "c3": MoEConfig("c3", T=4096, H=2048, N=64, I=1408, S=2, K_orig=6, K_base=1, budget=3 * 4096,
                    zipf_bias=True),
    # stack of 26 such layers with per-layer budgets and a residual stream.
    "c4": MoEConfig("c4", T=2048, H=2048, N=64, I=1408, S=2, K_orig=6, K_base=1, budget=3 * 2048,
                    zipf_bias=True, n_layers=26),
    # one layer of that stack on its own (profiling case for the mid-size regime: 96 rows per expert on average)
    "c4l": MoEConfig("c4l", T=2048, H=2048, N=64, I=1408, S=2, K_orig=6, K_base=1, budget=3 * 2048, zipf_bias=True),
    # large-expert layer, prefill.
    "c5": MoEConfig("c5", T=8192, H=4096, N=8, I=14336, S=0, K_orig=2, K_base=1, budget=12288,
                    gate_scale=C5_GATE_SCALE),
    # the other two model rows of the paper's Table 1, prefill: Qwen1.5-MoE-shaped (60 routed experts, Top-4, budgets
    # 2-3.5 per token) and OLMoE-shaped (64 routed experts, Top-8, budgets 4-7).  The paper gives the expert counts
    # and Top-K only; hidden and intermediate sizes and the shared expert are synthetic choices.
    "qwen": MoEConfig("qwen", T=4096, H=2048, N=60, I=1408, S=1, K_orig=4, K_base=1, budget=int(2.5 * 4096)),
    # the batch shapes of the paper's own timing run (App. A.2: batch 8; decode = 8 tokens per step, prefill = 8
    # prompts of 32 tokens) on the DeepSeek-V2-Lite-shaped layer, at half budget
    "d8": MoEConfig("d8", T=8, H=2048, N=64, I=1408, S=2, K_orig=6, K_base=1, budget=24, zipf_bias=True),
    "p256": MoEConfig("p256", T=256, H=2048, N=64, I=1408, S=2, K_orig=6, K_base=1, budget=768, zipf_bias=True),
    "olmoe": MoEConfig("olmoe", T=4096, H=2048, N=64, I=1024, S=0, K_orig=8, K_base=1, budget=5 * 4096),
}

C3_BUDGET_MULTS = (6.0, 4.5, 3.0, 2.0)

# tensor ids inside one layer's stream
_ID_X, _ID_WG, _ID_W13, _ID_W2, _ID_WS13, _ID_WS2, _ID_BIAS, _ID_BUDGET = range(8)


def zipf_gate_bias(cfg: MoEConfig, layer: int = 0) -> torch.Tensor:
    """fp32 [N]: 0.5 * r_e^-1.1 with r a seeded permutation of 1..N (peak 0.5 on the hottest expert)."""
    perm = permutation(cfg.N, stream_key(cfg.seed, layer, _ID_BIAS))
    return torch.tensor([0.5 * float(perm[e] + 1) ** -1.1 for e in range(cfg.N)], dtype=torch.float32)


def make_layer(cfg: MoEConfig, layer: int = 0, device="cpu", with_x: bool = True) -> Dict[str, Optional[torch.Tensor]]:
    """All tensors of one layer: x~N(0,1), weights~N(0,0.02^2), bf16; bias fp32 or None.

    Layouts: x [T,H]; W_gate [H,N]; W13 [N,2I,H] (rows 0..I-1 the gate projection W1,
    rows I..2I-1 the up projection W3); W2 [N,H,I]; shared experts likewise with S.
    """
    k = lambda tid: stream_key(cfg.seed, layer, tid)
    d: Dict[str, Optional[torch.Tensor]] = {}
    d["x"] = normal_bf16((cfg.T, cfg.H), 1.0, k(_ID_X), device) if with_x else None
    d["W_gate"] = normal_bf16((cfg.H, cfg.N), 0.02 * cfg.gate_scale, k(_ID_WG), device)
    d["W13"] = normal_bf16((cfg.N, 2 * cfg.I, cfg.H), 0.02, k(_ID_W13), device)
    d["W2"] = normal_bf16((cfg.N, cfg.H, cfg.I), 0.02, k(_ID_W2), device)
    if cfg.S > 0:
        d["Wsh13"] = normal_bf16((cfg.S, 2 * cfg.I, cfg.H), 0.02, k(_ID_WS13), device)
        d["Wsh2"] = normal_bf16((cfg.S, cfg.H, cfg.I), 0.02, k(_ID_WS2), device)
    else:
        d["Wsh13"] = None
        d["Wsh2"] = None
    d["gate_bias"] = zipf_gate_bias(cfg, layer).to(device) if cfg.zipf_bias else None
    return d


def stack_budgets(cfg: MoEConfig, total_per_token: Optional[int] = None) -> List[int]:
    """Per-layer integer k_l for the layer stack: a Dirichlet(alpha=2) split of
    `total_per_token` (default 3 per layer), each k_l clamped to [1, K_orig], sum exact.

    Gamma(2) deviates are -ln(u1*u2); the shares are rounded by largest remainder,
    clamped, and the sum is repaired by moving single units to/from the layers with
    the largest rounding slack (ties by layer index), so the result is deterministic.
    """
    L = cfg.n_layers
    total = 3 * L if total_per_token is None else int(total_per_token)
    assert L <= total <= cfg.K_orig * L
    u = uniform01(2 * L, stream_key(cfg.seed, 0, _ID_BUDGET))
    g = [-math.log(u[2 * i] * u[2 * i + 1]) for i in range(L)]
    sg = sum(g)
    share = [total * gi / sg for gi in g]
    k = [min(cfg.K_orig, max(1, int(math.floor(s)))) for s in share]
    while sum(k) != total:
        if sum(k) < total:
            cand = [i for i in range(L) if k[i] < cfg.K_orig]
            i = max(cand, key=lambda i: (share[i] - k[i], -i))
            k[i] += 1
        else:
            cand = [i for i in range(L) if k[i] > 1]
            i = min(cand, key=lambda i: (share[i] - k[i], i))
            k[i] -= 1
    return k


def score_rows(T: int, K_orig: int, key: int, ties: bool = False) -> torch.Tensor:
    """fp32 [T,K_orig] positive rows sorted descending: stand-in routing scores for
    selection-only tests.  With ties=True values are drawn from a 12-level grid so
    equal keys are common (tie-break coverage)."""
    idx = torch.arange(T * K_orig, dtype=torch.int64)
    s = _irwin_hall_int(key, idx).reshape(T, K_orig)
    if ties:
        v = ((s % 12) + 1).to(torch.float32) / 64.0
    else:
        v = (s.to(torch.float32) + 1.0) / float(12 * 65535 + 2)
    return torch.sort(v, dim=1, descending=True).values.contiguous()


def sensitivity_matrix(cfg: MoEConfig) -> List[List[float]]:
    """A seeded stand-in for Alloc-L's profiled matrix S [L, K_orig] (the real one needs a trained model and a
    calibration set): row i falls from a layer-specific level a_i at k = 1 to 0 at k = K_orig along (1 - (k-1)/(K-1))
    to a layer-specific power in [1, 3], with a_i in [0.5, 1.5] larger for earlier layers on average, as the paper
    reports for its profiles (earlier layers are more sensitive)."""
    L, K = cfg.n_layers, cfg.K_orig
    u = uniform01(2 * L, stream_key(cfg.seed, 0, _ID_BUDGET + 1))
    rows = []
    for i in range(L):
        a = 0.5 + (1.0 - i / max(L - 1, 1)) * 0.6 + 0.4 * u[2 * i]
        pw = 1.0 + 2.0 * u[2 * i + 1]
        rows.append([a * (1.0 - (k - 1) / max(K - 1, 1)) ** pw for k in range(1, K + 1)])
    return rows

