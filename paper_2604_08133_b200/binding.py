"""ctypes binding of liballocmoe.so: the same names as include/allocmoe.h, argument
marshalling only.  torch supplies device memory and streams; every step of the path runs in
the library's kernels.  There is no fallback: a missing library is an error."""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# ALLOCMOE_LIB selects another build of the same library (the checked build, see build.py)
LIB_PATH = os.environ.get("ALLOCMOE_LIB") or os.path.join(_PKG, "liballocmoe.so")

MOE_OK, MOE_ERR_ARG, MOE_ERR_BUDGET, MOE_ERR_WORKSPACE, MOE_ERR_CUDA, MOE_ERR_NONFINITE, MOE_ERR_TIMEOUT = range(7)

EXPORTS = ("moe_status_string", "moe_workspace_bytes", "moe_gate", "alloc_t_select", "moe_permute",
           "moe_grouped_ffn", "moe_shared_ffn", "moe_combine", "moe_layer_forward", "moe_layer_intermediates",
           "moe_rmsnorm", "moe_profile_enable", "moe_profile_read", "moe_permute_static", "moe_route", "alloc_l_solve",
           "moe_layer_forward_routed", "moe_selftest_wait_timeout", "moe_select_top_p", "moe_select_rel_threshold")
PROFILE_STAGES = ("gate", "route", "gather", "ffn_gemm1", "ffn_gemm2", "combine")


class MoeShape(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32), ("I", ctypes.c_int32),
                ("S", ctypes.c_int32), ("K_orig", ctypes.c_int32), ("K_base", ctypes.c_int32),
                ("flags", ctypes.c_uint32)]


class MoeError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn}: {status_string(status)} (status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the C-ABI library (built by `python -m paper_2604_08133_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_08133_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
        sp = ctypes.POINTER(MoeShape)
        L.moe_status_string.restype = ctypes.c_char_p
        L.moe_status_string.argtypes = [ctypes.c_int]
        L.moe_workspace_bytes.restype = sz
        L.moe_workspace_bytes.argtypes = [sp, i64]
        sigs = {
            "moe_gate": [sp, vp, vp, vp, vp, vp, vp, vp],
            "alloc_t_select": [sp, vp, i64, vp, vp, vp, sz, vp],
            "moe_permute": [sp, vp, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, sz, vp],
            "moe_permute_static": [sp, vp, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp],
            "moe_route": [sp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp],
            "moe_grouped_ffn": [sp, vp, vp, vp, i64, vp, vp, vp, vp, vp, sz, vp],
            "moe_layer_forward_routed": [sp, vp, vp, vp, vp, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp],
            "moe_selftest_wait_timeout": [sp, vp, i64, vp, vp, i64, vp, vp, sz, vp],
            "moe_select_top_p": [sp, vp, ctypes.c_float, vp, vp, vp, vp],
            "moe_select_rel_threshold": [sp, vp, ctypes.c_float, vp, vp, vp, vp],
            "moe_shared_ffn": [sp, vp, vp, vp, vp, vp, vp, sz, vp],
            "moe_combine": [sp, vp, vp, vp, vp, vp, vp, vp],
            "moe_layer_forward": [sp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, vp, vp, sz, vp],
            "moe_rmsnorm": [sp, vp, vp, vp],
            "moe_layer_intermediates": [sp, i64, vp, sz] + [ctypes.POINTER(vp)] * 7,
            "moe_profile_enable": [ctypes.c_int32],
            "moe_profile_read": [ctypes.POINTER(ctypes.c_float)],
        }
        L.alloc_l_solve.restype = ctypes.c_int
        L.alloc_l_solve.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.c_int32, ctypes.c_int32, i64,
                                    ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_double)]
        for name, argtypes in sigs.items():
            fn = getattr(L, name)
            fn.restype = ctypes.c_int
            fn.argtypes = argtypes
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().moe_status_string(int(status)).decode()


def make_shape(T, H, N, I, S, K_orig, K_base) -> MoeShape:
    return MoeShape(int(T), int(H), int(N), int(I), int(S), int(K_orig), int(K_base), 0)


def shape_of(cfg) -> MoeShape:
    return make_shape(cfg.T, cfg.H, cfg.N, cfg.I, cfg.S, cfg.K_orig, cfg.K_base)


def _p(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_contiguous()
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(fn: str, st: int):
    if st != MOE_OK:
        raise MoeError(fn, st)


def moe_workspace_bytes(shape: MoeShape, budget_max: int) -> int:
    return int(lib().moe_workspace_bytes(ctypes.byref(shape), int(budget_max)))


def new_workspace(shape: MoeShape, budget_max: int, device="cuda") -> torch.Tensor:
    n = moe_workspace_bytes(shape, budget_max)
    if n == 0:
        raise MoeError("moe_workspace_bytes", MOE_ERR_ARG)
    return torch.empty(n, dtype=torch.uint8, device=device)


def moe_gate(shape, x, W_gate, gate_bias, scores, topk_idx, topk_score, stream=None):
    _check("moe_gate", lib().moe_gate(ctypes.byref(shape), _p(x), _p(W_gate), _p(gate_bias), _p(scores),
                                      _p(topk_idx), _p(topk_score), _stream(stream)))


def alloc_t_select(shape, topk_score, budget, n_sel, dev_status, ws, stream=None):
    _check("alloc_t_select", lib().alloc_t_select(ctypes.byref(shape), _p(topk_score), int(budget), _p(n_sel),
                                                  _p(dev_status), _p(ws), ws.numel() if ws is not None else 0,
                                                  _stream(stream)))


def moe_permute(shape, x, topk_idx, topk_score, n_sel, budget, expert_offsets, perm_token, perm_weight, pair_pos,
                x_perm, dev_status, ws, stream=None):
    _check("moe_permute", lib().moe_permute(ctypes.byref(shape), _p(x), _p(topk_idx), _p(topk_score), _p(n_sel),
                                            int(budget), _p(expert_offsets), _p(perm_token), _p(perm_weight),
                                            _p(pair_pos), _p(x_perm), _p(dev_status), _p(ws), ws.numel(),
                                            _stream(stream)))


def alloc_l_solve(S, B: int):
    """Alloc-L (Eq. 3-6): the optimal per-layer K for a sensitivity matrix S [L, K_orig] (any array-like of floats)
    under the global budget B.  Returns (list of K_i, total cost).  Host only."""
    rows = [[float(v) for v in r] for r in S]
    Lr, K = len(rows), len(rows[0])
    flat = (ctypes.c_double * (Lr * K))(*[v for r in rows for v in r])
    out = (ctypes.c_int32 * Lr)()
    cost = ctypes.c_double(0.0)
    _check("alloc_l_solve", lib().alloc_l_solve(flat, Lr, K, int(B), out, ctypes.byref(cost)))
    return list(out), float(cost.value)


def moe_route(shape, topk_idx, topk_score, budget, n_sel, expert_offsets, perm_token, perm_weight, pair_pos, dev_status,
              stream=None):
    """alloc_t_select + the list-building part of moe_permute in one launch (T <= 8192)."""
    _check("moe_route", lib().moe_route(ctypes.byref(shape), _p(topk_idx), _p(topk_score), int(budget), _p(n_sel),
                                        _p(expert_offsets), _p(perm_token), _p(perm_weight), _p(pair_pos),
                                        _p(dev_status), _stream(stream)))


def moe_permute_static(shape, x, topk_idx, topk_score, n_sel, budget, expert_offsets, perm_token, perm_weight, pair_pos,
                       x_perm, dev_status, stream=None):
    """moe_permute without a workspace argument, for callers that cannot allocate device memory:
    the scratch is a fixed array inside the library (N * ceil(T/32) <= 65536)."""
    _check("moe_permute_static", lib().moe_permute_static(ctypes.byref(shape), _p(x), _p(topk_idx), _p(topk_score),
                                                          _p(n_sel), int(budget), _p(expert_offsets), _p(perm_token),
                                                          _p(perm_weight), _p(pair_pos), _p(x_perm), _p(dev_status),
                                                          _stream(stream)))


def moe_grouped_ffn(shape, x_or_xperm, perm_token, expert_offsets, budget, W13, W2, y_perm, dev_status, ws, stream=None):
    """perm_token None: x_or_xperm is x_perm [budget,H]; else it is x [T,H] and row p is x[perm_token[p]]."""
    _check("moe_grouped_ffn", lib().moe_grouped_ffn(ctypes.byref(shape), _p(x_or_xperm), _p(perm_token),
                                                    _p(expert_offsets), int(budget), _p(W13), _p(W2), _p(y_perm),
                                                    _p(dev_status), _p(ws), ws.numel(), _stream(stream)))


def moe_shared_ffn(shape, x, Wsh13, Wsh2, y_shared, dev_status, ws, stream=None):
    _check("moe_shared_ffn", lib().moe_shared_ffn(ctypes.byref(shape), _p(x), _p(Wsh13), _p(Wsh2), _p(y_shared),
                                                  _p(dev_status), _p(ws), ws.numel(), _stream(stream)))


def moe_combine(shape, y_perm, pair_pos, topk_score, n_sel, y_shared, out, stream=None):
    _check("moe_combine", lib().moe_combine(ctypes.byref(shape), _p(y_perm), _p(pair_pos), _p(topk_score), _p(n_sel),
                                            _p(y_shared), _p(out), _stream(stream)))


def moe_layer_forward(shape, x, W_gate, gate_bias, W13, W2, Wsh13, Wsh2, budget, out, dev_status, ws,
                      residual: Optional[torch.Tensor] = None, stream=None):
    _check("moe_layer_forward", lib().moe_layer_forward(ctypes.byref(shape), _p(x), _p(W_gate), _p(gate_bias), _p(W13),
                                                        _p(W2), _p(Wsh13), _p(Wsh2), int(budget), _p(residual),
                                                        _p(out), _p(dev_status), _p(ws), ws.numel(), _stream(stream)))


def moe_layer_forward_routed(shape, x, topk_idx, topk_score, n_sel, budget_max, budget_hint, W13, W2, Wsh13, Wsh2, out,
                             dev_status, ws, residual: Optional[torch.Tensor] = None, stream=None):
    """Permutation, experts and combine for a selection the caller holds (n_sel on the device)."""
    _check("moe_layer_forward_routed",
           lib().moe_layer_forward_routed(ctypes.byref(shape), _p(x), _p(topk_idx), _p(topk_score), _p(n_sel),
                                          int(budget_max), int(budget_hint), _p(W13), _p(W2), _p(Wsh13), _p(Wsh2),
                                          _p(residual), _p(out), _p(dev_status), _p(ws), ws.numel(), _stream(stream)))


def moe_selftest_wait_timeout(shape, expert_offsets, budget, W2, y_perm, wait_limit_clk, dev_status, ws, stream=None):
    """Launches expert GEMM-2 alone with a short wait limit: its bounded waits run out (see the header)."""
    _check("moe_selftest_wait_timeout",
           lib().moe_selftest_wait_timeout(ctypes.byref(shape), _p(expert_offsets), int(budget), _p(W2), _p(y_perm),
                                           int(wait_limit_clk), _p(dev_status), _p(ws), ws.numel(), _stream(stream)))


def moe_select_top_p(shape, topk_score, P, n_sel, total, dev_status, stream=None):
    """Top-P count per token (the Dynamic-MoE baseline); `total` (device int32 [1] or None) accumulates sum n_sel."""
    _check("moe_select_top_p", lib().moe_select_top_p(ctypes.byref(shape), _p(topk_score), float(P), _p(n_sel),
                                                      _p(total), _p(dev_status), _stream(stream)))


def moe_select_rel_threshold(shape, topk_score, beta, n_sel, total, dev_status, stream=None):
    """Skipping relative to the top-1 score (the NAEE baseline extended to Top-K)."""
    _check("moe_select_rel_threshold",
           lib().moe_select_rel_threshold(ctypes.byref(shape), _p(topk_score), float(beta), _p(n_sel), _p(total),
                                          _p(dev_status), _stream(stream)))


def moe_rmsnorm(shape, x, out, stream=None):
    _check("moe_rmsnorm", lib().moe_rmsnorm(ctypes.byref(shape), _p(x), _p(out), _stream(stream)))


def moe_layer_intermediates(shape, budget, ws) -> Dict[str, torch.Tensor]:
    """Views (copies to fresh tensors) of the routing intermediates a forward call left in `ws`."""
    ptrs = [ctypes.c_void_p() for _ in range(7)]
    _check("moe_layer_intermediates",
           lib().moe_layer_intermediates(ctypes.byref(shape), int(budget), _p(ws), ws.numel(),
                                         *[ctypes.byref(p) for p in ptrs]))
    base = ws.data_ptr()
    T, K, N, H, B = shape.T, shape.K_orig, shape.N, shape.H, int(budget)

    def view(ptr, nbytes, dtype, dims):
        off = ptr.value - base
        return ws[off:off + nbytes].view(dtype).reshape(*dims).clone()
    return dict(
        topk_idx=view(ptrs[0], T * K * 4, torch.int32, (T, K)),
        topk_score=view(ptrs[1], T * K * 4, torch.float32, (T, K)),
        n_sel=view(ptrs[2], T * 4, torch.int32, (T,)),
        expert_offsets=view(ptrs[3], (N + 1) * 4, torch.int32, (N + 1,)),
        perm_token=view(ptrs[4], B * 4, torch.int32, (B,)),
        pair_pos=view(ptrs[5], T * K * 4, torch.int32, (T, K)),
        y_perm=view(ptrs[6], B * H * 2, torch.bfloat16, (B, H)),
    )


def moe_profile_enable(on: bool):
    _check("moe_profile_enable", lib().moe_profile_enable(int(bool(on))))


def moe_profile_read() -> Dict[str, float]:
    """Device milliseconds of the six stages of the last moe_layer_forward call."""
    buf = (ctypes.c_float * len(PROFILE_STAGES))()
    _check("moe_profile_read", lib().moe_profile_read(buf))
    return {k: float(buf[i]) for i, k in enumerate(PROFILE_STAGES)}
