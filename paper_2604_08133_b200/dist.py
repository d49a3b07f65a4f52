"""Token-data-parallel use of the layer: every rank holds T tokens and the full weights.

Two modes.
  independent   each rank spends its own budget on its own tokens (no exchange at all): the layer
                call is `binding.moe_layer_forward` as it stands; `max_over_ranks` is the only
                collective, used for timing.
  global        Alloc-T as the paper states it pools the residual scores of ALL tokens of the
                batch (Sec. 3.3).  When the batch is sharded over ranks that needs one exchange: an
                all-gather of the [T, K_orig] score rows (80 KB in total at 4096 tokens), after
                which every rank runs the identical selection over the whole pool with the
                library's own kernel and keeps its slice of n_sel.  Everything after the
                selection is local again.

PyTorch is used for the process group and device memory only; every step of the layer runs in
the library's kernels.
"""
from __future__ import annotations

from typing import Callable, Optional, Tuple

import torch
import torch.distributed as dist

from . import binding as B


def world(group=None) -> Tuple[int, int]:
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(group), dist.get_world_size(group)
    return 0, 1


def max_over_ranks(value: float, device="cpu", group=None) -> float:
    """The slowest rank's value (a duration measured on each rank's own device)."""
    _, w = world(group)
    if w == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def gather_score_rows(topk_score_local: torch.Tensor, group=None) -> torch.Tensor:
    """[T, K] rows of every rank, stacked in rank order -> [W*T, K] (the flat index t*K + j of the
    tie rule then orders tokens by rank first, a fixed order every rank agrees on)."""
    _, w = world(group)
    if w == 1:
        return topk_score_local
    T, K = topk_score_local.shape
    pool = torch.empty(w * T, K, dtype=topk_score_local.dtype, device=topk_score_local.device)
    dist.all_gather_into_tensor(pool, topk_score_local.contiguous(), group=group)
    return pool


def _select_with_library(pool: torch.Tensor, K_base: int, budget: int) -> torch.Tensor:
    Tt, K = pool.shape
    shape = B.make_shape(Tt, 64, 8, 64, 0, K, K_base)     # the selection reads only T, K_orig, K_base
    n_sel = torch.empty(Tt, dtype=torch.int32, device=pool.device)
    status = torch.zeros(1, dtype=torch.int32, device=pool.device)
    B.alloc_t_select(shape, pool, budget, n_sel, status, None)
    if int(status.item()) != 0:
        raise B.MoeError("alloc_t_select", B.MOE_ERR_NONFINITE)
    return n_sel


def alloc_t_select_global(topk_score_local: torch.Tensor, K_base: int, budget_global: int, group=None,
                          select: Optional[Callable[[torch.Tensor, int, int], torch.Tensor]] = None
                          ) -> Tuple[torch.Tensor, int]:
    """Alloc-T over the tokens of all ranks.  `budget_global` is the total activation count of the whole
    batch (W*T*K_l).  Returns this rank's n_sel [T] and the number of activations it was given.
    `select(pool, K_base, budget) -> n_sel` defaults to the library's kernel; it exists so that the
    exchange can be exercised where no GPU is present."""
    rank, w = world(group)
    T = topk_score_local.shape[0]
    pool = gather_score_rows(topk_score_local, group)
    n_all = (select or _select_with_library)(pool, K_base, int(budget_global))
    mine = n_all[rank * T:(rank + 1) * T].contiguous()
    return mine, int(mine.sum().item())


def moe_layer_forward_global(shape: B.MoeShape, x, W_gate, gate_bias, W13, W2, Wsh13, Wsh2, budget_global: int,
                             out: torch.Tensor, dev_status: torch.Tensor, group=None) -> int:
    """The layer with the batch-wide Alloc-T: gate, exchange + selection, then permutation, experts and
    combine on this rank's tokens.  Returns this rank's activation count."""
    T, H, K = shape.T, shape.H, shape.K_orig
    dev = x.device
    topk_idx = torch.empty(T, K, dtype=torch.int32, device=dev)
    topk_score = torch.empty(T, K, dtype=torch.float32, device=dev)
    B.moe_gate(shape, x, W_gate, gate_bias, None, topk_idx, topk_score)
    n_sel, b_local = alloc_t_select_global(topk_score, shape.K_base, budget_global, group)
    # this rank's share may fall below K_base*T only if K_base is not guaranteed, never above K_orig*T
    ws = B.new_workspace(shape, max(b_local, shape.K_base * T), device=dev)
    off = torch.empty(shape.N + 1, dtype=torch.int32, device=dev)
    tok = torch.empty(max(b_local, 1), dtype=torch.int32, device=dev)
    wgt = torch.empty(max(b_local, 1), dtype=torch.float32, device=dev)
    pos = torch.empty(T, K, dtype=torch.int32, device=dev)
    x_perm = torch.empty(max(b_local, 1), H, dtype=torch.bfloat16, device=dev)
    y_perm = torch.empty(max(b_local, 1), H, dtype=torch.bfloat16, device=dev)
    B.moe_permute(shape, x, topk_idx, topk_score, n_sel, b_local, off, tok, wgt, pos, x_perm, dev_status, ws)
    if b_local > 0:
        B.moe_grouped_ffn(shape, x_perm, off, b_local, W13, W2, y_perm, dev_status, ws)
    y_shared = None
    if shape.S > 0:
        y_shared = torch.empty(T, H, dtype=torch.bfloat16, device=dev)
        B.moe_shared_ffn(shape, x, Wsh13, Wsh2, y_shared, dev_status, ws)
    B.moe_combine(shape, y_perm, pos, topk_score, n_sel, y_shared, out)
    return b_local
