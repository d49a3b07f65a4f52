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
                selection is local again and runs as ONE library call
                (`moe_layer_forward_routed`), which takes the kept counts from device memory: the
                host never learns this rank's share of the budget and never waits for the device.

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


def gather_score_rows(topk_score_local: torch.Tensor, group=None, out: Optional[torch.Tensor] = None,
                      always: bool = False) -> torch.Tensor:
    """[T, K] rows of every rank, stacked in rank order -> [W*T, K] (the flat index t*K + j of the
    tie rule then orders tokens by rank first, a fixed order every rank agrees on).  With one rank
    the input is returned as it is unless `always` asks for the collective to run all the same."""
    _, w = world(group)
    if w == 1 and not (always and dist.is_available() and dist.is_initialized()):
        return topk_score_local
    T, K = topk_score_local.shape
    pool = out if out is not None else torch.empty(w * T, K, dtype=topk_score_local.dtype,
                                                   device=topk_score_local.device)
    dist.all_gather_into_tensor(pool, topk_score_local.contiguous(), group=group)
    return pool


def select_with_library(pool: torch.Tensor, K_base: int, budget: int, n_sel: Optional[torch.Tensor] = None,
                        dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The library's Alloc-T kernel on a [T_pool, K] pool; errors go to `dev_status` (device), nothing is read back."""
    Tt, K = pool.shape
    shape = B.make_shape(Tt, 64, 8, 64, 0, K, K_base)     # the selection reads only T, K_orig, K_base
    if n_sel is None:
        n_sel = torch.empty(Tt, dtype=torch.int32, device=pool.device)
    if dev_status is None:
        dev_status = torch.zeros(1, dtype=torch.int32, device=pool.device)
    B.alloc_t_select(shape, pool, budget, n_sel, dev_status, None)
    return n_sel


def alloc_t_select_global(topk_score_local: torch.Tensor, K_base: int, budget_global: int, group=None,
                          select: Optional[Callable[[torch.Tensor, int, int], torch.Tensor]] = None
                          ) -> Tuple[torch.Tensor, torch.Tensor]:
    """Alloc-T over the tokens of all ranks.  `budget_global` is the total activation count of the whole
    batch (W*T*K_l).  Returns this rank's n_sel [T] and, as a 0-dim tensor on the same device (not
    read back here), the number of activations it was given.
    `select(pool, K_base, budget) -> n_sel` defaults to the library's kernel; it exists so that the
    exchange can be exercised where no GPU is present."""
    rank, w = world(group)
    T = topk_score_local.shape[0]
    pool = gather_score_rows(topk_score_local, group)
    n_all = (select or select_with_library)(pool, K_base, int(budget_global))
    mine = n_all[rank * T:(rank + 1) * T]
    return mine, mine.sum()


def local_budget_bound(shape: B.MoeShape, budget_global: int, w: int) -> int:
    """The most pairs one rank can be given: every other rank keeps at least K_base per token."""
    return max(0, min(shape.K_orig * shape.T, int(budget_global) - shape.K_base * shape.T * (w - 1)))


class GlobalAllocTLayer:
    """The layer with the batch-wide Alloc-T on one rank of a token-data-parallel group: gate ->
    all-gather of the score rows -> selection over the whole pool -> permutation, experts and combine
    on this rank's tokens.  All buffers are allocated once here; `forward` only enqueues work (four
    library calls and one collective) and never synchronises with the device."""

    def __init__(self, shape: B.MoeShape, device, group=None, always_collective: bool = False):
        self.shape, self.group, self.always = shape, group, always_collective
        self.rank, self.w = world(group)
        T, K = shape.T, shape.K_orig
        self.topk_idx = torch.empty(T, K, dtype=torch.int32, device=device)
        self.topk_score = torch.empty(T, K, dtype=torch.float32, device=device)
        self.pool = torch.empty(self.w * T, K, dtype=torch.float32, device=device)
        self.n_all = torch.empty(self.w * T, dtype=torch.int32, device=device)
        self.ws = B.new_workspace(shape, shape.K_orig * shape.T, device=device)

    def route(self, x, W_gate, gate_bias, budget_global: int, dev_status: torch.Tensor) -> torch.Tensor:
        """Gate, exchange and selection; returns this rank's n_sel [T] (a view, on the device)."""
        s = self.shape
        B.moe_gate(s, x, W_gate, gate_bias, None, self.topk_idx, self.topk_score)
        pool = gather_score_rows(self.topk_score, self.group, out=self.pool, always=self.always)
        select_with_library(pool, s.K_base, int(budget_global), self.n_all, dev_status)
        return self.n_all[self.rank * s.T:(self.rank + 1) * s.T]

    def forward(self, x, W_gate, gate_bias, W13, W2, Wsh13, Wsh2, budget_global: int, out: torch.Tensor,
                dev_status: torch.Tensor, residual: Optional[torch.Tensor] = None) -> None:
        s = self.shape
        n_sel = self.route(x, W_gate, gate_bias, budget_global, dev_status)
        B.moe_layer_forward_routed(s, x, self.topk_idx, self.topk_score, n_sel,
                                   local_budget_bound(s, budget_global, self.w), int(budget_global) // self.w,
                                   W13, W2, Wsh13, Wsh2, out, dev_status, self.ws, residual=residual)


def moe_layer_forward_global(shape: B.MoeShape, x, W_gate, gate_bias, W13, W2, Wsh13, Wsh2, budget_global: int,
                             out: torch.Tensor, dev_status: torch.Tensor, group=None) -> None:
    """One-off form of GlobalAllocTLayer.forward (allocates its buffers on every call)."""
    GlobalAllocTLayer(shape, x.device, group).forward(x, W_gate, gate_bias, W13, W2, Wsh13, Wsh2, budget_global, out,
                                                      dev_status)
