"""Off-line calibration of the token-level comparison rules (paper App. A.1: their thresholds are profiled so that
the resulting expert activations meet the target budget).  Host-side bisection only: the counting itself is the
library's kernel (or, in CPU tests, any callable with the same contract)."""
from __future__ import annotations

import struct
from typing import Callable, Tuple


def _f32(v: float) -> float:
    return struct.unpack("f", struct.pack("f", v))[0]


def calibrate(select: Callable[[object, float], Tuple[object, int]], scores, budget: int, increasing: bool,
              lo: float, hi: float) -> Tuple[float, int]:
    """The fp32 threshold whose kept total is the largest one not above `budget`.
    select(scores, threshold) -> (n_sel, total).  increasing: the total grows with the threshold (Top-P); otherwise it
    falls (relative skipping).  The total at one end of [lo, hi] must be within the budget.  Bisection over fp32
    values until the bracket closes, so the answer is exact, not approximate."""
    lo, hi = _f32(lo), _f32(hi)
    ok, bad = (lo, hi) if increasing else (hi, lo)      # `ok` keeps the total within the budget
    n_ok = select(scores, ok)[1]
    if n_ok > budget:
        raise ValueError("no threshold in the bracket meets the budget")
    if select(scores, bad)[1] <= budget:
        return bad, select(scores, bad)[1]
    while True:
        mid = _f32(0.5 * (ok + bad))
        if mid == ok or mid == bad:
            return ok, n_ok
        tot = select(scores, mid)[1]
        if tot <= budget:
            ok, n_ok = mid, tot
        else:
            bad = mid


def library_selector(rule: str, shape, dev_status):
    """select(scores, threshold) backed by the library's kernels; reads the kept total back (an off-line step)."""
    import torch
    from . import binding as B
    fn = B.moe_select_top_p if rule == "top_p" else B.moe_select_rel_threshold
    n_sel = torch.empty(shape.T, dtype=torch.int32, device="cuda")
    total = torch.zeros(1, dtype=torch.int32, device="cuda")

    def select(scores, thr):
        total.zero_()
        fn(shape, scores, thr, n_sel, total, dev_status)
        return n_sel, int(total.item())
    return select
