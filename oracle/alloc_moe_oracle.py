"""CPU oracle for the budget-constrained MoE layer forward (Alloc-MoE).

TEST INFRASTRUCTURE ONLY.  Plain, slow, numpy/fp64; written from the paper's
definitions; shares no code with the CUDA path and is imported only by tests,
the smoke check and the benchmark's CPU-baseline leg.  The product path never
calls it.

Passages followed
  Eq. 1 (Sec. 3.1)   w_t = Top-K(Softmax(x_t W_gate))            -> gate_logits, softmax_scores, topk_sorted
  Eq. 2 (Sec. 3.1)   y_t = sum_i w_{t,i} E_i(x_t), w=0 if inactive -> combine, layer_forward_dense
  Sec. 3.1 "Expert Activation Budget": a layer's total budget T*K_l may be
                     redistributed across tokens                  -> `budget` is that total
  Eq. 7-10 (Sec. 3.3) Alloc-T as a 0/1 programme                  -> alloc_t_bruteforce
  Sec. 3.3, procedure paragraph: keep Top-K_base per token, pool the other
                     K_orig-K_base scores of all tokens, take the global top
                     (K_l-K_base)*T                               -> alloc_t_select, alloc_t_select_threshold
  Sec. 3.3, last paragraph: K_base = K_l is plain Top-K routing   -> covered by tests
  Eq. 3-6 (Sec. 3.2) Alloc-L grouped-knapsack DP                  -> alloc_l_dp, alloc_l_bruteforce
  Sec. 2 / App. A.1  the token-level rules Alloc-T is compared with: Top-P count
                     (Dynamic-MoE) and skipping relative to the top-1 score (NAEE
                     extended to Top-K)                            -> top_p_count, rel_threshold_count

Readings where the paper is silent or inconsistent (each is listed in the design notes):
  * the candidate set holds each token's Top-K_orig pairs (the procedure paragraph's
    [T, K_orig] score tensor), not Top-K_l as the set's printed size suggests;
  * ties: per token the lower expert id ranks first; in the pool the lower flat
    index t*K_orig + j ranks first;
  * kept weights are the softmax probabilities over all N experts, not renormalised;
  * the expert network is SwiGLU: E(x) = W2 (silu(W1 x) * (W3 x)); shared experts
    run for every token with weight 1 outside the budget; an optional per-expert
    bias is added to the gate logits before the softmax.  (Workload parameters,
    not in the paper.)

Parity pins: every function here is pinned by tests/test_oracle_*.py (brute force on
tiny inputs, invariants, degenerate cases, library cross-checks, hand-worked
fixtures under tests/golden/).  The paper's accuracy tables are out of scope.
"""
from __future__ import annotations

import itertools
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------- Eq. 1
def gate_logits(x, W_gate, gate_bias=None) -> np.ndarray:
    """logits[t,e] = sum_h x[t,h] W_gate[h,e] (+ bias[e]); fp64.  Eq. 1's x_t . W_gate."""
    z = np.asarray(x, F64) @ np.asarray(W_gate, F64)
    if gate_bias is not None:
        z = z + np.asarray(gate_bias, F64)[None, :]
    return z


def softmax_scores(logits) -> np.ndarray:
    """Row softmax over ALL N experts (Eq. 1 applies Top-K to the softmax output),
    max-subtracted, fp64, rounded once to fp32: the routing-score tensor."""
    z = np.asarray(logits, F64)
    z = z - z.max(axis=1, keepdims=True)
    e = np.exp(z)
    return (e / e.sum(axis=1, keepdims=True)).astype(np.float32)


def topk_sorted(scores, K_orig: int) -> Tuple[np.ndarray, np.ndarray]:
    """Per token the K_orig largest scores, rows descending (the order Sec. 3.3's
    procedure assumes); equal scores rank the lower expert id first.
    Returns (topk_idx int32 [T,K_orig], topk_score fp32 [T,K_orig])."""
    s = np.asarray(scores, np.float32)
    T, N = s.shape
    idx = np.empty((T, K_orig), np.int32)
    val = np.empty((T, K_orig), np.float32)
    for t in range(T):
        order = sorted(range(N), key=lambda e: (-float(s[t, e]), e))[:K_orig]
        idx[t] = order
        val[t] = s[t, order]
    return idx, val


# ----------------------------------------------------------------------------- Alloc-T
def _check_budget(T: int, K_orig: int, K_base: int, budget: int) -> int:
    if not (0 <= K_base <= K_orig):
        raise ValueError("K_base must lie in [0, K_orig]")
    if not (K_base * T <= budget <= K_orig * T):
        raise ValueError("budget must lie in [K_base*T, K_orig*T]")
    return budget - K_base * T


def alloc_t_select(topk_score, K_base: int, budget: int) -> np.ndarray:
    """Alloc-T, the procedure of Sec. 3.3: columns j < K_base of every token are kept;
    the other T*(K_orig-K_base) scores are pooled and the R = budget - K_base*T largest
    are kept (ties: lower flat index t*K_orig+j first).  Returns the 0/1 matrix z [T,K_orig]."""
    s = np.asarray(topk_score, np.float32)
    T, K = s.shape
    R = _check_budget(T, K, K_base, budget)
    z = np.zeros((T, K), np.int8)
    z[:, :K_base] = 1
    pool = [(t, j) for t in range(T) for j in range(K_base, K)]
    pool.sort(key=lambda tj: (-float(s[tj]), tj[0] * K + tj[1]))
    for (t, j) in pool[:R]:
        z[t, j] = 1
    return z


def alloc_t_select_threshold(topk_score, K_base: int, budget: int) -> np.ndarray:
    """Second, independent form of the same procedure: find the value tau of the R-th
    largest pooled score with a partial sort, keep everything above tau, then fill
    the remaining places with scores equal to tau in ascending flat index."""
    s = np.asarray(topk_score, np.float32)
    T, K = s.shape
    R = _check_budget(T, K, K_base, budget)
    z = np.zeros((T, K), np.int8)
    z[:, :K_base] = 1
    if R == 0:
        return z
    resid = s[:, K_base:]
    flat = resid.reshape(-1)
    tau = np.partition(flat, flat.size - R)[flat.size - R]
    above = resid > tau
    z[:, K_base:][above] = 1
    need = R - int(above.sum())
    tj = np.argwhere(resid == tau)                  # row-major = ascending flat index
    for (t, j) in tj[:need]:
        z[t, K_base + j] = 1
    return z


def n_sel_from_mask(z) -> np.ndarray:
    """n_t = number of kept pairs of token t.  Valid as an encoding of z because rows
    are sorted descending and ties prefer the lower column, so a token's kept pairs
    are its first n_t columns (checked here)."""
    z = np.asarray(z)
    n = z.sum(axis=1).astype(np.int32)
    K = z.shape[1]
    prefix = (np.arange(K)[None, :] < n[:, None]).astype(z.dtype)
    if not np.array_equal(prefix, z):
        raise AssertionError("kept pairs of a token are not a prefix of its sorted row")
    return n


def alloc_t_objective(topk_score, z) -> float:
    """Eq. 8: sum of z * w, fp64."""
    return float((np.asarray(topk_score, F64) * np.asarray(z, F64)).sum())


def alloc_t_bruteforce(topk_score, K_base: int, budget: int):
    """Eq. 8-10 by exhaustive enumeration (tiny inputs only): maximise sum z*w subject to
    sum z <= budget and sum_e z[t,e] >= K_base for every t.  Returns (best objective,
    list of all maximising z matrices)."""
    s = np.asarray(topk_score, F64)
    T, K = s.shape
    n = T * K
    if n > 16:
        raise ValueError("brute force is for T*K_orig <= 16")
    w = s.reshape(-1)
    # every 0/1 assignment at once: row b of `allz` is the bit pattern of b
    allz = ((np.arange(1 << n, dtype=np.int64)[:, None] >> np.arange(n)[None, :]) & 1).astype(np.int8)
    feasible = allz.sum(axis=1) <= budget
    feasible &= (allz.reshape(-1, T, K).sum(axis=2) >= K_base).all(axis=1)
    obj = allz.astype(F64) @ w
    obj[~feasible] = -1.0
    best = float(obj.max())
    arg = [allz[b].reshape(T, K).copy() for b in np.flatnonzero(np.abs(obj - best) <= 1e-15)]
    return best, arg


# ----------------------------------------------------------------------------- token-level comparison rules
def top_p_count(topk_score, P: float) -> np.ndarray:
    """Top-P routing (Sec. 2; the Dynamic-MoE setting of App. A.1): a token activates experts in
    descending score order until their cumulative score reaches P.  n_t = the smallest n >= 1 with
    s[t,0] + ... + s[t,n-1] >= P, K_orig if the row never gets there.  The running sum and the
    comparison are fp32, columns in order: the decision is an integer, so it is taken in the
    precision the kernel uses."""
    s = np.asarray(topk_score, np.float32)
    T, K = s.shape
    thr = np.float32(P)
    n = np.full(T, K, np.int32)
    for t in range(T):
        cum = np.float32(0.0)
        for j in range(K):
            cum = np.float32(cum + s[t, j])
            if cum >= thr:
                n[t] = j + 1
                break
    return n


def rel_threshold_count(topk_score, beta: float) -> np.ndarray:
    """Expert skipping relative to the top-1 score (App. A.1, the NAEE setting extended from Top-2
    to Top-K): the k-th expert of a token is skipped when its score is below beta times the token's
    top-1 score.  Rows are sorted descending, so the kept experts are a prefix; the top-1 expert is
    never skipped.  fp32 product and comparison."""
    s = np.asarray(topk_score, np.float32)
    T, K = s.shape
    n = np.ones(T, np.int32)
    for t in range(T):
        cut = np.float32(np.float32(beta) * s[t, 0])
        for j in range(1, K):
            if s[t, j] >= cut:
                n[t] = j + 1
            else:
                break
    return n


# ----------------------------------------------------------------------------- permutation
def permute(topk_idx, topk_score, n_sel, N: int) -> Dict[str, np.ndarray]:
    """Kept pairs listed expert-ascending, token-ascending inside an expert.
      expert_offsets [N+1]: exclusive prefix of per-expert counts, offsets[N] = total
      perm_token [B], perm_weight [B]: token and routing score of each listed pair
      pair_pos [T,K_orig]: position of pair (t,j) in the list, -1 if not kept."""
    idx = np.asarray(topk_idx)
    sc = np.asarray(topk_score, np.float32)
    n = np.asarray(n_sel)
    T, K = idx.shape
    kept = [(int(idx[t, j]), t, j) for t in range(T) for j in range(int(n[t]))]
    kept.sort(key=lambda etj: (etj[0], etj[1]))
    B = len(kept)
    offsets = np.zeros(N + 1, np.int32)
    perm_token = np.empty(B, np.int32)
    perm_weight = np.empty(B, np.float32)
    pair_pos = np.full((T, K), -1, np.int32)
    for p, (e, t, j) in enumerate(kept):
        offsets[e + 1] += 1
        perm_token[p] = t
        perm_weight[p] = sc[t, j]
        pair_pos[t, j] = p
    offsets = np.cumsum(offsets).astype(np.int32)
    return dict(expert_offsets=offsets, perm_token=perm_token, perm_weight=perm_weight, pair_pos=pair_pos)


# ----------------------------------------------------------------------------- experts, Eq. 2
def silu(a: np.ndarray) -> np.ndarray:
    return a / (1.0 + np.exp(-a))


def expert_ffn(x_rows, W13_e, W2_e) -> np.ndarray:
    """One SwiGLU expert on a block of rows: (silu(x W1^T) * (x W3^T)) W2^T, fp64.
    W13_e is [2I,H] (W1 rows then W3 rows), W2_e is [H,I]."""
    xr = np.asarray(x_rows, F64)
    W13 = np.asarray(W13_e, F64)
    I = W13.shape[0] // 2
    g = xr @ W13[:I].T
    u = xr @ W13[I:].T
    return (silu(g) * u) @ np.asarray(W2_e, F64).T


def shared_experts(x, Wsh13, Wsh2, rows: Optional[Sequence[int]] = None) -> np.ndarray:
    """sum_s E^sh_s(x_t) for the given rows (all rows by default), weight 1."""
    xr = np.asarray(x, F64) if rows is None else np.asarray(x, F64)[list(rows)]
    out = np.zeros((xr.shape[0], np.asarray(Wsh2).shape[1]), F64)
    for s in range(np.asarray(Wsh13).shape[0]):
        out += expert_ffn(xr, Wsh13[s], Wsh2[s])
    return out


def combine(x, topk_idx, topk_score, n_sel, W13, W2, Wsh13=None, Wsh2=None,
            rows: Optional[Sequence[int]] = None) -> np.ndarray:
    """Eq. 2 restricted to the kept pairs: out_t = sum_{j<n_t} score[t,j] E_{idx[t,j]}(x_t)
    (+ shared experts).  `rows` limits the computation to a sample of tokens.  fp64."""
    xx = np.asarray(x, F64)
    idx = np.asarray(topk_idx)
    sc = np.asarray(topk_score, F64)
    n = np.asarray(n_sel)
    rows = list(range(xx.shape[0])) if rows is None else list(rows)
    H = xx.shape[1]
    out = np.zeros((len(rows), H), F64)
    by_expert: Dict[int, List[Tuple[int, int, int]]] = {}
    for r, t in enumerate(rows):
        for j in range(int(n[t])):
            by_expert.setdefault(int(idx[t, j]), []).append((r, t, j))
    for e in sorted(by_expert):
        lst = by_expert[e]
        y = expert_ffn(xx[[t for (_, t, _) in lst]], W13[e], W2[e])
        for q, (r, t, j) in enumerate(lst):
            out[r] += sc[t, j] * y[q]
    if Wsh13 is not None:
        out += shared_experts(xx, Wsh13, Wsh2, rows)
    return out


def route(x, W_gate, gate_bias, K_orig: int, K_base: int, budget: int) -> Dict[str, np.ndarray]:
    """Eq. 1 then Alloc-T: scores, sorted Top-K_orig, kept counts n_sel."""
    scores = softmax_scores(gate_logits(x, W_gate, gate_bias))
    topk_idx, topk_score = topk_sorted(scores, K_orig)
    z = alloc_t_select_threshold(topk_score, K_base, budget)
    return dict(scores=scores, topk_idx=topk_idx, topk_score=topk_score, z=z, n_sel=n_sel_from_mask(z))


def layer_forward(x, W_gate, gate_bias, W13, W2, Wsh13, Wsh2, K_orig: int, K_base: int, budget: int,
                  rows: Optional[Sequence[int]] = None) -> Dict[str, np.ndarray]:
    """The whole budgeted layer: Eq. 1, Alloc-T, permutation, experts, Eq. 2.  `out` is fp64."""
    r = route(x, W_gate, gate_bias, K_orig, K_base, budget)
    r.update(permute(r["topk_idx"], r["topk_score"], r["n_sel"], np.asarray(W_gate).shape[1]))
    r["out"] = combine(x, r["topk_idx"], r["topk_score"], r["n_sel"], W13, W2, Wsh13, Wsh2, rows)
    return r


def layer_forward_dense(x, W_gate, gate_bias, W13, W2, Wsh13, Wsh2, K_orig, K_base, budget) -> np.ndarray:
    """Eq. 2 literally: every one of the N experts runs on every token and is weighted by
    w[t,i], which is the softmax score if (t,i) is kept and 0 otherwise (small inputs only)."""
    xx = np.asarray(x, F64)
    r = route(x, W_gate, gate_bias, K_orig, K_base, budget)
    T, N = r["scores"].shape
    w = np.zeros((T, N), F64)
    for t in range(T):
        for j in range(K_orig):
            if r["z"][t, j]:
                w[t, r["topk_idx"][t, j]] = r["topk_score"][t, j]
    out = np.zeros_like(xx)
    for i in range(N):
        out += w[:, i:i + 1] * expert_ffn(xx, W13[i], W2[i])
    if Wsh13 is not None:
        out += shared_experts(xx, Wsh13, Wsh2)
    return out


def bf16_round(a) -> np.ndarray:
    """Round fp64/fp32 values to the nearest bf16 (ties to even), returned as fp32.
    Used only where the layer stack hands x_{l+1} to the next layer in bf16 storage."""
    f = np.asarray(a, np.float32).copy()
    u = f.view(np.uint32)
    lsb = (u >> 16) & 1
    u += 0x7FFF + lsb
    u &= 0xFFFF0000
    return f


def rmsnorm(x, eps: float = 1e-6) -> np.ndarray:
    """x[t] / sqrt(mean_h x[t,h]^2 + eps), unit gain, fp64 (the pre-norm of the layer stack)."""
    xx = np.asarray(x, F64)
    return xx / np.sqrt((xx * xx).mean(axis=1, keepdims=True) + eps)


def stack_forward(x0, layers: Sequence[Dict[str, np.ndarray]], K_orig: int, K_base: int,
                  budgets: Sequence[int], prenorm: bool = True) -> List[np.ndarray]:
    """Residual stack with the stream stored in bf16 between layers (storage format of the
    workload): x_{l+1} = x_l + MoE_l(norm(x_l)), norm = RMS normalisation rounded to bf16, or the
    identity with prenorm=False.  The literal recurrence x + MoE(x) squares the stream's scale
    every layer (SwiGLU is quadratic in its input) and overflows within a dozen layers, so the
    stack workload is run pre-norm, as the transformer blocks it stands for are.
    Returns [x_1, ..., x_L] as fp32 arrays."""
    xs = []
    x = np.asarray(x0, np.float32)
    for lw, b in zip(layers, budgets):
        xin = bf16_round(rmsnorm(x)) if prenorm else x
        out = layer_forward(xin, lw["W_gate"], lw.get("gate_bias"), lw["W13"], lw["W2"],
                            lw.get("Wsh13"), lw.get("Wsh2"), K_orig, K_base, b)["out"]
        x = bf16_round(np.asarray(x, F64) + out)
        xs.append(x)
    return xs


# ----------------------------------------------------------------------------- Alloc-L (host side)
def alloc_l_dp(S, B: int) -> Tuple[List[int], float]:
    """Eq. 3-6: choose K_i in 1..K_orig per layer minimising sum S[i,K_i] with sum K_i <= B.
    DP[i,b] = min_k DP[i-1,b-k] + S[i,k]; DP[-1,0] = 0, DP[-1,b>0] = +inf; the answer is the
    best DP[L-1,b] over b <= B, recovered by backtracking.  S[i,k-1] holds the cost of k.
    Ties: the smaller k, then the smaller b."""
    S = np.asarray(S, F64)
    L, K = S.shape
    if B < L:
        raise ValueError("budget below one activation per layer")
    INF = float("inf")
    prev = [0.0] + [INF] * B
    choice = np.zeros((L, B + 1), np.int32)
    for i in range(L):
        cur = [INF] * (B + 1)
        for b in range(B + 1):
            for k in range(1, min(K, b) + 1):
                v = prev[b - k] + S[i, k - 1]
                if v < cur[b]:
                    cur[b] = v
                    choice[i, b] = k
        prev = cur
    b = min(range(B + 1), key=lambda bb: (prev[bb], bb))
    best = prev[b]
    ks = [0] * L
    for i in range(L - 1, -1, -1):
        ks[i] = int(choice[i, b])
        b -= ks[i]
    return ks, float(best)


def alloc_l_bruteforce(S, B: int) -> float:
    """Eq. 3-5 by enumeration of all K_orig^L allocations (tiny L only): the optimal cost."""
    S = np.asarray(S, F64)
    L, K = S.shape
    best = float("inf")
    for ks in itertools.product(range(1, K + 1), repeat=L):
        if sum(ks) <= B:
            best = min(best, float(sum(S[i, ks[i] - 1] for i in range(L))))
    return best
