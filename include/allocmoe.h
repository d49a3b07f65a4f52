/*
 * allocmoe.h -- C ABI of the budget-constrained MoE layer forward (Alloc-MoE hot path)
 * for NVIDIA B200 (sm_100a).
 *
 * The layer (paper Sec. 3.1 and 3.3):
 *   Eq. 1   scores = Softmax(x . W_gate) over all N experts, Top-K_orig kept per token
 *   Alloc-T (Sec. 3.3, procedure paragraph; the 0/1 programme of Eq. 8-10): every token keeps
 *           its Top-K_base experts; the other K_orig-K_base scores of ALL tokens are pooled and
 *           the globally largest  budget - K_base*T  of them are kept
 *   Eq. 2   y_t = sum over kept (t,i) of score[t,i] * E_i(x_t)   (+ shared experts)
 *
 * Conventions for every entry point
 *   - Every pointer marked "device" is device memory owned by the caller, 16-byte aligned,
 *     valid until the stream has run the call.  The library allocates no device memory,
 *     never synchronises and launches only on `stream` (a cudaStream_t passed as void*).
 *   - bf16 tensors are passed as `const uint16_t*` (raw bfloat16 bits), row-major, last index
 *     contiguous.
 *   - `budget` is the layer's TOTAL activation count  T*K_l  (Sec. 3.1, "Expert Activation
 *     Budget"), so fractional per-token averages need no rounding rule.  It must satisfy
 *     K_base*T <= budget <= K_orig*T  (below: Eq. 10 is infeasible; above: the candidate
 *     set is exhausted); anything else returns MOE_ERR_BUDGET.
 *   - Host-checkable errors return a status before anything is launched and leave outputs
 *     untouched.  Conditions only the device can see (a non-finite or negative score, kept
 *     counts that do not add up to `budget`, a bounded wait that ran out) are written to the
 *     caller's `dev_status` word (device, int32, OR-ed bit mask of 1 << moe_status; the
 *     caller zeroes it) and the kernels return normally; outputs are then unspecified but
 *     every access stays in bounds.
 *   - Ties (the paper is silent): inside a token the lower expert id ranks first; inside the
 *     Alloc-T pool the lower flat index t*K_orig + j ranks first.  With rows sorted
 *     descending the kept pairs of token t are its columns 0 .. n_sel[t]-1.
 */
#ifndef ALLOCMOE_H_
#define ALLOCMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MOE_OK = 0,
  MOE_ERR_ARG = 1,        /* null / misaligned pointer, unsupported shape */
  MOE_ERR_BUDGET = 2,     /* budget outside [K_base*T, K_orig*T], or sum n_sel != budget */
  MOE_ERR_WORKSPACE = 3,  /* workspace too small */
  MOE_ERR_CUDA = 4,       /* a CUDA runtime / driver call failed */
  MOE_ERR_NONFINITE = 5,  /* a routing score is NaN, Inf or negative */
  MOE_ERR_TIMEOUT = 6     /* a bounded device-side wait gave up */
} moe_status;

/* T tokens, H hidden size, N routed experts, I expert intermediate size, S shared experts,
 * K_orig nominal Top-K (candidates per token), K_base guaranteed experts per token (Eq. 10).
 * Supported: H % 64 == 0, I % 64 == 0, 8 <= N <= 128 with N % 4 == 0, 1 <= K_orig <= min(N, 16),
 * 0 <= K_base <= K_orig, S >= 0, T >= 1, T*K_orig < 2^31.  flags must be 0. */
typedef struct {
  int32_t T, H, N, I, S, K_orig, K_base;
  uint32_t flags;
} moe_shape;

const char* moe_status_string(moe_status s);

/* Bytes of device scratch that any call below needs for this shape with budgets up to
 * budget_max (0 on an invalid shape). */
size_t moe_workspace_bytes(const moe_shape* shape, int64_t budget_max);

/* Eq. 1.  logits = x . W_gate (+ gate_bias), fp32 accumulation; scores = row softmax over all
 * N experts in fp32; per token the K_orig largest scores, sorted descending (ties: lower expert
 * id first).
 *   x          device bf16 [T,H]
 *   W_gate     device bf16 [H,N]      (the paper's W_gate in R^{H x N})
 *   gate_bias  device fp32 [N] or NULL: added to the logits before the softmax
 *   scores     device fp32 [T,N] or NULL (full softmax output, optional)
 *   topk_idx   device int32 [T,K_orig]
 *   topk_score device fp32 [T,K_orig]
 * From about a thousand tokens on, with 64 or 128 experts, the contraction runs on the tensor cores fed by TMA; its
 * waits are bounded, and should one run out the affected tokens' scores are written as NaN (alloc_t_select then
 * reports MOE_ERR_NONFINITE; inside moe_layer_forward MOE_ERR_TIMEOUT is raised as well). */
moe_status moe_gate(const moe_shape* shape, const uint16_t* x, const uint16_t* W_gate,
                    const float* gate_bias, float* scores, int32_t* topk_idx, float* topk_score,
                    void* stream);

/* Alloc-T (Sec. 3.3).  Input rows sorted descending; output n_sel[t] in [K_base, K_orig] with
 * sum n_sel = budget: K_base plus the number of token t's residual scores among the
 * budget - K_base*T largest of the pool.  Exact: scores are compared as values (their IEEE bit
 * patterns, which order identically for non-negative floats), ties by flat index.
 *   topk_score device fp32 [T,K_orig]
 *   n_sel      device int32 [T]
 *   dev_status device int32 [1]  (see above)
 *   ws         device scratch, ws_bytes >= moe_workspace_bytes() */
moe_status alloc_t_select(const moe_shape* shape, const float* topk_score, int64_t budget,
                          int32_t* n_sel, int32_t* dev_status, void* ws, size_t ws_bytes,
                          void* stream);

/* Permutation of the kept (token, expert) pairs into per-expert segments: the step between Alloc-T's
 * selection (Sec. 3.3) and the per-expert feed-forward executions of Sec. 3.1.  The paper names no such
 * step -- it masks the scores and leaves the dispatch to the serving stack; the order below is this
 * library's choice.  Lists the kept pairs expert-ascending and token-ascending inside an expert.
 *   expert_offsets device int32 [N+1]   exclusive prefix of per-expert counts, [N] = budget
 *   perm_token     device int32 [budget] token of each listed pair
 *   perm_weight    device fp32  [budget] its routing score
 *   pair_pos       device int32 [T,K_orig] list position of pair (t,j), -1 if not kept
 *   x_perm         device bf16 [budget,H] or NULL: row p is x[perm_token[p]] */
moe_status moe_permute(const moe_shape* shape, const uint16_t* x, const int32_t* topk_idx,
                       const float* topk_score, const int32_t* n_sel, int64_t budget,
                       int32_t* expert_offsets, int32_t* perm_token, float* perm_weight,
                       int32_t* pair_pos, uint16_t* x_perm, int32_t* dev_status,
                       void* ws, size_t ws_bytes, void* stream);

/* alloc_t_select and the list-building part of moe_permute (everything but the x_perm gather) in
 * one launch: one CTA up to 1024 tokens, a thread-block cluster of ceil(T/1024) CTAs that exchange
 * their radix histograms and per-expert counts through distributed shared memory up to 8192 tokens.
 * This is the form moe_layer_forward uses at those sizes, where four separate launches cost more
 * than the work.  Outputs are bit-identical to the two separate calls.  T > 8192: MOE_ERR_ARG.
 * Needs no workspace. */
moe_status moe_route(const moe_shape* shape, const int32_t* topk_idx, const float* topk_score, int64_t budget,
                     int32_t* n_sel, int32_t* expert_offsets, int32_t* perm_token, float* perm_weight,
                     int32_t* pair_pos, int32_t* dev_status, void* stream);

/* The same operation as moe_permute for callers that have no device memory of their own to lend
 * and may not allocate any: code that runs inside a host application which handed out all GPU
 * memory at start-up (an inference-engine plug-in, a fixed-arena embedded deployment), or a
 * latency-critical loop in which the implicit device-wide synchronisation of cudaMalloc/cudaFree
 * is not acceptable.  (The paper has no counterpart: it describes no permutation step.)
 * Instead of a workspace, the per-(expert, 32-token segment) counters live in a fixed 256 KB
 * array inside the library image, present on every GPU that loads the library until the process
 * exits.  Inputs and outputs are passed exactly as for moe_permute and the results are identical.
 *   Limit   N * ceil(T/32) <= 65536 (e.g. T <= 32768 at N = 64); larger shapes return
 *           MOE_ERR_WORKSPACE and nothing is launched.
 *   Set-up  the first call on each device looks up the array's device address (the device must
 *           be current, as for every call); make that first call before any stream capture
 *           begins.
 *   Sharing all calls on a device use the one array.  Nothing in it has to start at zero (each
 *           call writes every counter before reading it), so back-to-back calls on one stream are
 *           fine; two calls whose kernels can overlap on the GPU (different streams) race on it
 *           and give undefined results.
 * The call allocates nothing and calls no allocating routine. */
moe_status moe_permute_static(const moe_shape* shape, const uint16_t* x, const int32_t* topk_idx,
                              const float* topk_score, const int32_t* n_sel, int64_t budget,
                              int32_t* expert_offsets, int32_t* perm_token, float* perm_weight,
                              int32_t* pair_pos, uint16_t* x_perm, int32_t* dev_status,
                              void* stream);

/* Routed experts: one expert feed-forward execution per kept (token, expert) pair (Sec. 3.1, the cost
 * model behind the activation budget).  For every listed pair p of expert e:
 *   h = silu(x_p W1_e^T) * (x_p W3_e^T)  (fp32 accumulation, h stored as bf16)
 *   y_perm[p] = h W2_e^T                 (fp32 accumulation, stored as bf16)
 *   x_or_xperm device bf16: with perm_token == NULL the rows in list order, [budget,H] (moe_permute's
 *              x_perm); with perm_token given the tokens themselves, x [T,H], and row p is
 *              x[perm_token[p]] -- read by index straight from x where expert runs are short (at most 32
 *              rows per expert on average), gathered once into the workspace otherwise
 *   perm_token device int32 [budget] or NULL
 *   W13     device bf16 [N,2I,H]    rows 0..I-1 of an expert are W1, rows I..2I-1 are W3
 *   W2      device bf16 [N,H,I]
 *   y_perm  device bf16 [budget,H]
 * Experts with no rows read no weights.  expert_offsets (device int32 [N+1]) is trusted to be
 * non-decreasing within [0, budget]; values outside are clamped to that range on the device, and so are
 * the entries of perm_token to [0, T), so an inconsistent list gives meaningless rows but no access
 * outside x, y_perm or the workspace. */
moe_status moe_grouped_ffn(const moe_shape* shape, const uint16_t* x_or_xperm, const int32_t* perm_token,
                           const int32_t* expert_offsets, int64_t budget, const uint16_t* W13,
                           const uint16_t* W2, uint16_t* y_perm, int32_t* dev_status, void* ws,
                           size_t ws_bytes, void* stream);

/* Shared experts: y_shared[t] = sum_s E^sh_s(x_t) for every token (weight 1, outside the
 * budget; a workload parameter, the paper's budgets count routed experts only).
 *   Wsh13 device bf16 [S,2I,H], Wsh2 device bf16 [S,H,I], y_shared device bf16 [T,H] */
moe_status moe_shared_ffn(const moe_shape* shape, const uint16_t* x, const uint16_t* Wsh13,
                          const uint16_t* Wsh2, uint16_t* y_shared, int32_t* dev_status, void* ws,
                          size_t ws_bytes, void* stream);

/* Eq. 2 over the kept pairs: out[t] = sum_{j<n_sel[t]} topk_score[t,j] * y_perm[pair_pos[t,j]]
 * (+ y_shared[t]); fp32, j ascending, one rounding to bf16.
 *   y_shared device bf16 [T,H] or NULL;  out device bf16 [T,H] */
moe_status moe_combine(const moe_shape* shape, const uint16_t* y_perm, const int32_t* pair_pos,
                       const float* topk_score, const int32_t* n_sel, const uint16_t* y_shared,
                       uint16_t* out, void* stream);

/* The whole budgeted layer (Eq. 1, Alloc-T of Sec. 3.3 / Eq. 8-10, Eq. 2) on one stream: moe_gate,
 * alloc_t_select, moe_permute, moe_grouped_ffn (+ moe_shared_ffn when S > 0), moe_combine; all
 * intermediates live in `ws`.
 * Wsh13 / Wsh2 are ignored when S == 0.
 *   residual  device bf16 [T,H] or NULL: added to the result, out = residual + MoE(x) (fp32 add,
 *             one bf16 rounding): the step of a residual layer stack.  May alias x, not out. */
moe_status moe_layer_forward(const moe_shape* shape, const uint16_t* x, const uint16_t* W_gate,
                             const float* gate_bias, const uint16_t* W13, const uint16_t* W2,
                             const uint16_t* Wsh13, const uint16_t* Wsh2, int64_t budget,
                             const uint16_t* residual, uint16_t* out, int32_t* dev_status, void* ws,
                             size_t ws_bytes, void* stream);

/* The layer from a selection the caller already holds: permutation, experts and Eq. 2 for the given
 * Top-K_orig rows and kept counts.  This is the local part of Alloc-T over a batch that is sharded across
 * GPUs (Sec. 3.3 pools the scores of all tokens): each rank runs moe_gate, the ranks exchange their score
 * rows, every rank runs alloc_t_select on the whole pool and hands its own slice of n_sel to this call.
 * How many pairs this rank keeps is then known to the device only, so the call takes an upper bound:
 *   n_sel       device int32 [T], values in [0, K_orig]
 *   budget_max  upper bound of sum n_sel; sizes the workspace (moe_workspace_bytes(shape, budget_max)).
 *               A larger sum raises MOE_ERR_BUDGET in dev_status; every access stays in bounds.
 *   budget_hint expected sum (0: budget_max); only picks between kernel variants, any value is correct
 * Everything else as for moe_layer_forward.  Nothing is read back to the host. */
moe_status moe_layer_forward_routed(const moe_shape* shape, const uint16_t* x, const int32_t* topk_idx,
                                    const float* topk_score, const int32_t* n_sel, int64_t budget_max,
                                    int64_t budget_hint, const uint16_t* W13, const uint16_t* W2,
                                    const uint16_t* Wsh13, const uint16_t* Wsh2, const uint16_t* residual,
                                    uint16_t* out, int32_t* dev_status, void* ws, size_t ws_bytes,
                                    void* stream);

/* The two token-level rules the paper measures Alloc-T against (Sec. 2, related work; App. A.1, baseline
 * settings), with Alloc-T's output format so that moe_layer_forward_routed can run the layer on them.  They
 * decide token by token from a threshold that those methods calibrate off line to meet a target budget;
 * nothing is pooled, so the kept total is whatever the threshold gives (read it from `total`).
 *   moe_select_top_p          Top-P routing: n_sel[t] = the smallest n >= 1 with
 *                             topk_score[t,0] + ... + topk_score[t,n-1] >= P (fp32, summed in column order),
 *                             K_orig if the row never reaches P
 *   moe_select_rel_threshold  expert skipping relative to the top-1 score: column j >= 1 is dropped when
 *                             topk_score[t,j] < beta * topk_score[t,0] (fp32 product); n_sel[t] counts the
 *                             leading columns that stay, at least 1
 *   topk_score device fp32 [T,K_orig], rows descending;  n_sel device int32 [T]
 *   total      device int32 [1] or NULL: sum of n_sel is ADDED to it (the caller zeroes it)
 *   dev_status MOE_ERR_NONFINITE is raised for a NaN, Inf or negative score, as in alloc_t_select */
moe_status moe_select_top_p(const moe_shape* shape, const float* topk_score, float P, int32_t* n_sel,
                            int32_t* total, int32_t* dev_status, void* stream);
moe_status moe_select_rel_threshold(const moe_shape* shape, const float* topk_score, float beta, int32_t* n_sel,
                                    int32_t* total, int32_t* dev_status, void* stream);

/* Pre-norm of a residual layer stack (not part of the paper's method; the layer stack workload
 * needs it, see the stack recurrence x_{l+1} = x_l + MoE(norm(x_l))): out[t] = x[t] / sqrt(mean_h
 * x[t,h]^2 + 1e-6), unit gain, fp32 math, one bf16 rounding.  x, out device bf16 [T,H]. */
moe_status moe_rmsnorm(const moe_shape* shape, const uint16_t* x, uint16_t* out, void* stream);

/* Device addresses of the routing intermediates that moe_layer_forward, called with this shape,
 * this budget and this workspace, leaves in `ws` (for inspection and tests; valid until ws is
 * reused; the carve-up depends on the budget).  Any output pointer may be NULL. */
moe_status moe_layer_intermediates(const moe_shape* shape, int64_t budget, void* ws,
                                   size_t ws_bytes, int32_t** topk_idx, float** topk_score,
                                   int32_t** n_sel, int32_t** expert_offsets,
                                   int32_t** perm_token, int32_t** pair_pos, uint16_t** y_perm);

/* Alloc-L, the layer-level allocation (Sec. 3.2, Eq. 3-6): K_i in 1..K_orig per layer minimising
 * sum_i S[i, K_i] subject to sum_i K_i <= B, solved exactly by the grouped-knapsack dynamic
 * programme of Eq. 6 with backtracking.  Host code, run once off line; no GPU involved.
 *   S        host fp64 [L, K_orig] row-major; S[i, k-1] is the sensitivity cost of giving layer i
 *            k experts per token (the paper's S[i, k]); must be finite
 *   B        global budget per token; B < L returns MOE_ERR_BUDGET (Eq. 5 infeasible)
 *   K_out    host int32 [L]: the optimal allocation (ties: the smaller k, then the smaller total)
 *   cost_out host fp64 [1] or NULL: its total cost
 * K_orig <= 255.  MOE_ERR_WORKSPACE if the host cannot allocate the L * (min(B, L*K_orig) + 1)
 * bytes of backtracking state. */
moe_status alloc_l_solve(const double* S, int32_t L, int32_t K_orig, int64_t B, int32_t* K_out, double* cost_out);

/* Instrumentation (no counterpart in the paper): with profiling on, moe_layer_forward records
 * CUDA events at its stage boundaries; moe_profile_read waits for the last forward call and
 * returns the device time in milliseconds of its 6 stages: gate; route (Alloc-T selection and the
 * permutation's lists in one launch; beyond 8192 tokens the selection alone); gather (the copy of
 * the routed rows, absent where the expert GEMM reads x by index; beyond 8192 tokens also the
 * permutation's lists); expert GEMM-1 (with SwiGLU); expert GEMM-2; combine.  Host-side state only
 * (events); one forward call at a time may be in flight while profiling.  Off by default. */
#define MOE_PROFILE_STAGES 6
moe_status moe_profile_enable(int32_t on);
moe_status moe_profile_read(float* stage_ms /* host [MOE_PROFILE_STAGES] */);

/* Self-test of the failure path (no counterpart in the paper).  Every device-side wait of the expert
 * GEMMs is bounded: a wait that outlasts its limit raises MOE_ERR_TIMEOUT in dev_status, the CTA's other
 * roles leave their loops at their next poll, the CTA waits for its copies in flight, frees its tensor
 * memory and returns.  In production the limit is about half a second and nothing reaches it.  This
 * call makes it happen on purpose, harmlessly: it launches expert GEMM-2 alone, with the row-block
 * counters that GEMM-1 would fill cleared and never filled, and with the waits' limit set to
 * wait_limit_clk SM clocks (1000 .. 2e9).  Expected outcome: the call returns MOE_OK, the kernel ends
 * within a few multiples of the limit, dev_status holds 1 << MOE_ERR_TIMEOUT, y_perm is not written,
 * and the next ordinary call on the same workspace is correct.
 *   expert_offsets device int32 [N+1]; budget = rows of y_perm; W2 device bf16 [N,H,I];
 *   y_perm device bf16 [budget,H]; ws as for moe_grouped_ffn */
moe_status moe_selftest_wait_timeout(const moe_shape* shape, const int32_t* expert_offsets, int64_t budget,
                                     const uint16_t* W2, uint16_t* y_perm, int64_t wait_limit_clk,
                                     int32_t* dev_status, void* ws, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ALLOCMOE_H_ */
