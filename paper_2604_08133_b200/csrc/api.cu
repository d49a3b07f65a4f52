// C-ABI entry points (see include/allocmoe.h): argument checks, workspace carve-up, launches.
// Nothing here allocates or synchronises; every launch goes to the caller's stream.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include "allocmoe.h"

#include "ffn.h"
#include "shape_check.h"

// launchers defined next to their kernels
moe_status launch_moe_gate(const moe_shape*, const uint16_t*, const uint16_t*, const float*, float*, int32_t*, float*,
                           int32_t*, int, int32_t*, cudaStream_t);
moe_status launch_alloc_t_select(const moe_shape*, const float*, int64_t, int32_t*, int32_t*, cudaStream_t);
moe_status launch_moe_permute(const moe_shape*, const uint16_t*, const int32_t*, const float*, const int32_t*, int64_t,
                              int32_t*, int32_t*, float*, int32_t*, uint16_t*, int32_t*, int32_t*, bool, cudaStream_t);
moe_status launch_gather_rows(const moe_shape*, const uint16_t*, const int32_t*, int64_t, const int32_t*, uint16_t*,
                              int32_t*, cudaStream_t);
bool moe_route_fits(const moe_shape*);
moe_status launch_moe_route(const moe_shape*, const float*, const int32_t*, int64_t, bool, int32_t*, int32_t*, int32_t*,
                            float*, int32_t*, int32_t*, cudaStream_t);
moe_status launch_moe_combine(const moe_shape*, const uint16_t*, const int32_t*, const float*, const int32_t*,
                              const uint16_t*, const uint16_t*, long long, uint16_t*, cudaStream_t);
moe_status launch_rmsnorm(const moe_shape*, const uint16_t*, uint16_t*, cudaStream_t);
moe_status launch_token_rule_select(const moe_shape*, const float*, int, float, int32_t*, int32_t*, int32_t*, cudaStream_t);

namespace {

using allocmoe::aligned16;
using allocmoe::shape_ok;

bool budget_ok(const moe_shape* s, int64_t budget) {
  return budget >= (int64_t)s->K_base * s->T && budget <= (int64_t)s->K_orig * s->T;
}

// Fixed carve-up of the workspace; every region starts on a 256-byte boundary.
struct WsLayout {
  size_t topk_idx, topk_score, n_sel, expert_offsets, perm_token, perm_weight, pair_pos, seg_counts;
  size_t x_perm, h, y_perm, h_sh, y_shared, gemm_done, total;
};

WsLayout ws_layout(const moe_shape* s, int64_t budget_max) {
  WsLayout L{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t at = off;
    off += (bytes + 255) & ~(size_t)255;
    return at;
  };
  const size_t T = s->T, H = s->H, N = s->N, I = s->I, S = s->S, K = s->K_orig, B = (size_t)budget_max;
  L.topk_idx = take(T * K * 4);
  L.topk_score = take(T * K * 4);
  L.n_sel = take(T * 4);
  L.expert_offsets = take((N + 1) * 4);
  L.perm_token = take(B * 4);
  L.perm_weight = take(B * 4);
  L.pair_pos = take(T * K * 4);
  L.seg_counts = take(N * ((T + 31) / 32) * 4);
  L.x_perm = take(B * H * 2);
  L.h = take(B * I * 2);
  L.y_perm = take(B * H * 2);
  L.h_sh = take(T * S * I * 2);
  L.y_shared = take(T * H * 2);
  L.gemm_done = take(ffn_done_ints(s, budget_max) * 4);
  L.total = off;
  return L;
}

// One NVTX range per C-ABI call (header-only NVTX: a no-op costing a few nanoseconds unless a profiler is
// attached), so that a timeline shows which entry point enqueued which kernels.
struct ApiRange {
  explicit ApiRange(const char* name) { nvtxRangePushA(name); }
  ~ApiRange() { nvtxRangePop(); }
  ApiRange(const ApiRange&) = delete;
  ApiRange& operator=(const ApiRange&) = delete;
};

template <typename T>
T* at(void* ws, size_t off) { return reinterpret_cast<T*>(static_cast<unsigned char*>(ws) + off); }

// Optional stage timing of moe_layer_forward (off by default): events at the stage boundaries.
constexpr int kProfStages = 6;   // gate, route, gather, ffn GEMM-1, ffn GEMM-2, combine
bool g_prof_on = false;
cudaEvent_t g_prof_ev[kProfStages + 1];
void prof_mark(int i, cudaStream_t st) {
  if (g_prof_on) cudaEventRecord(g_prof_ev[i], st);
}

}  // namespace

extern "C" {

const char* moe_status_string(moe_status s) {
  switch (s) {
    case MOE_OK: return "ok";
    case MOE_ERR_ARG: return "invalid argument (null or misaligned pointer, unsupported shape)";
    case MOE_ERR_BUDGET: return "budget outside [K_base*T, K_orig*T] or kept counts do not add up to it";
    case MOE_ERR_WORKSPACE: return "workspace too small";
    case MOE_ERR_CUDA: return "CUDA call failed";
    case MOE_ERR_NONFINITE: return "routing score is NaN, Inf or negative";
    case MOE_ERR_TIMEOUT: return "bounded device wait gave up";
  }
  return "unknown status";
}

size_t moe_workspace_bytes(const moe_shape* shape, int64_t budget_max) {
  if (!shape_ok(shape) || budget_max < 0 || budget_max > (int64_t)shape->K_orig * shape->T) return 0;
  return ws_layout(shape, budget_max).total;
}

moe_status moe_gate(const moe_shape* shape, const uint16_t* x, const uint16_t* W_gate, const float* gate_bias,
                    float* scores, int32_t* topk_idx, float* topk_score, void* stream) {
  ApiRange nvtx_range("moe_gate");
  if (!shape_ok(shape) || !x || !W_gate || !topk_idx || !topk_score) return MOE_ERR_ARG;
  if (!aligned16(x) || !aligned16(W_gate) || !aligned16(topk_idx) || !aligned16(topk_score)) return MOE_ERR_ARG;
  return launch_moe_gate(shape, x, W_gate, gate_bias, scores, topk_idx, topk_score, nullptr, 0, nullptr,
                         (cudaStream_t)stream);
}

moe_status alloc_t_select(const moe_shape* shape, const float* topk_score, int64_t budget, int32_t* n_sel,
                          int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  ApiRange nvtx_range("alloc_t_select");
  (void)ws;
  (void)ws_bytes;
  if (!shape_ok(shape) || !topk_score || !n_sel || !dev_status) return MOE_ERR_ARG;
  if (!aligned16(topk_score) || !aligned16(n_sel)) return MOE_ERR_ARG;
  if (!budget_ok(shape, budget)) return MOE_ERR_BUDGET;
  return launch_alloc_t_select(shape, topk_score, budget, n_sel, dev_status, (cudaStream_t)stream);
}

moe_status moe_permute(const moe_shape* shape, const uint16_t* x, const int32_t* topk_idx, const float* topk_score,
                       const int32_t* n_sel, int64_t budget, int32_t* expert_offsets, int32_t* perm_token,
                       float* perm_weight, int32_t* pair_pos, uint16_t* x_perm, int32_t* dev_status, void* ws,
                       size_t ws_bytes, void* stream) {
  ApiRange nvtx_range("moe_permute");
  if (!shape_ok(shape) || !topk_idx || !topk_score || !n_sel || !expert_offsets || !perm_token || !perm_weight ||
      !pair_pos || !dev_status || !ws)
    return MOE_ERR_ARG;
  if (x_perm != nullptr && (!x || !aligned16(x) || !aligned16(x_perm))) return MOE_ERR_ARG;
  if (!aligned16(ws)) return MOE_ERR_ARG;
  if (!budget_ok(shape, budget)) return MOE_ERR_BUDGET;
  const WsLayout L = ws_layout(shape, budget);
  if (ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  return launch_moe_permute(shape, x, topk_idx, topk_score, n_sel, budget, expert_offsets, perm_token, perm_weight,
                            pair_pos, x_perm, dev_status, at<int32_t>(ws, L.seg_counts), true, (cudaStream_t)stream);
}

moe_status moe_route(const moe_shape* shape, const int32_t* topk_idx, const float* topk_score, int64_t budget,
                     int32_t* n_sel, int32_t* expert_offsets, int32_t* perm_token, float* perm_weight, int32_t* pair_pos,
                     int32_t* dev_status, void* stream) {
  ApiRange nvtx_range("moe_route");
  if (!shape_ok(shape) || !topk_idx || !topk_score || !n_sel || !expert_offsets || !perm_token || !perm_weight ||
      !pair_pos || !dev_status)
    return MOE_ERR_ARG;
  if (!aligned16(topk_idx) || !aligned16(topk_score) || !aligned16(n_sel)) return MOE_ERR_ARG;
  if (!moe_route_fits(shape)) return MOE_ERR_ARG;
  if (!budget_ok(shape, budget)) return MOE_ERR_BUDGET;
  return launch_moe_route(shape, topk_score, topk_idx, budget, false, n_sel, expert_offsets, perm_token, perm_weight,
                          pair_pos, dev_status, (cudaStream_t)stream);
}

moe_status moe_grouped_ffn(const moe_shape* shape, const uint16_t* x_or_xperm, const int32_t* perm_token,
                           const int32_t* expert_offsets, int64_t budget, const uint16_t* W13, const uint16_t* W2,
                           uint16_t* y_perm, int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  ApiRange nvtx_range("moe_grouped_ffn");
  if (!shape_ok(shape) || !x_or_xperm || !expert_offsets || !W13 || !W2 || !y_perm || !dev_status || !ws)
    return MOE_ERR_ARG;
  if (!aligned16(x_or_xperm) || !aligned16(W13) || !aligned16(W2) || !aligned16(y_perm) || !aligned16(ws))
    return MOE_ERR_ARG;
  if (budget < 0 || budget > (int64_t)shape->K_orig * shape->T) return MOE_ERR_BUDGET;
  const WsLayout L = ws_layout(shape, budget);
  if (ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  FfnArgs a;
  a.s = shape;
  a.a_routed = x_or_xperm;
  a.gather_idx = perm_token;
  if (perm_token != nullptr && budget > 0 && !ffn_gathers(shape, budget)) {
    // long expert runs: one copy of the rows into the workspace, then 128-row box loads, is faster than
    // fetching every tile's rows four at a time
    const moe_status r = launch_gather_rows(shape, x_or_xperm, perm_token, budget, nullptr, at<uint16_t>(ws, L.x_perm), dev_status, st);
    if (r != MOE_OK) return r;
    a.a_routed = at<uint16_t>(ws, L.x_perm);
    a.gather_idx = nullptr;
  }
  a.expert_offsets = expert_offsets;
  a.budget = budget;
  a.W13 = W13;
  a.W2 = W2;
  a.h = at<uint16_t>(ws, L.h);
  a.y_perm = y_perm;
  a.dev_status = dev_status;
  a.done = at<int32_t>(ws, L.gemm_done);
  a.stream = st;
  return launch_ffn(a);
}

moe_status moe_shared_ffn(const moe_shape* shape, const uint16_t* x, const uint16_t* Wsh13, const uint16_t* Wsh2,
                          uint16_t* y_shared, int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  ApiRange nvtx_range("moe_shared_ffn");
  if (!shape_ok(shape) || shape->S < 1 || !x || !Wsh13 || !Wsh2 || !y_shared || !dev_status || !ws) return MOE_ERR_ARG;
  if (!aligned16(x) || !aligned16(Wsh13) || !aligned16(Wsh2) || !aligned16(y_shared) || !aligned16(ws)) return MOE_ERR_ARG;
  const WsLayout L = ws_layout(shape, 0);
  if (ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  FfnArgs a;
  a.s = shape;
  a.x_shared = x;
  a.Wsh13 = Wsh13;
  a.Wsh2 = Wsh2;
  a.h_sh = at<uint16_t>(ws, L.h_sh);
  a.y_shared = y_shared;
  a.dev_status = dev_status;
  a.done = at<int32_t>(ws, L.gemm_done);
  a.stream = (cudaStream_t)stream;
  return launch_ffn(a);
}

moe_status moe_combine(const moe_shape* shape, const uint16_t* y_perm, const int32_t* pair_pos,
                       const float* topk_score, const int32_t* n_sel, const uint16_t* y_shared, uint16_t* out,
                       void* stream) {
  ApiRange nvtx_range("moe_combine");
  if (!shape_ok(shape) || !y_perm || !pair_pos || !topk_score || !n_sel || !out) return MOE_ERR_ARG;
  if (!aligned16(y_perm) || !aligned16(out) || (y_shared && !aligned16(y_shared))) return MOE_ERR_ARG;
  return launch_moe_combine(shape, y_perm, pair_pos, topk_score, n_sel, y_shared, nullptr,
                            (long long)shape->K_orig * shape->T, out, (cudaStream_t)stream);
}

moe_status moe_layer_forward(const moe_shape* shape, const uint16_t* x, const uint16_t* W_gate, const float* gate_bias,
                             const uint16_t* W13, const uint16_t* W2, const uint16_t* Wsh13, const uint16_t* Wsh2,
                             int64_t budget, const uint16_t* residual, uint16_t* out, int32_t* dev_status, void* ws,
                             size_t ws_bytes, void* stream) {
  ApiRange nvtx_range("moe_layer_forward");
  if (!shape_ok(shape) || !x || !W_gate || !W13 || !W2 || !out || !dev_status || !ws) return MOE_ERR_ARG;
  if (shape->S > 0 && (!Wsh13 || !Wsh2)) return MOE_ERR_ARG;
  if (!aligned16(x) || !aligned16(W_gate) || !aligned16(W13) || !aligned16(W2) || !aligned16(out) || !aligned16(ws))
    return MOE_ERR_ARG;
  if (shape->S > 0 && (!aligned16(Wsh13) || !aligned16(Wsh2))) return MOE_ERR_ARG;
  if (residual != nullptr && (!aligned16(residual) || residual == out)) return MOE_ERR_ARG;
  if (!budget_ok(shape, budget)) return MOE_ERR_BUDGET;
  const WsLayout L = ws_layout(shape, budget);
  if (ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  int32_t* topk_idx = at<int32_t>(ws, L.topk_idx);
  float* topk_score = at<float>(ws, L.topk_score);
  int32_t* n_sel = at<int32_t>(ws, L.n_sel);
  int32_t* expert_offsets = at<int32_t>(ws, L.expert_offsets);
  int32_t* perm_token = at<int32_t>(ws, L.perm_token);
  float* perm_weight = at<float>(ws, L.perm_weight);
  int32_t* pair_pos = at<int32_t>(ws, L.pair_pos);
  uint16_t* x_perm = at<uint16_t>(ws, L.x_perm);
  uint16_t* y_perm = at<uint16_t>(ws, L.y_perm);
  uint16_t* y_shared = shape->S > 0 ? at<uint16_t>(ws, L.y_shared) : nullptr;

  // for short expert runs GEMM-1 fetches the routed tokens' rows from x by index and no permuted copy is made
  if (ffn_gathers(shape, budget)) x_perm = nullptr;

  prof_mark(0, st);
  // the gate launch also clears the expert GEMMs' row-block counters (no memset between kernels of the call)
  moe_status r = launch_moe_gate(shape, x, W_gate, gate_bias, nullptr, topk_idx, topk_score, at<int32_t>(ws, L.gemm_done),
                                 (int)ffn_done_ints(shape, budget), dev_status, st);
  if (r != MOE_OK) return r;
  prof_mark(1, st);
  if (moe_route_fits(shape)) {
    // selection and permutation bookkeeping in one launch, then the row gather
    r = launch_moe_route(shape, topk_score, topk_idx, budget, false, n_sel, expert_offsets, perm_token, perm_weight,
                         pair_pos, dev_status, st);
    if (r != MOE_OK) return r;
    prof_mark(2, st);
    if (budget > 0 && x_perm != nullptr) r = launch_gather_rows(shape, x, perm_token, budget, nullptr, x_perm, dev_status, st);
  } else {
    r = launch_alloc_t_select(shape, topk_score, budget, n_sel, dev_status, st);
    if (r != MOE_OK) return r;
    prof_mark(2, st);
    r = launch_moe_permute(shape, x, topk_idx, topk_score, n_sel, budget, expert_offsets, perm_token, perm_weight,
                           pair_pos, x_perm, dev_status, at<int32_t>(ws, L.seg_counts), true, st);
  }
  if (r != MOE_OK) return r;
  prof_mark(3, st);
  FfnArgs a;
  a.s = shape;
  a.a_routed = x_perm != nullptr ? x_perm : x;
  a.gather_idx = x_perm != nullptr ? nullptr : perm_token;
  a.expert_offsets = expert_offsets;
  a.budget = budget;
  a.W13 = W13;
  a.W2 = W2;
  a.h = at<uint16_t>(ws, L.h);
  a.y_perm = y_perm;
  a.x_shared = shape->S > 0 ? x : nullptr;
  a.Wsh13 = Wsh13;
  a.Wsh2 = Wsh2;
  a.h_sh = at<uint16_t>(ws, L.h_sh);
  a.y_shared = y_shared;
  a.dev_status = dev_status;
  a.done = at<int32_t>(ws, L.gemm_done);
  a.done_is_clear = true;
  a.stream = st;
  a.between = g_prof_on ? g_prof_ev[4] : nullptr;
  r = launch_ffn(a);
  if (r != MOE_OK) return r;
  prof_mark(5, st);
  r = launch_moe_combine(shape, y_perm, pair_pos, topk_score, n_sel, y_shared, residual, budget, out,
                         st);
  prof_mark(6, st);
  return r;
}

moe_status moe_layer_forward_routed(const moe_shape* shape, const uint16_t* x, const int32_t* topk_idx,
                                    const float* topk_score, const int32_t* n_sel, int64_t budget_max,
                                    int64_t budget_hint, const uint16_t* W13, const uint16_t* W2, const uint16_t* Wsh13,
                                    const uint16_t* Wsh2, const uint16_t* residual, uint16_t* out, int32_t* dev_status,
                                    void* ws, size_t ws_bytes, void* stream) {
  ApiRange nvtx_range("moe_layer_forward_routed");
  if (!shape_ok(shape) || !x || !topk_idx || !topk_score || !n_sel || !W13 || !W2 || !out || !dev_status || !ws)
    return MOE_ERR_ARG;
  if (shape->S > 0 && (!Wsh13 || !Wsh2)) return MOE_ERR_ARG;
  // n_sel is read one int at a time: a slice of a longer array (this rank's part of the pool's counts) is fine
  if (!aligned16(x) || !aligned16(topk_idx) || !aligned16(topk_score) || !aligned16(W13) || !aligned16(W2) ||
      !aligned16(out) || !aligned16(ws) || (reinterpret_cast<uintptr_t>(n_sel) & 3u) != 0)
    return MOE_ERR_ARG;
  if (shape->S > 0 && (!aligned16(Wsh13) || !aligned16(Wsh2))) return MOE_ERR_ARG;
  if (residual != nullptr && (!aligned16(residual) || residual == out)) return MOE_ERR_ARG;
  if (budget_max < 0 || budget_max > (int64_t)shape->K_orig * shape->T) return MOE_ERR_BUDGET;
  if (budget_hint < 0) return MOE_ERR_BUDGET;
  const WsLayout L = ws_layout(shape, budget_max);
  if (ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const int64_t expected = (budget_hint > 0 && budget_hint < budget_max) ? budget_hint : budget_max;
  int32_t* expert_offsets = at<int32_t>(ws, L.expert_offsets);
  int32_t* perm_token = at<int32_t>(ws, L.perm_token);
  float* perm_weight = at<float>(ws, L.perm_weight);
  int32_t* pair_pos = at<int32_t>(ws, L.pair_pos);
  uint16_t* x_perm = at<uint16_t>(ws, L.x_perm);
  uint16_t* y_perm = at<uint16_t>(ws, L.y_perm);
  uint16_t* y_shared = shape->S > 0 ? at<uint16_t>(ws, L.y_shared) : nullptr;
  if (ffn_gathers(shape, expected)) x_perm = nullptr;

  moe_status r;
  if (moe_route_fits(shape)) {
    r = launch_moe_route(shape, topk_score, topk_idx, budget_max, true, const_cast<int32_t*>(n_sel), expert_offsets,
                         perm_token, perm_weight, pair_pos, dev_status, st);
    if (r != MOE_OK) return r;
    if (budget_max > 0 && x_perm != nullptr)
      r = launch_gather_rows(shape, x, perm_token, budget_max, expert_offsets + shape->N, x_perm, dev_status, st);
  } else {
    r = launch_moe_permute(shape, x, topk_idx, topk_score, n_sel, budget_max, expert_offsets, perm_token, perm_weight,
                           pair_pos, x_perm, dev_status, at<int32_t>(ws, L.seg_counts), false, st);
  }
  if (r != MOE_OK) return r;
  FfnArgs a;
  a.s = shape;
  a.a_routed = x_perm != nullptr ? x_perm : x;
  a.gather_idx = x_perm != nullptr ? nullptr : perm_token;
  a.expert_offsets = expert_offsets;
  a.budget = budget_max;
  a.budget_hint = expected;
  a.W13 = W13;
  a.W2 = W2;
  a.h = at<uint16_t>(ws, L.h);
  a.y_perm = y_perm;
  a.x_shared = shape->S > 0 ? x : nullptr;
  a.Wsh13 = Wsh13;
  a.Wsh2 = Wsh2;
  a.h_sh = at<uint16_t>(ws, L.h_sh);
  a.y_shared = y_shared;
  a.dev_status = dev_status;
  a.done = at<int32_t>(ws, L.gemm_done);
  a.stream = st;
  r = launch_ffn(a);
  if (r != MOE_OK) return r;
  return launch_moe_combine(shape, y_perm, pair_pos, topk_score, n_sel, y_shared, residual, budget_max, out, st);
}

moe_status moe_selftest_wait_timeout(const moe_shape* shape, const int32_t* expert_offsets, int64_t budget,
                                     const uint16_t* W2, uint16_t* y_perm, int64_t wait_limit_clk, int32_t* dev_status,
                                     void* ws, size_t ws_bytes, void* stream) {
  ApiRange nvtx_range("moe_selftest_wait_timeout");
  if (!shape_ok(shape) || !expert_offsets || !W2 || !y_perm || !dev_status || !ws) return MOE_ERR_ARG;
  if (!aligned16(W2) || !aligned16(y_perm) || !aligned16(ws)) return MOE_ERR_ARG;
  if (budget < 1 || budget > (int64_t)shape->K_orig * shape->T) return MOE_ERR_BUDGET;
  if (wait_limit_clk < 1000 || wait_limit_clk > 2000000000ll) return MOE_ERR_ARG;
  const WsLayout L = ws_layout(shape, budget);
  if (ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  FfnArgs a;
  a.s = shape;
  a.a_routed = at<uint16_t>(ws, L.x_perm);   // never read: GEMM-1 is not launched
  a.expert_offsets = expert_offsets;
  a.budget = budget;
  a.W13 = W2;                                 // only a tensor map is built from it
  a.W2 = W2;
  a.h = at<uint16_t>(ws, L.h);
  a.y_perm = y_perm;
  a.dev_status = dev_status;
  a.done = at<int32_t>(ws, L.gemm_done);      // cleared by launch_ffn, then never incremented
  a.wait_limit_clk = wait_limit_clk;
  a.gemm2_only = true;
  a.stream = (cudaStream_t)stream;
  return launch_ffn(a);
}

moe_status moe_select_top_p(const moe_shape* shape, const float* topk_score, float P, int32_t* n_sel, int32_t* total,
                            int32_t* dev_status, void* stream) {
  ApiRange nvtx_range("moe_select_top_p");
  if (!shape_ok(shape) || !topk_score || !n_sel || !dev_status || !(P == P)) return MOE_ERR_ARG;
  return launch_token_rule_select(shape, topk_score, 0, P, n_sel, total, dev_status, (cudaStream_t)stream);
}

moe_status moe_select_rel_threshold(const moe_shape* shape, const float* topk_score, float beta, int32_t* n_sel,
                                    int32_t* total, int32_t* dev_status, void* stream) {
  ApiRange nvtx_range("moe_select_rel_threshold");
  if (!shape_ok(shape) || !topk_score || !n_sel || !dev_status || !(beta >= 0.f)) return MOE_ERR_ARG;
  return launch_token_rule_select(shape, topk_score, 1, beta, n_sel, total, dev_status, (cudaStream_t)stream);
}

moe_status moe_rmsnorm(const moe_shape* shape, const uint16_t* x, uint16_t* out, void* stream) {
  ApiRange nvtx_range("moe_rmsnorm");
  if (!shape_ok(shape) || !x || !out || !aligned16(x) || !aligned16(out)) return MOE_ERR_ARG;
  return launch_rmsnorm(shape, x, out, (cudaStream_t)stream);
}

moe_status moe_profile_enable(int32_t on) {
  if (on && !g_prof_on) {
    for (int i = 0; i <= kProfStages; ++i)
      if (cudaEventCreate(&g_prof_ev[i]) != cudaSuccess) return MOE_ERR_CUDA;
    g_prof_on = true;
  } else if (!on && g_prof_on) {
    g_prof_on = false;
    for (int i = 0; i <= kProfStages; ++i) cudaEventDestroy(g_prof_ev[i]);
  }
  return MOE_OK;
}

moe_status moe_profile_read(float* stage_ms) {
  if (!g_prof_on || !stage_ms) return MOE_ERR_ARG;
  if (cudaEventSynchronize(g_prof_ev[kProfStages]) != cudaSuccess) return MOE_ERR_CUDA;
  for (int i = 0; i < kProfStages; ++i)
    if (cudaEventElapsedTime(&stage_ms[i], g_prof_ev[i], g_prof_ev[i + 1]) != cudaSuccess) return MOE_ERR_CUDA;
  return MOE_OK;
}

moe_status moe_layer_intermediates(const moe_shape* shape, int64_t budget_max, void* ws, size_t ws_bytes,
                                   int32_t** topk_idx, float** topk_score, int32_t** n_sel, int32_t** expert_offsets,
                                   int32_t** perm_token, int32_t** pair_pos, uint16_t** y_perm) {
  if (!shape_ok(shape) || !ws) return MOE_ERR_ARG;
  if (budget_max < 0 || budget_max > (int64_t)shape->K_orig * shape->T) return MOE_ERR_BUDGET;
  const WsLayout L = ws_layout(shape, budget_max);
  if (ws_bytes < L.total) return MOE_ERR_WORKSPACE;
  if (topk_idx) *topk_idx = at<int32_t>(ws, L.topk_idx);
  if (topk_score) *topk_score = at<float>(ws, L.topk_score);
  if (n_sel) *n_sel = at<int32_t>(ws, L.n_sel);
  if (expert_offsets) *expert_offsets = at<int32_t>(ws, L.expert_offsets);
  if (perm_token) *perm_token = at<int32_t>(ws, L.perm_token);
  if (pair_pos) *pair_pos = at<int32_t>(ws, L.pair_pos);
  if (y_perm) *y_perm = at<uint16_t>(ws, L.y_perm);
  return MOE_OK;
}

}  // extern "C"
