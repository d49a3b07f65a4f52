// moe_permute: lists the kept (token, expert) pairs expert-ascending, token-ascending inside an
// expert, without any order-dependent atomics, so the result is the unique stable placement.
//
// Tokens are cut into segments of 32 (one warp, lane = token).  A token's experts are distinct,
// so inside a segment expert e is hit by at most one pair per lane and a 32-bit mask per expert
// (built with shared-memory atomicOr, which commutes) carries both the count (popc) and every
// pair's rank (popc of the lower lanes).  Three small kernels:
//   count : seg_counts[e][seg] = popc(mask[e])
//   scan  : exclusive scan of seg_counts in (expert, segment) order -> base position of every
//           (expert, segment) run; expert_offsets[e] is the base of (e, 0)
//   place : pos = base[e][seg] + rank -> perm_token, perm_weight, pair_pos
// and a row gather x_perm[p] = x[perm_token[p]] with 128-bit loads and stores.
#include "routing.cuh"

namespace allocmoe {

constexpr int kPermWarps = 8;

__global__ void __launch_bounds__(kPermWarps * 32)
permute_count_kernel(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ n_sel, int T, int N,
                     int K_orig, int nseg, int32_t* __restrict__ seg_counts) {
  __shared__ uint32_t masks[kPermWarps][kMaxExperts];
  const int warp = threadIdx.x >> 5;
  const int seg = blockIdx.x * kPermWarps + warp;
  pdl_prologue_done();
  if (seg >= nseg) return;
  permute_count_warp(masks[warp], topk_idx, n_sel, seg, T, N, K_orig, nseg, seg_counts);
}

// One CTA.  In-place exclusive scan of seg_counts (N*nseg ints, expert-major).
__global__ void __launch_bounds__(1024, 1)
permute_scan_kernel(int32_t* __restrict__ seg_counts, int N, int nseg, long long budget, int exact,
                    int32_t* __restrict__ expert_offsets, int32_t* dev_status) {
  __shared__ int scan_ws[33];
  pdl_prologue_done();
  permute_scan_block(seg_counts, N, nseg, budget, exact != 0, expert_offsets, dev_status, scan_ws);
}

__global__ void __launch_bounds__(kPermWarps * 32)
permute_place_kernel(const int32_t* __restrict__ topk_idx, const float* __restrict__ topk_score,
                     const int32_t* __restrict__ n_sel, int T, int N, int K_orig, int nseg,
                     const int32_t* __restrict__ seg_base, long long budget, int32_t* __restrict__ perm_token,
                     float* __restrict__ perm_weight, int32_t* __restrict__ pair_pos) {
  __shared__ uint32_t masks[kPermWarps][kMaxExperts];
  const int warp = threadIdx.x >> 5;
  const int seg = blockIdx.x * kPermWarps + warp;
  pdl_prologue_done();
  if (seg >= nseg) return;
  permute_place_warp(masks[warp], topk_idx, topk_score, n_sel, seg, T, N, K_orig, nseg, seg_base, budget, perm_token,
                     perm_weight, pair_pos);
}

// x_perm[p, :] = x[perm_token[p], :]; one CTA per row, 16 bytes per thread per step.  rows_dev (optional):
// the list's length as the device knows it (expert_offsets[N]) when `rows` is only an upper bound.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ perm_token, int T, int row_vec,
                   long long rows, const int32_t* __restrict__ rows_dev, uint4* __restrict__ x_perm, int32_t* dev_status) {
  pdl_prologue_done();
  if (rows_dev != nullptr) rows = min(rows, (long long)max(*rows_dev, 0));
  for (long long p = blockIdx.x; p < rows; p += gridDim.x) {
    const int t = clamp_index(perm_token[p], 0, T - 1, dev_status);
    const uint4* src = x + (long long)t * row_vec;
    uint4* dst = x_perm + p * row_vec;
    for (int c = threadIdx.x; c < row_vec; c += blockDim.x) dst[c] = __ldg(src + c);
  }
}

}  // namespace allocmoe

using namespace allocmoe;

moe_status launch_gather_rows(const moe_shape* s, const uint16_t* x, const int32_t* perm_token, int64_t budget,
                              const int32_t* rows_dev, uint16_t* x_perm, int32_t* dev_status, cudaStream_t stream) {
  const int row_vec = s->H / 8;
  const long long g = budget < (1ll << 20) ? budget : (1ll << 20);
  return launch_dependent(gather_rows_kernel, dim3((unsigned)g), dim3(256), 0, stream, 1, reinterpret_cast<const uint4*>(x),
                          perm_token, (int)s->T, row_vec, (long long)budget, rows_dev,
                          reinterpret_cast<uint4*>(x_perm), dev_status) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

size_t permute_ws_ints(const moe_shape* s) { return (size_t)s->N * ((s->T + 31) / 32); }

moe_status launch_moe_permute(const moe_shape* s, const uint16_t* x, const int32_t* topk_idx, const float* topk_score,
                              const int32_t* n_sel, int64_t budget, int32_t* expert_offsets, int32_t* perm_token,
                              float* perm_weight, int32_t* pair_pos, uint16_t* x_perm, int32_t* dev_status,
                              int32_t* seg_counts, bool exact, cudaStream_t stream) {
  const int nseg = (s->T + 31) / 32;
  const int grid = (nseg + kPermWarps - 1) / kPermWarps;
  bool ok = launch_dependent(permute_count_kernel, dim3((unsigned)grid), dim3(kPermWarps * 32), 0, stream, 1, topk_idx, n_sel,
                             (int)s->T, (int)s->N, (int)s->K_orig, nseg, seg_counts) == cudaSuccess;
  ok = ok && launch_dependent(permute_scan_kernel, dim3(1), dim3(1024), 0, stream, 1, seg_counts, (int)s->N, nseg,
                              (long long)budget, exact ? 1 : 0, expert_offsets, dev_status) == cudaSuccess;
  ok = ok && launch_dependent(permute_place_kernel, dim3((unsigned)grid), dim3(kPermWarps * 32), 0, stream, 1, topk_idx,
                              topk_score, n_sel, (int)s->T, (int)s->N, (int)s->K_orig, nseg,
                              static_cast<const int32_t*>(seg_counts), (long long)budget, perm_token, perm_weight,
                              pair_pos) == cudaSuccess;
  if (!ok) return MOE_ERR_CUDA;
  if (x_perm != nullptr && budget > 0)
    return launch_gather_rows(s, x, perm_token, budget, exact ? nullptr : expert_offsets + s->N, x_perm, dev_status, stream);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------
// moe_permute_static: moe_permute for callers that cannot allocate device memory.
//
// The per-(expert, 32-token segment) counters that moe_permute keeps in the caller's workspace
// live here in a fixed array inside the library image instead.  Each GPU that loads the library
// carries these 256 KB until the process exits.
#include <mutex>

#include <nvtx3/nvToolsExt.h>

#include "shape_check.h"

namespace {

constexpr int kStaticSegCounts = 65536;   // N * ceil(T/32) may not exceed this (256 KB of int32)
static __device__ __align__(256) int32_t g_static_seg_counts[kStaticSegCounts];

int32_t* g_static_seg_ptr[allocmoe::kMaxDevices] = {};
std::mutex g_static_mutex;

// In host code the array's name is only a handle; the address a kernel can use has to be asked for
// while the owning device is current.  Done once per device, on that device's first call.
moe_status static_scratch(int32_t** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= allocmoe::kMaxDevices) return MOE_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_seg_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_seg_counts) != cudaSuccess || p == nullptr) return MOE_ERR_CUDA;
    g_static_seg_ptr[dev] = static_cast<int32_t*>(p);
  }
  *out = g_static_seg_ptr[dev];
  return MOE_OK;
}

}  // namespace

extern "C" moe_status moe_permute_static(const moe_shape* shape, const uint16_t* x, const int32_t* topk_idx,
                                         const float* topk_score, const int32_t* n_sel, int64_t budget,
                                         int32_t* expert_offsets, int32_t* perm_token, float* perm_weight,
                                         int32_t* pair_pos, uint16_t* x_perm, int32_t* dev_status, void* stream) {
  nvtxRangePushA("moe_permute_static");
  struct Pop { ~Pop() { nvtxRangePop(); } } pop;
  const moe_shape* s = shape;
  if (!allocmoe::shape_ok(s)) return MOE_ERR_ARG;   // the same shapes as moe_permute accepts
  if (!topk_idx || !topk_score || !n_sel || !expert_offsets || !perm_token || !perm_weight || !pair_pos || !dev_status)
    return MOE_ERR_ARG;
  if (x_perm != nullptr && (!x || !allocmoe::aligned16(x) || !allocmoe::aligned16(x_perm))) return MOE_ERR_ARG;
  if (budget < (int64_t)s->K_base * s->T || budget > (int64_t)s->K_orig * s->T) return MOE_ERR_BUDGET;
  // the fixed array bounds the problem size: refuse anything larger, touch nothing
  if ((long long)s->N * ((s->T + 31) / 32) > (long long)kStaticSegCounts) return MOE_ERR_WORKSPACE;
  int32_t* seg_counts = nullptr;
  const moe_status st = static_scratch(&seg_counts);
  if (st != MOE_OK) return st;
  // Every counter a call reads is written by its own count kernel first, so whatever an earlier
  // call left in the array needs no clearing.
  return launch_moe_permute(s, x, topk_idx, topk_score, n_sel, budget, expert_offsets, perm_token, perm_weight,
                            pair_pos, x_perm, dev_status, seg_counts, true, (cudaStream_t)stream);
}
