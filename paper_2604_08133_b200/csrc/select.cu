// alloc_t_select: Alloc-T's token-level redistribution (Sec. 3.3, procedure paragraph).
//
// Every token keeps its first K_base columns.  The other P = T*(K_orig-K_base) scores form one
// pool; the R = budget - K_base*T largest are kept.  The kernel finds the exact R-th largest key
// tau with a most-significant-digit-first radix select (4 passes of 8 bits over the IEEE bit
// patterns, which order like the values for non-negative floats), then counts per token the
// keys above tau and hands the remaining places to keys equal to tau in ascending flat index.
// Because rows are sorted descending, the kept pairs of a token are its first n_sel[t] columns.
//
// One CTA of 1024 threads: the pool is at most a few tens of thousands of keys (80 KB at
// T=4096, K_orig=6), far below what keeps a GPU busy, so the cost is latency.  Keys are staged
// in shared memory when they fit and re-read from global memory (L2) otherwise.
#include "common.cuh"

namespace allocmoe {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelMaxSmemKeys = 40960;   // 160 KB of keys + 32 KB of per-warp histograms

struct SelectSmem {
  int warp_hist[kSelWarps][256];
  int hist[256];
  int scan_ws[33];
  uint32_t prefix;
  int remaining;
};

__global__ void __launch_bounds__(kSelThreads, 1)
alloc_t_select_kernel(const float* __restrict__ topk_score, int T, int K_orig, int K_base, long long R,
                      int use_smem_keys, int32_t* __restrict__ n_sel, int32_t* dev_status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SelectSmem& sm = *reinterpret_cast<SelectSmem*>(smem_raw);
  uint32_t* skeys = reinterpret_cast<uint32_t*>(smem_raw + sizeof(SelectSmem));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Kr = K_orig - K_base;
  const long long P = (long long)T * Kr;
  const uint32_t* bits = reinterpret_cast<const uint32_t*>(topk_score);

  if (R <= 0 || Kr == 0) {   // nothing to redistribute: plain Top-K_base
    for (int t = tid; t < T; t += kSelThreads) n_sel[t] = K_base;
    return;
  }

  // Stage the pool and validate: a NaN, an Inf or a negative score has bits >= 0x7F800000.
  bool bad = false;
  for (long long i = tid; i < P; i += kSelThreads) {
    const int t = (int)(i / Kr), j = K_base + (int)(i % Kr);
    const uint32_t k = bits[(long long)t * K_orig + j];
    bad |= (k >= 0x7F800000u);
    if (use_smem_keys) skeys[i] = k;
  }
  if (bad) set_dev_status(dev_status, MOE_ERR_NONFINITE);
  if (tid == 0) { sm.prefix = 0u; sm.remaining = (int)R; }
  __syncthreads();

  uint32_t prefix_mask = 0u;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int b = lane; b < 256; b += 32) sm.warp_hist[warp][b] = 0;
    __syncwarp();
    const uint32_t prefix = sm.prefix;
    for (long long i = tid; i < P; i += kSelThreads) {
      uint32_t k;
      if (use_smem_keys) {
        k = skeys[i];
      } else {
        const int t = (int)(i / Kr), j = K_base + (int)(i % Kr);
        k = bits[(long long)t * K_orig + j];
      }
      if ((k & prefix_mask) == prefix) atomicAdd(&sm.warp_hist[warp][(k >> shift) & 255u], 1);
    }
    __syncthreads();
    if (tid < 256) {
      int s = 0;
#pragma unroll 8
      for (int w = 0; w < kSelWarps; ++w) s += sm.warp_hist[w][tid];
      sm.hist[tid] = s;
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns digits 255-8l .. 248-8l (descending); find the digit where the running count
      // from the top first reaches `remaining`.
      int c[8], lsum = 0;
#pragma unroll
      for (int q = 0; q < 8; ++q) { c[q] = sm.hist[255 - (lane * 8 + q)]; lsum += c[q]; }
      int incl = lsum;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        int o = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += o;
      }
      int above = incl - lsum;           // keys in strictly higher digits than this lane's
      const int rem = sm.remaining;
      if (above < rem && rem <= incl) {  // exactly one lane
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          if (above < rem && rem <= above + c[q]) {
            sm.prefix = prefix | ((uint32_t)(255 - (lane * 8 + q)) << shift);
            sm.remaining = rem - above;
            above = rem;                 // stop
          } else {
            above += c[q];
          }
        }
      }
    }
    prefix_mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t tau = sm.prefix;
  const int need_eq = sm.remaining;       // how many keys equal to tau are kept (>= 1)

  // Per token: keys above tau, then ties in flat order.  Threads own contiguous token ranges.
  const int tpt = (T + kSelThreads - 1) / kSelThreads;
  const int t_lo = min(T, tid * tpt), t_hi = min(T, t_lo + tpt);
  int my_eq = 0;
  for (int t = t_lo; t < t_hi; ++t)
    for (int j = K_base; j < K_orig; ++j) my_eq += (bits[(long long)t * K_orig + j] == tau);
  int total_eq;
  int ties_before = block_exclusive_scan(my_eq, sm.scan_ws, &total_eq);
  for (int t = t_lo; t < t_hi; ++t) {
    int gt = 0, eq = 0;
    for (int j = K_base; j < K_orig; ++j) {
      const uint32_t k = bits[(long long)t * K_orig + j];
      gt += (k > tau);
      eq += (k == tau);
    }
    const int room = max(0, need_eq - ties_before);
    n_sel[t] = K_base + gt + min(eq, room);
    ties_before += eq;
  }
}

}  // namespace allocmoe

using namespace allocmoe;

size_t select_dynamic_smem(long long P, int* use_smem_keys) {
  *use_smem_keys = (P <= kSelMaxSmemKeys) ? 1 : 0;
  return sizeof(SelectSmem) + (*use_smem_keys ? (size_t)P * 4 : 0);
}

moe_status launch_alloc_t_select(const moe_shape* s, const float* topk_score, int64_t budget, int32_t* n_sel,
                                 int32_t* dev_status, cudaStream_t stream) {
  const long long R = budget - (long long)s->K_base * s->T;
  const long long P = (long long)s->T * (s->K_orig - s->K_base);
  int use_smem = 0;
  const size_t smem = select_dynamic_smem(P, &use_smem);
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(alloc_t_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(sizeof(SelectSmem) + (size_t)kSelMaxSmemKeys * 4)) != cudaSuccess)
      return MOE_ERR_CUDA;
    attr_done = true;
  }
  alloc_t_select_kernel<<<1, kSelThreads, smem, stream>>>(topk_score, s->T, s->K_orig, s->K_base, R, use_smem, n_sel,
                                                          dev_status);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
