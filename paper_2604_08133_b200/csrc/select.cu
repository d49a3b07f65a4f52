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
#include "routing.cuh"

namespace allocmoe {

__global__ void __launch_bounds__(kSelThreads, 1)
alloc_t_select_kernel(const float* __restrict__ topk_score, int T, int K_orig, int K_base, long long R,
                      int use_smem_keys, int32_t* __restrict__ n_sel, int32_t* dev_status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_prologue_done();
  alloc_t_select_block(smem_raw, topk_score, T, K_orig, K_base, R, use_smem_keys, n_sel, dev_status);
}

// ------------------------------------------------------------------------------------------------
// The two token-level rules the paper compares Alloc-T with (Sec. 2; App. A.1), as selection kernels with
// the same output (n_sel) so that the rest of the layer can run on them for a speed comparison.  Both look at
// one token at a time -- no pool, no budget: the kept total follows from the threshold, which those methods
// calibrate off line.
//   mode 0, Top-P count (the Dynamic-MoE baseline):  n_t = the smallest n >= 1 whose cumulative score
//           s[t,0] + ... + s[t,n-1] reaches P, K_orig if none does; fp32 sums in column order.
//   mode 1, relative threshold (the NAEE baseline extended to Top-K):  column j >= 1 is skipped when
//           s[t,j] < beta * s[t,0] (fp32 product); rows are sorted, so n_t = 1 + the columns 1.. not skipped.
// One thread per token; `total` (optional) receives sum n_t by one integer atomic per CTA.
__global__ void __launch_bounds__(256)
token_rule_select_kernel(const float* __restrict__ topk_score, int T, int K_orig, int mode, float thr,
                         int32_t* __restrict__ n_sel, int32_t* __restrict__ total, int32_t* dev_status) {
  __shared__ int warp_sum[8];
  pdl_prologue_done();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  int n = 0;
  if (t < T) {
    float s[16];
    bool bad = false;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      s[j] = j < K_orig ? topk_score[(long long)t * K_orig + j] : 0.f;
      bad |= (__float_as_uint(s[j]) >= 0x7F800000u);      // NaN, Inf or negative
    }
    if (bad) set_dev_status(dev_status, MOE_ERR_NONFINITE);
    if (mode == 0) {
      float cum = 0.f;
      n = K_orig;
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (j < K_orig) {
          cum = __fadd_rn(cum, s[j]);
          if (cum >= thr && n == K_orig) n = j + 1;
        }
    } else {
      const float cut = __fmul_rn(thr, s[0]);
      n = 1;
#pragma unroll
      for (int j = 1; j < 16; ++j)
        if (j < K_orig && n == j && s[j] >= cut) n = j + 1;   // a prefix: stops at the first skipped column
    }
    n_sel[t] = n;
  }
  if (total != nullptr) {
    int v = n;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
      int a = 0;
      for (int w = 0; w < 8; ++w) a += warp_sum[w];
      atomicAdd(total, a);
    }
  }
}

}  // namespace allocmoe

using namespace allocmoe;

moe_status launch_token_rule_select(const moe_shape* s, const float* topk_score, int mode, float thr, int32_t* n_sel,
                                    int32_t* total, int32_t* dev_status, cudaStream_t stream) {
  const unsigned grid = (unsigned)((s->T + 255) / 256);
  return launch_dependent(token_rule_select_kernel, dim3(grid), dim3(256), 0, stream, 1, topk_score, (int)s->T,
                          (int)s->K_orig, mode, thr, n_sel, total, dev_status) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

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
  static PerDeviceOnce attr_set;
  if (!ensure_dynamic_smem(alloc_t_select_kernel, sizeof(SelectSmem) + (size_t)kSelMaxSmemKeys * 4, attr_set))
    return MOE_ERR_CUDA;
  return launch_dependent(alloc_t_select_kernel, dim3(1), dim3(kSelThreads), smem, stream, 1, topk_score, (int)s->T,
                          (int)s->K_orig, (int)s->K_base, R, use_smem, n_sel, dev_status) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}
