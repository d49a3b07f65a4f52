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
  static PerDeviceOnce attr_set;
  if (!ensure_dynamic_smem(alloc_t_select_kernel, sizeof(SelectSmem) + (size_t)kSelMaxSmemKeys * 4, attr_set))
    return MOE_ERR_CUDA;
  return launch_dependent(alloc_t_select_kernel, dim3(1), dim3(kSelThreads), smem, stream, 1, topk_score, (int)s->T,
                          (int)s->K_orig, (int)s->K_base, R, use_smem, n_sel, dev_status) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}
