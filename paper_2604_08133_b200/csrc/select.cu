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
#include <cooperative_groups.h>

#include "routing.cuh"

namespace cg = cooperative_groups;

namespace allocmoe {

__global__ void __launch_bounds__(kSelThreads, 1)
alloc_t_select_kernel(const float* __restrict__ topk_score, int T, int K_orig, int K_base, long long R,
                      int use_smem_keys, int32_t* __restrict__ n_sel, int32_t* dev_status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_prologue_done();
  alloc_t_select_block(smem_raw, topk_score, T, K_orig, K_base, R, use_smem_keys, n_sel, dev_status);
}

// ------------------------------------------------------------------------------------------------
// Pools beyond one CTA's shared memory (more than kSelMaxSmemKeys keys: the batch-wide selection over several
// ranks' tokens, or a single batch of tens of thousands of tokens): the same exact radix select on a thread-block
// cluster.  CTA r stages the keys of a contiguous range of tokens in its own shared memory, histograms them per
// pass, the CTAs read one another's 256-bin histograms through distributed shared memory and all take the same
// digit decision; ties are handed out in flat order by a block scan of per-thread tie counts plus the tie totals
// of the lower-ranked CTAs (ranks follow token order).  Same result as the one-CTA kernel, bit for bit.
struct SelectClusterSmem {
  int warp_hist[kSelWarps][256];
  int hist[2][256];        // this CTA's histogram of the current digit (read by the peers), double-buffered by pass
  int ghist[256];          // the cluster's
  int scan_ws[33];
  uint32_t prefix;
  int remaining;
  int bucket;
  int eq_total;            // keys equal to tau among this CTA's tokens (read by the peers)
};

__global__ void __launch_bounds__(kSelThreads, 1)
alloc_t_select_cluster_kernel(const float* __restrict__ topk_score, int T, int K_orig, int K_base, long long R,
                              int tokens_per_cta, int32_t* __restrict__ n_sel, int32_t* dev_status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SelectClusterSmem& sm = *reinterpret_cast<SelectClusterSmem*>(smem_raw);
  uint32_t* skeys = reinterpret_cast<uint32_t*>(smem_raw + sizeof(SelectClusterSmem));
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank(), n_ranks = (int)cluster.num_blocks();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Kr = K_orig - K_base;
  const int t_begin = min(T, rank * tokens_per_cta), t_end = min(T, t_begin + tokens_per_cta);
  const int Tl = t_end - t_begin;                       // this CTA's tokens
  const int Pl = Tl * Kr;                               // and keys (<= kSelMaxSmemKeys by the launcher's choice)
  const uint32_t* bits = reinterpret_cast<const uint32_t*>(topk_score);
  pdl_prologue_done();

  // stage and validate this CTA's keys (a NaN, an Inf or a negative score has bits >= 0x7F800000)
  bool bad = false;
  for (int i = tid; i < Tl; i += kSelThreads) {
    const int t = t_begin + i;
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (j >= K_base && j < K_orig) {
        const uint32_t k = bits[(long long)t * K_orig + j];
        bad |= (k >= 0x7F800000u);
        skeys[i * Kr + (j - K_base)] = k;
      }
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
    for (int i = tid; i < Pl; i += kSelThreads) {
      const uint32_t k = skeys[i];
      if ((k & prefix_mask) == prefix) atomicAdd(&sm.warp_hist[warp][(k >> shift) & 255u], 1);
    }
    __syncthreads();
    if (tid < 256) {
      int a = 0;
#pragma unroll 8
      for (int w = 0; w < kSelWarps; ++w) a += sm.warp_hist[w][tid];
      sm.hist[pass & 1][tid] = a;
    }
    cluster.sync();   // every CTA's histogram of this pass is complete (and the previous pass's reads are over)
    if (tid < 256) {
      int a = 0;
      for (int r = 0; r < n_ranks; ++r) a += cluster.map_shared_rank(&sm.hist[pass & 1][0], r)[tid];
      sm.ghist[tid] = a;
    }
    __syncthreads();
    if (warp == 0) radix_choose_digit(sm.ghist, shift, prefix, &sm.prefix, &sm.remaining, &sm.bucket);
    prefix_mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t tau = sm.prefix;
  const int need_eq = sm.remaining;       // how many keys equal to tau are kept (>= 1)

  // threads own contiguous token ranges of the CTA's range, so thread order is flat order
  const int tpt = (Tl + kSelThreads - 1) / kSelThreads;
  const int i_lo = min(Tl, tid * tpt), i_hi = min(Tl, i_lo + tpt);
  if (sm.bucket == need_eq) {             // every key equal to tau is kept: no order among ties matters
    for (int i = i_lo; i < i_hi; ++i) {
      int n = K_base;
      for (int j = 0; j < Kr; ++j) n += (skeys[i * Kr + j] >= tau);
      n_sel[t_begin + i] = n;
    }
  } else {
    int my_eq = 0;
    for (int i = i_lo; i < i_hi; ++i)
      for (int j = 0; j < Kr; ++j) my_eq += (skeys[i * Kr + j] == tau);
    int cta_eq;
    int ties_before = block_exclusive_scan(my_eq, sm.scan_ws, &cta_eq);
    if (tid == 0) sm.eq_total = cta_eq;
    cluster.sync();
    for (int r = 0; r < rank; ++r) ties_before += *cluster.map_shared_rank(&sm.eq_total, r);
    for (int i = i_lo; i < i_hi; ++i) {
      int gt = 0, eq = 0;
      for (int j = 0; j < Kr; ++j) {
        const uint32_t k = skeys[i * Kr + j];
        gt += (k > tau);
        eq += (k == tau);
      }
      n_sel[t_begin + i] = K_base + gt + min(eq, max(0, need_eq - ties_before));
      ties_before += eq;
    }
  }
  cluster.sync();    // no CTA leaves while a peer may still read its shared memory
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
  // a pool too large for one CTA's shared memory goes to a cluster of up to 8 CTAs, each staging its share
  if (R > 0 && P > kSelMaxSmemKeys && P <= 8ll * kSelMaxSmemKeys) {
    const int Kr = s->K_orig - s->K_base;
    int n_ctas = (int)((P + kSelMaxSmemKeys - 1) / kSelMaxSmemKeys);
    int tokens_per_cta = (s->T + n_ctas - 1) / n_ctas;
    while ((long long)tokens_per_cta * Kr > kSelMaxSmemKeys) {     // rounding up must not overflow a CTA's share
      ++n_ctas;
      tokens_per_cta = (s->T + n_ctas - 1) / n_ctas;
    }
    if (n_ctas <= 8) {
      const size_t csmem = sizeof(SelectClusterSmem) + (size_t)tokens_per_cta * Kr * 4;
      static PerDeviceOnce cattr_set;
      if (!ensure_dynamic_smem(alloc_t_select_cluster_kernel, sizeof(SelectClusterSmem) + (size_t)kSelMaxSmemKeys * 4, cattr_set))
        return MOE_ERR_CUDA;
      return launch_dependent_cluster(alloc_t_select_cluster_kernel, dim3((unsigned)n_ctas), dim3(kSelThreads), csmem, stream,
                                      dim3((unsigned)n_ctas, 1, 1), topk_score, (int)s->T, (int)s->K_orig, (int)s->K_base, R,
                                      tokens_per_cta, n_sel, dev_status) == cudaSuccess
                 ? MOE_OK
                 : MOE_ERR_CUDA;
    }
  }
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
