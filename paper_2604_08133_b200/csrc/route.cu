// Fused routing step of moe_layer_forward: Alloc-T selection (Sec. 3.3) and the permutation's
// count / scan / place in ONE launch of one CTA.
//
// Each of the four steps is a few microseconds of work for a single CTA at the sizes a layer call
// sees (at most a few tens of thousands of (token, expert) pairs); launched separately they cost
// four launch latencies and three trips of their small intermediates through L2.  Here n_sel goes
// from the selection to the permutation through the CTA's own global writes (ordered by the block
// barrier), and the per-(expert, 32-token segment) counters live in the shared memory that held
// the selection's key pool.  The stand-alone entry points (alloc_t_select, moe_permute) keep their
// own kernels; both paths run the same device functions (routing.cuh) and give identical results.
#include "routing.cuh"

namespace allocmoe {

constexpr int kRouteWarps = kSelThreads / 32;

// Dynamic shared memory: [SelectSmem][pool: keys during the selection, then seg_counts].
// The per-warp masks of the permutation reuse SelectSmem::warp_hist (32 warps x 256 ints >= 32 x 128).
__global__ void __launch_bounds__(kSelThreads, 1)
moe_route_kernel(const float* __restrict__ topk_score, const int32_t* __restrict__ topk_idx, int T, int N, int K_orig,
                 int K_base, long long budget, int use_smem_keys, int32_t* __restrict__ n_sel,
                 int32_t* __restrict__ expert_offsets, int32_t* __restrict__ perm_token,
                 float* __restrict__ perm_weight, int32_t* __restrict__ pair_pos, int32_t* dev_status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SelectSmem& sm = *reinterpret_cast<SelectSmem*>(smem_raw);
  int32_t* seg_counts = reinterpret_cast<int32_t*>(smem_raw + sizeof(SelectSmem));
  const int warp = threadIdx.x >> 5;
  const int nseg = (T + 31) / 32;
  pdl_prologue_done();

  alloc_t_select_block(smem_raw, topk_score, T, K_orig, K_base, budget - (long long)K_base * T, use_smem_keys, n_sel,
                       dev_status);   // ends with a block barrier: n_sel is visible, the pool is free

  // Every warp owns at most one 32-token segment here (moe_route_fits), so the masks and expert ids
  // built for the count are still there for the placement: nothing is loaded twice.
  uint32_t* mask = reinterpret_cast<uint32_t*>(sm.warp_hist[warp]);
  const int lane = threadIdx.x & 31;
  const int seg = warp;
  int e_loc[16], n = 0;
  if (seg < nseg) {
    build_masks(mask, topk_idx, n_sel, seg * 32 + lane, T, N, K_orig, lane, e_loc, n);
    for (int e = lane; e < N; e += 32) seg_counts[(long long)e * nseg + seg] = __popc(mask[e]);
  }
  __syncthreads();
  permute_scan_block(seg_counts, N, nseg, budget, expert_offsets, dev_status, sm.scan_ws);
  __syncthreads();
  if (seg < nseg)
    permute_place_from_masks(mask, e_loc, n, topk_score, seg, T, K_orig, nseg, seg_counts, budget, perm_token,
                             perm_weight, pair_pos);
}

}  // namespace allocmoe

using namespace allocmoe;

// True when the fused kernel is the better choice: every warp of its one CTA gets at most one
// 32-token segment (T <= 1024; beyond that the multi-CTA count and place kernels win back more than
// the launches cost), and the permutation's counters fit the shared-memory pool.
bool moe_route_fits(const moe_shape* s) {
  const long long nseg = (s->T + 31) / 32;
  return nseg <= kRouteWarps && (long long)s->N * nseg <= (long long)kSelMaxSmemKeys;
}

moe_status launch_moe_route(const moe_shape* s, const float* topk_score, const int32_t* topk_idx, int64_t budget,
                            int32_t* n_sel, int32_t* expert_offsets, int32_t* perm_token, float* perm_weight,
                            int32_t* pair_pos, int32_t* dev_status, cudaStream_t stream) {
  const long long P = (long long)s->T * (s->K_orig - s->K_base);
  const int use_smem_keys = (P <= kSelMaxSmemKeys) ? 1 : 0;
  const long long counters = (long long)s->N * ((s->T + 31) / 32);
  const long long pool_ints = (use_smem_keys && P > counters) ? P : counters;
  const size_t smem = sizeof(SelectSmem) + (size_t)pool_ints * 4;
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(moe_route_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(sizeof(SelectSmem) + (size_t)kSelMaxSmemKeys * 4)) != cudaSuccess)
      return MOE_ERR_CUDA;
    attr_done = true;
  }
  return launch_dependent(moe_route_kernel, dim3(1), dim3(kSelThreads), smem, stream, 1, topk_score, topk_idx, (int)s->T,
                          (int)s->N, (int)s->K_orig, (int)s->K_base, (long long)budget, use_smem_keys, n_sel,
                          expert_offsets, perm_token, perm_weight, pair_pos, dev_status) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}
