// Fused routing step of moe_layer_forward: Alloc-T selection (Sec. 3.3) and the permutation's
// count / scan / place in ONE launch -- of one CTA up to 1024 tokens (moe_route_kernel), of a
// thread-block cluster of 1024-token CTAs up to 8192 tokens (moe_route_cluster_kernel, below).
//
// Each of the four steps is a few microseconds of work for a single CTA at the sizes a layer call
// sees (at most a few tens of thousands of (token, expert) pairs); launched separately they cost
// four launch latencies and three trips of their small intermediates through L2.  Here n_sel goes
// from the selection to the permutation through the CTA's own global writes (ordered by the block
// barrier), and the per-(expert, 32-token segment) counters live in the shared memory that held
// the selection's key pool.  The stand-alone entry points (alloc_t_select, moe_permute) keep their
// own kernels; both paths run the same device functions (routing.cuh) and give identical results.
#include <cooperative_groups.h>

#include "routing.cuh"

namespace cg = cooperative_groups;

namespace allocmoe {

constexpr int kRouteWarps = kSelThreads / 32;

// Dynamic shared memory: [SelectSmem][pool: keys during the selection, then seg_counts].
// The per-warp masks of the permutation reuse SelectSmem::warp_hist (32 warps x 256 ints >= 32 x 128).
__global__ void __launch_bounds__(kSelThreads, 1)
moe_route_kernel(const float* __restrict__ topk_score, const int32_t* __restrict__ topk_idx, int T, int N, int K_orig,
                 int K_base, long long budget, int use_smem_keys, int n_sel_given, int32_t* __restrict__ n_sel,
                 int32_t* __restrict__ expert_offsets, int32_t* __restrict__ perm_token,
                 float* __restrict__ perm_weight, int32_t* __restrict__ pair_pos, int32_t* dev_status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SelectSmem& sm = *reinterpret_cast<SelectSmem*>(smem_raw);
  int32_t* seg_counts = reinterpret_cast<int32_t*>(smem_raw + sizeof(SelectSmem));
  const int warp = threadIdx.x >> 5;
  const int nseg = (T + 31) / 32;
  pdl_prologue_done();

  // n_sel_given: the caller's n_sel is the input (a selection made over a larger pool, of which this batch is a
  // part); the kept pairs then number at most `budget`, not exactly `budget`.
  if (!n_sel_given)
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
  permute_scan_block(seg_counts, N, nseg, budget, !n_sel_given, expert_offsets, dev_status, sm.scan_ws);
  __syncthreads();
  if (seg < nseg)
    permute_place_from_masks(mask, e_loc, n, topk_score, seg, T, K_orig, nseg, seg_counts, budget, perm_token,
                             perm_weight, pair_pos);
}

// ------------------------------------------------------------------------------------------------
// The same step for 1024 < T <= 8192: ONE launch of a thread-block cluster of ceil(T / 1024) CTAs.
// CTA r owns tokens [1024 r, 1024 (r + 1)), one per thread, which keeps the token's residual keys in
// registers.  Each radix pass histograms the CTA's own keys; the CTAs read one another's
// 256-bin histograms through distributed shared memory after a cluster barrier and all take the
// same digit decision.  Ties are resolved in flat order by an exclusive scan of per-token tie
// counts inside the CTA plus the tie totals of the lower-ranked CTAs.  The thread that computes
// n_sel[t] is lane t % 32 of the warp that owns t's 32-token segment, so the count goes on to the
// permutation in a register: per-segment masks, per-CTA scan over the segments, expert totals
// exchanged through distributed shared memory, placement.  Results are identical to
// alloc_t_select followed by moe_permute.
constexpr int kRouteClusterMax = 8;            // portable cluster size

struct RouteClusterSmem {
  int warp_hist[kRouteWarps][256];   // per-warp histograms; afterwards each warp's expert masks
  int hist[2][256];                  // this CTA's histogram of the current digit (read by the peers)
  int ghist[256];                    // the cluster's
  int scan_ws[33];
  uint32_t prefix;
  int remaining;
  int bucket;
  int eq_total;                      // keys equal to tau among this CTA's tokens (read by the peers)
  int tot[kMaxExperts];              // kept pairs per expert among this CTA's tokens (read by the peers)
  int ebase[kMaxExperts];            // first list position of expert e's pairs from this CTA
  int lbase[kMaxExperts * kRouteWarps];   // [e][warp]: kept pairs of e in this CTA's lower segments, then positions
};

__global__ void __launch_bounds__(kSelThreads, 1)
moe_route_cluster_kernel(const float* __restrict__ topk_score, const int32_t* __restrict__ topk_idx, int T, int N,
                         int K_orig, int K_base, long long budget, int n_sel_given, int32_t* __restrict__ n_sel,
                         int32_t* __restrict__ expert_offsets, int32_t* __restrict__ perm_token,
                         float* __restrict__ perm_weight, int32_t* __restrict__ pair_pos, int32_t* dev_status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  RouteClusterSmem& sm = *reinterpret_cast<RouteClusterSmem*>(smem_raw);
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank(), n_ranks = (int)cluster.num_blocks();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t = rank * kSelThreads + tid;          // this thread's token
  const bool have = t < T;
  const int Kr = K_orig - K_base;
  const long long R = budget - (long long)K_base * T;
  pdl_prologue_done();

  // ---------------- Alloc-T selection (Sec. 3.3)
  int n_mine = K_base;
  if (n_sel_given) {                       // the caller's selection (see moe_route_kernel)
    if (have) n_mine = n_sel[t];
  } else if (R > 0 && Kr > 0) {
    const uint32_t* bits = reinterpret_cast<const uint32_t*>(topk_score);
    uint32_t k[16];
    bool bad = false;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      k[j] = 0u;
      if (have && j >= K_base && j < K_orig) {
        k[j] = bits[(long long)t * K_orig + j];
        bad |= (k[j] >= 0x7F800000u);      // NaN, Inf or negative
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
      if (have) {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (j >= K_base && j < K_orig && (k[j] & prefix_mask) == prefix)
            atomicAdd(&sm.warp_hist[warp][(k[j] >> shift) & 255u], 1);
      }
      __syncthreads();
      if (tid < 256) {
        int a = 0;
#pragma unroll 8
        for (int w = 0; w < kRouteWarps; ++w) a += sm.warp_hist[w][tid];
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
    const int need_eq = sm.remaining;     // how many keys equal to tau are kept (>= 1)
    int gt = 0, eq = 0;
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (have && j >= K_base && j < K_orig) {
        gt += (k[j] > tau);
        eq += (k[j] == tau);
      }
    if (sm.bucket == need_eq) {           // every key equal to tau is kept: no order among ties matters
      n_mine = K_base + gt + eq;
    } else {                              // ties in flat order: tokens in order, CTAs in rank order
      int cta_eq;
      int ties_before = block_exclusive_scan(eq, sm.scan_ws, &cta_eq);
      if (tid == 0) sm.eq_total = cta_eq;
      cluster.sync();
      for (int r = 0; r < rank; ++r) ties_before += *cluster.map_shared_rank(&sm.eq_total, r);
      n_mine = K_base + gt + min(eq, max(0, need_eq - ties_before));
    }
  }
  if (have && !n_sel_given) n_sel[t] = n_mine;

  // ---------------- permutation: counts per (expert, segment), this CTA's segments = its warps
  uint32_t* mask = reinterpret_cast<uint32_t*>(sm.warp_hist[warp]);
  int e_loc[16], n = 0;
  __syncthreads();   // the last histogram reads are over before the masks overwrite warp_hist
  build_masks(mask, topk_idx, n_sel, t, T, N, K_orig, lane, e_loc, n, have ? n_mine : 0);
  for (int e = lane; e < N; e += 32) sm.lbase[e * kRouteWarps + warp] = __popc(mask[e]);
  __syncthreads();
  for (int e = warp; e < N; e += kRouteWarps) {   // exclusive scan over the CTA's 32 segments, lane = segment
    const int c = sm.lbase[e * kRouteWarps + lane];
    int incl = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int o = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += o;
    }
    sm.lbase[e * kRouteWarps + lane] = incl - c;
    if (lane == 31) sm.tot[e] = incl;
  }
  cluster.sync();    // every CTA's per-expert totals are complete
  int all = 0, before = 0;
  if (tid < N) {
    for (int r = 0; r < n_ranks; ++r) {
      const int v = cluster.map_shared_rank(&sm.tot[0], r)[tid];
      all += v;
      if (r < rank) before += v;
    }
  }
  int total;
  const int off = block_exclusive_scan(all, sm.scan_ws, &total);
  if (tid < N) {
    sm.ebase[tid] = off + before;
    if (rank == 0) expert_offsets[tid] = off;
  }
  if (rank == 0 && tid == 0) {
    expert_offsets[N] = total;
    if (n_sel_given ? (long long)total > budget : (long long)total != budget) set_dev_status(dev_status, MOE_ERR_BUDGET);
  }
  __syncthreads();
  for (int i = tid; i < N * kRouteWarps; i += kSelThreads) sm.lbase[i] += sm.ebase[i / kRouteWarps];
  __syncthreads();
  permute_place_from_masks(mask, e_loc, n, topk_score, rank * kRouteWarps + warp, T, K_orig, kRouteWarps, sm.lbase, budget,
                           perm_token, perm_weight, pair_pos, warp);
  cluster.sync();    // no CTA leaves while a peer may still read its shared memory
}

}  // namespace allocmoe

using namespace allocmoe;

// True when one launch can do the whole routing step: one CTA up to 1024 tokens (every warp gets at
// most one 32-token segment and the permutation's counters fit the shared-memory pool), a cluster of
// up to 8 such CTAs up to 8192 tokens.
bool moe_route_fits(const moe_shape* s) {
  return s->T <= (long long)kRouteClusterMax * kSelThreads;
}

static bool route_one_cta(const moe_shape* s) {
  const long long nseg = (s->T + 31) / 32;
  return nseg <= kRouteWarps && (long long)s->N * nseg <= (long long)kSelMaxSmemKeys;
}

// n_sel_given: n_sel is an input and only the permutation's lists are built; `budget` is then an upper bound.
moe_status launch_moe_route(const moe_shape* s, const float* topk_score, const int32_t* topk_idx, int64_t budget,
                            bool n_sel_given, int32_t* n_sel, int32_t* expert_offsets, int32_t* perm_token,
                            float* perm_weight, int32_t* pair_pos, int32_t* dev_status, cudaStream_t stream) {
  if (!route_one_cta(s)) {
    const unsigned n_ctas = (unsigned)((s->T + kSelThreads - 1) / kSelThreads);
    static PerDeviceOnce cattr_set;
    if (!ensure_dynamic_smem(moe_route_cluster_kernel, sizeof(RouteClusterSmem), cattr_set)) return MOE_ERR_CUDA;
    return launch_dependent_cluster(moe_route_cluster_kernel, dim3(n_ctas), dim3(kSelThreads), sizeof(RouteClusterSmem),
                                    stream, dim3(n_ctas, 1, 1), topk_score, topk_idx, (int)s->T, (int)s->N,
                                    (int)s->K_orig, (int)s->K_base, (long long)budget, n_sel_given ? 1 : 0, n_sel,
                                    expert_offsets, perm_token, perm_weight, pair_pos, dev_status) == cudaSuccess
               ? MOE_OK
               : MOE_ERR_CUDA;
  }
  const long long P = (long long)s->T * (s->K_orig - s->K_base);
  const int use_smem_keys = (P <= kSelMaxSmemKeys && !n_sel_given) ? 1 : 0;
  const long long counters = (long long)s->N * ((s->T + 31) / 32);
  const long long pool_ints = (use_smem_keys && P > counters) ? P : counters;
  const size_t smem = sizeof(SelectSmem) + (size_t)pool_ints * 4;
  static PerDeviceOnce attr_set;
  if (!ensure_dynamic_smem(moe_route_kernel, sizeof(SelectSmem) + (size_t)kSelMaxSmemKeys * 4, attr_set)) return MOE_ERR_CUDA;
  return launch_dependent(moe_route_kernel, dim3(1), dim3(kSelThreads), smem, stream, 1, topk_score, topk_idx, (int)s->T,
                          (int)s->N, (int)s->K_orig, (int)s->K_base, (long long)budget, use_smem_keys, n_sel_given ? 1 : 0,
                          n_sel, expert_offsets, perm_token, perm_weight, pair_pos, dev_status) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}
