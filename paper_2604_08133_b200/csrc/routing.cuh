// Device-side building blocks of the routing steps, shared by the stand-alone kernels
// (alloc_t_select, moe_permute) and by the fused routing kernel that moe_layer_forward uses.
#pragma once

#include "common.cuh"

namespace allocmoe {

// ------------------------------------------------------------------ Alloc-T selection (Sec. 3.3)
constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelMaxSmemKeys = 40960;   // 160 KB of keys + 32 KB of per-warp histograms

struct SelectSmem {
  int warp_hist[kSelWarps][256];
  int hist[256];
  int scan_ws[33];
  uint32_t prefix;
  int remaining;
  int bucket;
};

// One warp: given the histogram of the current 8-bit digit over the keys that share `prefix`, find the
// digit in which the running count from the top first reaches *remaining, append it to the prefix,
// and leave in *remaining the rank wanted inside that digit and in *bucket the digit's key count.
DEV void radix_choose_digit(const int* hist, int shift, uint32_t prefix, uint32_t* prefix_out, int* remaining,
                            int* bucket) {
  const int lane = threadIdx.x & 31;
  // lane l owns digits 255-8l .. 248-8l (descending)
  int c[8], lsum = 0;
#pragma unroll
  for (int q = 0; q < 8; ++q) { c[q] = hist[255 - (lane * 8 + q)]; lsum += c[q]; }
  int incl = lsum;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  int above = incl - lsum;           // keys in strictly higher digits than this lane's
  const int rem = *remaining;
  __syncwarp();
  if (above < rem && rem <= incl) {  // exactly one lane
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      if (above < rem && rem <= above + c[q]) {
        *prefix_out = prefix | ((uint32_t)(255 - (lane * 8 + q)) << shift);
        *remaining = rem - above;
        *bucket = c[q];              // keys that share the prefix chosen so far
        above = rem;                 // stop
      } else {
        above += c[q];
      }
    }
  }
}

// The selection, run by one CTA of kSelThreads threads.  `smem_raw`: sizeof(SelectSmem) bytes, then
// room for the pool's keys when use_smem_keys is set.  Ends with a block-wide barrier after which
// n_sel is visible to the whole CTA.
DEV void alloc_t_select_block(unsigned char* smem_raw, const float* __restrict__ topk_score, int T, int K_orig,
                              int K_base, long long R, int use_smem_keys, int32_t* __restrict__ n_sel,
                              int32_t* dev_status) {
  SelectSmem& sm = *reinterpret_cast<SelectSmem*>(smem_raw);
  uint32_t* skeys = reinterpret_cast<uint32_t*>(smem_raw + sizeof(SelectSmem));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Kr = K_orig - K_base;
  const long long P = (long long)T * Kr;
  const uint32_t* bits = reinterpret_cast<const uint32_t*>(topk_score);

  if (R <= 0 || Kr == 0) {   // nothing to redistribute: plain Top-K_base
    for (int t = tid; t < T; t += kSelThreads) n_sel[t] = K_base;
    __syncthreads();
    return;
  }

  // Stage the pool and validate: a NaN, an Inf or a negative score has bits >= 0x7F800000.
  // One token per thread and step: its residual columns are independent loads.
  bool bad = false;
#pragma unroll 2
  for (int t = tid; t < T; t += kSelThreads) {
    uint32_t k[16];
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (j >= K_base && j < K_orig) k[j] = bits[(long long)t * K_orig + j];
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (j >= K_base && j < K_orig) {
        bad |= (k[j] >= 0x7F800000u);
        if (use_smem_keys) skeys[(long long)t * Kr + (j - K_base)] = k[j];
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
    if (warp == 0) radix_choose_digit(sm.hist, shift, prefix, &sm.prefix, &sm.remaining, &sm.bucket);
    prefix_mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t tau = sm.prefix;
  const int need_eq = sm.remaining;       // how many keys equal to tau are kept (>= 1)

  // After the last pass `bucket` is the number of keys equal to tau.  When all of them are kept (always
  // the case when tau occurs once) no order among ties matters: one coalesced sweep over the tokens.
  if (sm.bucket == need_eq) {
    for (int t = tid; t < T; t += kSelThreads) {
      int n = K_base;
      for (int j = K_base; j < K_orig; ++j) {
        const uint32_t k = use_smem_keys ? skeys[(long long)t * Kr + (j - K_base)] : bits[(long long)t * K_orig + j];
        n += (k >= tau);
      }
      n_sel[t] = n;
    }
    __syncthreads();
    return;
  }

  // Per token: keys above tau, then ties in flat order.  Threads own contiguous token ranges.
  const int tpt = (T + kSelThreads - 1) / kSelThreads;
  const int t_lo = min(T, tid * tpt), t_hi = min(T, t_lo + tpt);
  int my_eq = 0;
  for (int t = t_lo; t < t_hi; ++t)
    for (int j = K_base; j < K_orig; ++j) {
      const uint32_t k = use_smem_keys ? skeys[(long long)t * Kr + (j - K_base)] : bits[(long long)t * K_orig + j];
      my_eq += (k == tau);
    }
  int total_eq;
  int ties_before = block_exclusive_scan(my_eq, sm.scan_ws, &total_eq);
  for (int t = t_lo; t < t_hi; ++t) {
    int gt = 0, eq = 0;
    for (int j = K_base; j < K_orig; ++j) {
      const uint32_t k = use_smem_keys ? skeys[(long long)t * Kr + (j - K_base)] : bits[(long long)t * K_orig + j];
      gt += (k > tau);
      eq += (k == tau);
    }
    const int room = max(0, need_eq - ties_before);
    n_sel[t] = K_base + gt + min(eq, room);
    ties_before += eq;
  }
  __syncthreads();
}


// ------------------------------------------------------------------ permutation
constexpr int kMaxExperts = 128;

// One warp, lane = token of the segment: mask[e] bit l set iff token l keeps expert e; e_out / n_out are
// the lane's kept expert ids and their number.  n_raw < 0: the count is read from n_sel[t].
DEV void build_masks(uint32_t* mask, const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ n_sel,
                     int t, int T, int N, int K_orig, int lane, int (&e_out)[16], int& n_out, int n_known = -1) {
  for (int e = lane; e < N; e += 32) mask[e] = 0u;
  __syncwarp();
  n_out = 0;
  if (t < T) {
    // the count and all K_orig expert ids travel together (one round trip); ids past the count are ignored
    const int n_raw = n_known >= 0 ? n_known : n_sel[t];
#pragma unroll
    for (int j = 0; j < 16; ++j) e_out[j] = (j < K_orig) ? topk_idx[(long long)t * K_orig + j] : 0;
    n_out = min(max(n_raw, 0), K_orig);
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if (j < n_out) {
        const int e = min(max(e_out[j], 0), N - 1);   // keeps every access in bounds on corrupt input
        e_out[j] = e;
        atomicOr(&mask[e], 1u << lane);
      }
    }
  }
  __syncwarp();
}

// One warp, one 32-token segment: seg_counts[e][seg] = number of kept pairs of expert e.
DEV void permute_count_warp(uint32_t* mask, const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ n_sel,
                            int seg, int T, int N, int K_orig, int nseg, int32_t* seg_counts) {
  const int lane = threadIdx.x & 31;
  int e_loc[16], n;
  build_masks(mask, topk_idx, n_sel, seg * 32 + lane, T, N, K_orig, lane, e_loc, n);
  for (int e = lane; e < N; e += 32) seg_counts[(long long)e * nseg + seg] = __popc(mask[e]);
}

// The whole CTA: in-place exclusive scan of seg_counts (N*nseg ints, expert-major; shared or global
// memory), expert_offsets, and the check that the kept pairs add up to the budget.
// exact: the kept pairs must number exactly `budget`; otherwise `budget` is only an upper bound (the caller's
// n_sel came from a selection over a larger pool and this batch's share is known to the device alone).
DEV void permute_scan_block(int32_t* seg_counts, int N, int nseg, long long budget, bool exact,
                            int32_t* __restrict__ expert_offsets, int32_t* dev_status, int* scan_ws) {
  const long long M = (long long)N * nseg;
  const int per = (int)((M + blockDim.x - 1) / blockDim.x);
  const long long lo = min(M, (long long)threadIdx.x * per), hi = min(M, lo + per);
  int sum = 0;
  for (long long i = lo; i < hi; ++i) sum += seg_counts[i];
  int total;
  int run = block_exclusive_scan(sum, scan_ws, &total);
  for (long long i = lo; i < hi; ++i) {
    const int c = seg_counts[i];
    seg_counts[i] = run;
    if (i % nseg == 0) expert_offsets[i / nseg] = run;
    run += c;
  }
  if (threadIdx.x == 0) {
    expert_offsets[N] = total;
    if (exact ? (long long)total != budget : (long long)total > budget) set_dev_status(dev_status, MOE_ERR_BUDGET);
  }
}

DEV void permute_place_from_masks(const uint32_t* mask, const int (&e_loc)[16], int n,
                                  const float* __restrict__ topk_score, int seg, int T, int K_orig, int nseg,
                                  const int32_t* seg_base, long long budget, int32_t* __restrict__ perm_token,
                                  float* __restrict__ perm_weight, int32_t* __restrict__ pair_pos, int base_col = -1);

// One warp, one 32-token segment: list positions of its kept pairs.
DEV void permute_place_warp(uint32_t* mask, const int32_t* __restrict__ topk_idx, const float* __restrict__ topk_score,
                            const int32_t* __restrict__ n_sel, int seg, int T, int N, int K_orig, int nseg,
                            const int32_t* seg_base, long long budget, int32_t* __restrict__ perm_token,
                            float* __restrict__ perm_weight, int32_t* __restrict__ pair_pos) {
  const int lane = threadIdx.x & 31;
  int e_loc[16], n;
  build_masks(mask, topk_idx, n_sel, seg * 32 + lane, T, N, K_orig, lane, e_loc, n);
  permute_place_from_masks(mask, e_loc, n, topk_score, seg, T, K_orig, nseg, seg_base, budget, perm_token, perm_weight,
                           pair_pos);
}

// The placement proper, from the segment's masks and this lane's expert ids (build_masks).  The first list
// position of (expert e, this segment) is seg_base[e * nseg + col], col = seg unless base_col is given.
DEV void permute_place_from_masks(const uint32_t* mask, const int (&e_loc)[16], int n,
                                  const float* __restrict__ topk_score, int seg, int T, int K_orig, int nseg,
                                  const int32_t* seg_base, long long budget, int32_t* __restrict__ perm_token,
                                  float* __restrict__ perm_weight, int32_t* __restrict__ pair_pos, int base_col) {
  const int lane = threadIdx.x & 31;
  const int t = seg * 32 + lane;
  if (t >= T) return;
  const int col = base_col >= 0 ? base_col : seg;
  const uint32_t lower = (1u << lane) - 1u;
  float w[16];   // all of the token's scores in one round trip
#pragma unroll
  for (int j = 0; j < 16; ++j) w[j] = (j < K_orig) ? topk_score[(long long)t * K_orig + j] : 0.f;
  int pos[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    pos[j] = -1;
    if (j < n) {
      const int e = e_loc[j];
      const int q = seg_base[(long long)e * nseg + col] + __popc(mask[e] & lower);
      if (q >= 0 && q < budget) pos[j] = q;   // always true when sum n_sel == budget
    }
  }
#pragma unroll
  for (int j = 0; j < 16; ++j)
    if (j < K_orig && pos[j] >= 0) {
      perm_token[pos[j]] = t;
      perm_weight[pos[j]] = w[j];
    }
#pragma unroll
  for (int j = 0; j < 16; ++j)
    if (j < K_orig) pair_pos[(long long)t * K_orig + j] = pos[j];
}

}  // namespace allocmoe
