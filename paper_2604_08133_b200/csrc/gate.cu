// moe_gate: Eq. 1 fused -- logits = x . W_gate (+ bias), row softmax over all N experts (fp32),
// and the K_orig largest scores per token sorted descending (ties: lower expert id first).
//
// The contraction is small (2*T*H*N flops; 1 GFLOP at T=4096, H=2048, N=64) and x is read once,
// so the kernel is bound by streaming x from HBM and, at decode sizes, by latency.  A CTA owns
// 16*NW tokens (one warp per 16 tokens; NW = 2 for small batches, 4 from 2048 tokens on, which
// halves the re-reads of W_gate from L2), all N experts and every KS-th chunk of 128 along H; the
// KS CTAs that share a token tile form a thread-block cluster (KS <= 8), so that T = 64 tokens
// still put 16 CTAs to work and no CTA walks more than a few chunks.  Chunks of x and W_gate are
// staged in shared memory with 16-byte cp.async (3 stages) and multiplied with mma.sync m16n8k16
// bf16 -> fp32.  The KS partial logits of a token are then added in rank order through
// distributed shared memory, and each CTA finishes softmax and Top-K for its 16*NW/KS tokens.  W_gate is stored [H,N] (N contiguous, the
// paper's R^{H x N}), which is the "column" operand of mma.sync when read with ldmatrix.trans.
#include <cooperative_groups.h>

#include "common.cuh"
#include "tmap.h"

namespace cg = cooperative_groups;

namespace allocmoe {

constexpr int kGateKC = 128;       // H chunk
constexpr int kGateStages = 3;
constexpr int kGateXStride = kGateKC + 8;   // bf16 elements per staged x row (272 B: conflict-free ldmatrix)

DEV void ldmatrix_x4(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(p)));
}
DEV void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(p)));
}
DEV void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// The KS partial logit tiles of this CTA's share of the tile's tokens (rows first_row .. of every tile rred[k]),
// added in rank order into local shared memory: sum[rr][e] = rred[0][..] + rred[1][..] + ...  Every thread takes
// a few elements and issues its KS loads from the peers' shared memory back to back (inside gate_finish's
// per-token loop the same loads went out one after the other).  Ends with a block barrier.
// (Pushing the partial rows to their owner with remote stores instead was measured slower: 11.5 -> 14.9 us at
// 4096 tokens, 25 us with eight ranks.)
template <int NP>
DEV void gate_reduce_partials(const float* const (&rred)[8], int KS, int first_row, int rows_per, float* sum) {
  constexpr int RS = NP + 1;
  for (int i = threadIdx.x; i < rows_per * NP; i += blockDim.x) {
    const int rr = i / NP, e = i % NP;
    const int at = (first_row + rr) * RS + e;
    float v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = k < KS ? rred[k][at] : 0.f;
    float a = v[0];
#pragma unroll
    for (int k = 1; k < 8; ++k)
      if (k < KS) a += v[k];
    sum[rr * RS + e] = a;
  }
  __syncthreads();
}

// Softmax (fp32, expf) and sorted Top-K_orig for the tokens ks_rank*rows_per .. of the tile, from their summed
// logits sum[rr][e] (the bias is added here).  GS lanes work on one token, lane g of them owns
// experts g, g+GS, ...; a warp finishes 32/GS tokens at a time.
template <int NP, int NW, int GS>
DEV void gate_finish(const float* sum, int KS, int ks_rank, int t0, int T, int N, int K_orig,
                     const float* __restrict__ gate_bias, float* __restrict__ scores, int32_t* __restrict__ topk_idx,
                     float* __restrict__ topk_score) {
  constexpr int EPL = (NP + GS - 1) / GS, TPW = 32 / GS, RS = NP + 1, kGateTM = 16 * NW;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int rows_per = kGateTM / KS;
  const int g8 = lane % GS, slot = lane / GS;
  for (int rr0 = warp * TPW; rr0 < rows_per; rr0 += NW * TPW) {   // uniform across the warp
    const int rr = rr0 + slot;
    const int r = ks_rank * rows_per + rr;
    const int t = t0 + r;
    const bool valid = rr < rows_per && t < T;
    float v[EPL];
    float mx = -INFINITY;
#pragma unroll
    for (int q = 0; q < EPL; ++q) {
      const int e = g8 + GS * q;
      float a = -INFINITY;
      if (valid && e < N) {
        a = sum[rr * RS + e];
        if (gate_bias != nullptr) a += gate_bias[e];
      }
      v[q] = a;
      mx = fmaxf(mx, v[q]);
    }
#pragma unroll
    for (int d = GS / 2; d >= 1; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    float sum = 0.f;
#pragma unroll
    for (int q = 0; q < EPL; ++q) {
      v[q] = (valid && g8 + GS * q < N) ? expf(v[q] - mx) : 0.f;
      sum += v[q];
    }
#pragma unroll
    for (int d = GS / 2; d >= 1; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
#pragma unroll
    for (int q = 0; q < EPL; ++q) {
      v[q] = valid ? v[q] / sum : 0.f;
      const int e = g8 + GS * q;
      if (scores != nullptr && valid && e < N) scores[(long long)t * N + e] = v[q];
    }
    uint32_t taken = 0u;
    for (int j = 0; j < K_orig; ++j) {
      float bv = -1.f;
      int be = 0x7fffffff;
#pragma unroll
      for (int q = 0; q < EPL; ++q) {
        const int e = g8 + GS * q;
        if (e < N && !((taken >> q) & 1u) && v[q] > bv) { bv = v[q]; be = e; }   // ascending e: first max wins
      }
#pragma unroll
      for (int d = GS / 2; d >= 1; d >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, d);
        const int oe = __shfl_xor_sync(0xffffffffu, be, d);
        if (ov > bv || (ov == bv && oe < be)) { bv = ov; be = oe; }
      }
      if (be % GS == g8 && be < N) taken |= 1u << (be / GS);
      if (g8 == 0 && valid) {
        topk_idx[(long long)t * K_orig + j] = be < N ? be : 0;
        topk_score[(long long)t * K_orig + j] = bv;
      }
    }
  }
}

// NT16 = number of 16-wide expert tiles (N padded to 16*NT16); NW = warps = 16-token slabs per CTA.
template <int NT16, int NW>
__global__ void __launch_bounds__(32 * NW)
moe_gate_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ W_gate,
                const float* __restrict__ gate_bias, int T, int H, int N, int K_orig, int w_stride,
                float* __restrict__ scores, int32_t* __restrict__ topk_idx, float* __restrict__ topk_score,
                int32_t* __restrict__ zero_ptr, int zero_n) {
  cg::cluster_group cluster = cg::this_cluster();
  const int KS = (int)cluster.num_blocks();        // CTAs per token tile (cluster spans blockIdx.y)
  const int ks_rank = (int)cluster.block_rank();
  constexpr int NP = NT16 * 16;
  constexpr int kGateTM = 16 * NW, kGateThreads = 32 * NW;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int x_stage_bytes = kGateTM * kGateXStride * 2;
  const int w_stage_bytes = kGateKC * w_stride * 2;
  const int stage_bytes = x_stage_bytes + w_stage_bytes;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t0 = blockIdx.x * kGateTM;
  const int nchunks_all = (H + kGateKC - 1) / kGateKC;
  const int nchunks = (nchunks_all - ks_rank + KS - 1) / KS;   // this CTA's chunks: ks_rank, ks_rank + KS, ...
  const int n_vec = N / 8;   // 16-byte pieces per W_gate row
  pdl_prologue_done();
  // Side job for the layer call: clear the expert GEMMs' row-block counters.  As the first kernel of the call this
  // one runs after everything that read them; doing it here keeps a memset out of the stream, which would sit
  // between two kernels and stop the later one from starting early as a programmatic dependent.
  if (zero_ptr != nullptr && blockIdx.x == 0 && blockIdx.y == 0)
    for (int i = tid; i < zero_n; i += kGateThreads) zero_ptr[i] = 0;

  auto issue = [&](int chunk) {
    if (chunk < nchunks) {
      unsigned char* st = smem_raw + (chunk % kGateStages) * stage_bytes;
      __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(st);
      __nv_bfloat16* ws = reinterpret_cast<__nv_bfloat16*>(st + x_stage_bytes);
      const int k0 = (ks_rank + chunk * KS) * kGateKC;
      for (int i = tid; i < kGateTM * (kGateKC / 8); i += kGateThreads) {
        const int r = i / (kGateKC / 8), c = i % (kGateKC / 8);
        const int t = t0 + r, k = k0 + c * 8;
        const bool ok = (t < T) && (k < H);
        cp_async_16(xs + r * kGateXStride + c * 8, x + (ok ? ((long long)t * H + k) : 0), ok);
      }
      if ((N & 7) == 0) {
        for (int i = tid; i < kGateKC * (NP / 8); i += kGateThreads) {
          const int r = i / (NP / 8), c = i % (NP / 8);
          const int k = k0 + r;
          const bool ok = (k < H) && (c < n_vec);
          cp_async_16(ws + r * w_stride + c * 8, W_gate + (ok ? ((long long)k * N + c * 8) : 0), ok);
        }
      } else {   // N a multiple of 4 only: rows of W_gate start on 8-byte boundaries
        for (int i = tid; i < kGateKC * (NP / 4); i += kGateThreads) {
          const int r = i / (NP / 4), c = i % (NP / 4);
          const int k = k0 + r;
          const bool ok = (k < H) && (c < N / 4);
          cp_async_8(ws + r * w_stride + c * 4, W_gate + (ok ? ((long long)k * N + c * 4) : 0), ok);
        }
      }
    }
    cp_async_commit();
  };

  float acc[NT16 * 2][4];   // this warp's 16 tokens x NP experts
#pragma unroll
  for (int n = 0; n < NT16 * 2; ++n)
#pragma unroll
    for (int q = 0; q < 4; ++q) acc[n][q] = 0.f;

  issue(0);
  issue(1);
  for (int chunk = 0; chunk < nchunks; ++chunk) {
    issue(chunk + 2);
    cp_async_wait<2>();
    __syncthreads();
    const unsigned char* st = smem_raw + (chunk % kGateStages) * stage_bytes;
    const __nv_bfloat16* xs = reinterpret_cast<const __nv_bfloat16*>(st);
    const __nv_bfloat16* ws = reinterpret_cast<const __nv_bfloat16*>(st + x_stage_bytes);
#pragma unroll
    for (int ks = 0; ks < kGateKC / 16; ++ks) {
      const int kk = ks * 16;
      uint32_t a[4];
      ldmatrix_x4(a, xs + (warp * 16 + (lane & 15)) * kGateXStride + kk + (lane >> 4) * 8);
#pragma unroll
      for (int n16 = 0; n16 < NT16; ++n16) {
        uint32_t b[4];
        ldmatrix_x4_trans(b, ws + (kk + (lane & 7) + ((lane >> 3) & 1) * 8) * w_stride + n16 * 16 + (lane >> 4) * 8);
        mma_bf16_16816(acc[n16 * 2], a, b[0], b[1]);
        mma_bf16_16816(acc[n16 * 2 + 1], a, b[2], b[3]);
      }
    }
    __syncthreads();
  }
  cp_async_wait<0>();
  __syncthreads();

  // This CTA's partial logits: red[row][col], fp32, aliasing the staging buffers.
  float* red = reinterpret_cast<float*>(smem_raw);
  constexpr int RS = NP + 1;
  {
    const int g = lane >> 2, tq = lane & 3;
#pragma unroll
    for (int n = 0; n < NT16 * 2; ++n) {
      float* base = red + ((warp * 16 + g) * RS + n * 8 + tq * 2);
      base[0] = acc[n][0];
      base[1] = acc[n][1];
      base[8 * RS] = acc[n][2];
      base[8 * RS + 1] = acc[n][3];
    }
  }
  cluster.sync();   // every CTA's partial logits are in its red[0 .. 16*NW*RS)

  // Softmax and sorted Top-K_orig of this CTA's share of the tile's tokens: eight lanes per token where a warp
  // has at least four tokens to finish (large batches), sixteen where it has two, else the whole warp on one
  // token (fewer loads per lane).
  const float* rred[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) rred[k] = cluster.map_shared_rank(red, k < KS ? k : 0);
  const float* sum = red;            // one CTA per tile: its partial tile is the sum
  if (KS > 1) {
    float* s2 = red + kGateTM * RS;  // behind this CTA's own partial tile, which the peers are still reading
    gate_reduce_partials<NP>(rred, KS, ks_rank * (kGateTM / KS), kGateTM / KS, s2);
    sum = s2;
  }
  if (kGateTM / KS >= NW * 4)
    gate_finish<NP, NW, 8>(sum, KS, ks_rank, t0, T, N, K_orig, gate_bias, scores, topk_idx, topk_score);
  else if (kGateTM / KS >= NW * 2)
    gate_finish<NP, NW, 16>(sum, KS, ks_rank, t0, T, N, K_orig, gate_bias, scores, topk_idx, topk_score);
  else
    gate_finish<NP, NW, 32>(sum, KS, ks_rank, t0, T, N, K_orig, gate_bias, scores, topk_idx, topk_score);
  cluster.sync();   // no CTA leaves while a peer may still read its partial sums
}

// ------------------------------------------------------------------------------------------------
// Large batches (about a thousand tokens and more) with N = 64 or 128 experts: the contraction on the
// 5th-generation tensor cores.  On B200 the mma.sync path above tops out near 190 TFLOP/s for the whole
// GPU, which made the kernel above compute-bound on 4096 tokens (17 us however its chunks were loaded:
// cp.async, per-row bulk copies and TMA boxes all measured the same); tcgen05.mma removes that bound.
//
// Same decomposition: a cluster of KS CTAs per token tile (128 tokens here = UMMA M), rank r taking 64-wide
// blocks r, r + KS, ... of H, partial logits added in rank order through distributed shared memory, then
// gate_finish.  Per block one TMA box of x (128 tokens x 64, K-major, the A operand) and one box per 64
// experts of W_gate (64 rows of H x 64 experts: N-contiguous, i.e. an MN-major B operand, which the
// instruction descriptor's B-major bit and the shared-memory descriptor below express: 8-row groups along K
// are 1024 bytes apart, 64-expert blocks one box apart), all written with the 128-byte swizzle.  A CTA's
// blocks (at most 8) all have their own stage, so every load is issued up front and no stage is reused.
// One thread issues the loads and the MMAs (M = 128, N = 64 or 128, K = 16; fp32 accumulator in TMEM); then
// all eight warps read the accumulator (warp w: lanes 32 (w % 4).., half of the columns each) into shared
// memory for the cluster-wide reduction.
//
// Waits are bounded.  A wait that runs out marks the tile's scores NaN (which the selection reports as
// MOE_ERR_NONFINITE) and raises MOE_ERR_TIMEOUT in dev_status when the caller gave one; the CTA still takes
// part in every cluster barrier, waits for its copies in flight and frees its tensor memory before it exits.
constexpr int kUGateTM = 128;
constexpr int kUGateBK = 64;
constexpr int kUGateMaxStages = 8;
constexpr int kUGateXBytes = kUGateTM * kUGateBK * 2;      // 16 KB
constexpr int kUGateWBoxBytes = kUGateBK * 64 * 2;         // 8 KB per 64 experts

// MN-major operand, 128-byte swizzle: rows of 64 elements along N (128 bytes) per K index, groups of eight K
// rows 1024 bytes apart (stride byte offset), 64-element blocks along N `n_block_bytes` apart (leading byte
// offset).  Advancing 16 along K adds 2048 bytes to the start address.
DEV uint64_t umma_desc_mn_sw128(uint32_t smem_addr, uint32_t n_block_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
  d |= (uint64_t)((n_block_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

template <int NB64>   // N = 64 * NB64
__global__ void __launch_bounds__(256, 1)
moe_gate_umma_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                     const float* __restrict__ gate_bias, int T, int H, int N, int K_orig,
                     float* __restrict__ scores, int32_t* __restrict__ topk_idx, float* __restrict__ topk_score,
                     int32_t* __restrict__ zero_ptr, int zero_n, int32_t* dev_status) {
  cg::cluster_group cluster = cg::this_cluster();
  const int KS = (int)cluster.num_blocks();
  const int ks_rank = (int)cluster.block_rank();
  constexpr int NP = 64 * NB64, NW = 8, kThreads = 256;
  constexpr int kStageBytes = kUGateXBytes + NB64 * kUGateWBoxBytes;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  __shared__ uint64_t full[kUGateMaxStages];
  __shared__ uint64_t acc_done;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t0 = blockIdx.x * kUGateTM;
  const int nblocks_all = (H + kUGateBK - 1) / kUGateBK;
  const int nblocks = (nblocks_all - ks_rank + KS - 1) / KS;   // this CTA's blocks of H: ks_rank, ks_rank + KS, ... (<= 8)
  if (tid == 0) {
    for (int i = 0; i < kUGateMaxStages; ++i) mbar_init(&full[i], 1);
    mbar_init(&acc_done, 1);
    s_abort = 0;
    fence_barrier_init();
    prefetch_tensormap(&tm_x);
    prefetch_tensormap(&tm_w);
  }
  if (warp == 1) {
    tmem_alloc(&s_tmem, NP);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = s_tmem;
  pdl_prologue_done();
  if (zero_ptr != nullptr && blockIdx.x == 0 && blockIdx.y == 0)      // see moe_gate_kernel
    for (int i = tid; i < zero_n; i += kThreads) zero_ptr[i] = 0;

  if (tid == 0) {
    // every block of this CTA has its own stage: all loads go out at once (columns past H and rows past T read as zero)
    for (int b = 0; b < nblocks; ++b) {
      const int k0 = (ks_rank + b * KS) * kUGateBK;
      unsigned char* st = ring + b * kStageBytes;
      mbar_expect_tx(&full[b], (uint32_t)kStageBytes);
      tma_load_2d(st, &tm_x, &full[b], k0, t0);
#pragma unroll
      for (int nb = 0; nb < NB64; ++nb) tma_load_2d(st + kUGateXBytes + nb * kUGateWBoxBytes, &tm_w, &full[b], nb * 64, k0);
    }
    // instruction descriptor: fp32 accumulator, bf16 A and B, A K-major, B MN-major (bit 16)
    constexpr uint32_t idesc = umma_idesc_bf16(kUGateTM, NP) | (1u << 16);
    bool ok = true;
    for (int b = 0; b < nblocks && ok; ++b) {
      {   // bounded wait for the block's stage
        if (!mbar_try_wait(&full[b], 0u)) {
          const long long t_start = clock64();
          while (!mbar_try_wait(&full[b], 0u))
            if (clock64() - t_start > kWaitLimitClk) { ok = false; break; }
        }
      }
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t sa = smem_u32(ring + b * kStageBytes);
      const uint64_t da = umma_desc_sw128(sa);
      const uint64_t db = umma_desc_mn_sw128(sa + kUGateXBytes, (uint32_t)kUGateWBoxBytes);
#pragma unroll
      for (int k = 0; k < kUGateBK / 16; ++k)
        umma_bf16(tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * (2048 >> 4)), idesc, (b | k) != 0 ? 1u : 0u);
    }
    if (!ok) s_abort = 1;
    umma_commit(&acc_done);      // arrives once every MMA issued above has completed (at once if there were none)
  }
  __syncwarp();
  // every warp: wait for the accumulator (bounded; lane 0 polls)
  {
    int ok = 1;
    if (lane == 0 && !mbar_try_wait(&acc_done, 0u)) {
      const long long t_start = clock64();
      while (!mbar_try_wait(&acc_done, 0u)) {
        __nanosleep(32);
        if (clock64() - t_start > 2 * kWaitLimitClk) { ok = 0; break; }
      }
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (!ok) s_abort = 1;
  }
  tc_fence_after_sync();
  __syncthreads();   // s_abort is final; the MMAs no longer read the stages, which red[] aliases below
  const bool aborted = s_abort != 0;

  // partial logits to shared memory: red[row][col], fp32.  Warp w reads TMEM lanes 32 (w % 4) .. + 31 (= token rows)
  // and the column half w / 4.
  float* red = reinterpret_cast<float*>(ring);
  constexpr int RS = NP + 1;
  if (!aborted) {
    const int q = warp & 3, half = warp >> 2;
    const int row = q * 32 + lane;
    constexpr int kColsPerWarp = NP / 2;
#pragma unroll
    for (int c = 0; c < kColsPerWarp / 32; ++c) {
      uint32_t v[32];
      const int col0 = half * kColsPerWarp + c * 32;
      tmem_ld_32x32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)col0, v);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; ++i) red[row * RS + col0 + i] = __uint_as_float(v[i]);
    }
  } else {   // NaN partial sums give NaN scores in every CTA of the cluster
    if (tid == 0) {
      for (int b = 0; b < nblocks; ++b) mbar_wait_drain(&full[b], 0u);   // copies still in flight land first
      set_dev_status(dev_status, MOE_ERR_TIMEOUT);
    }
    __syncthreads();
    for (int i = tid; i < kUGateTM * RS; i += kThreads) red[i] = __int_as_float(0x7fc00000);
  }
  tc_fence_before_sync();
  cluster.sync();   // every CTA's partial logits are in its red[0 .. 128*RS)

  const float* rred[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) rred[k] = cluster.map_shared_rank(red, k < KS ? k : 0);
  const float* sum = red;            // one CTA per tile: its partial tile is the sum
  if (KS > 1) {
    float* s2 = red + kUGateTM * RS;  // behind this CTA's own partial tile, which the peers are still reading
    gate_reduce_partials<NP>(rred, KS, ks_rank * (kUGateTM / KS), kUGateTM / KS, s2);
    sum = s2;
  }
  if (kUGateTM / KS >= NW * 4)
    gate_finish<NP, NW, 8>(sum, KS, ks_rank, t0, T, N, K_orig, gate_bias, scores, topk_idx, topk_score);
  else if (kUGateTM / KS >= NW * 2)
    gate_finish<NP, NW, 16>(sum, KS, ks_rank, t0, T, N, K_orig, gate_bias, scores, topk_idx, topk_score);
  else
    gate_finish<NP, NW, 32>(sum, KS, ks_rank, t0, T, N, K_orig, gate_bias, scores, topk_idx, topk_score);
  cluster.sync();   // no CTA leaves while a peer may still read its partial sums
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, NP);
  }
}

}  // namespace allocmoe

using namespace allocmoe;

static int gate_w_stride(int NP) {
  int s16 = NP / 8 + 1;        // row stride in 16-byte units: odd keeps ldmatrix.trans conflict-free
  if ((s16 & 1) == 0) s16 += 1;
  return s16 * 8;
}

template <int NT16, int NW>
static moe_status gate_launch_t(const moe_shape* s, const uint16_t* x, const uint16_t* W_gate, const float* gate_bias,
                                float* scores, int32_t* topk_idx, float* topk_score, int32_t* zero_ptr, int zero_n,
                                cudaStream_t stream) {
  constexpr int NP = NT16 * 16, TM = 16 * NW;
  const int w_stride = gate_w_stride(NP);
  size_t pipe = (size_t)kGateStages * (TM * kGateXStride * 2 + kGateKC * w_stride * 2);
  size_t red = (size_t)TM * (NP + 1) * 4;   // the partial tile, and as much again for the summed logits
  size_t smem = pipe > 2 * red ? pipe : 2 * red;
  static PerDeviceOnce attr_set;
  if (!ensure_dynamic_smem(moe_gate_kernel<NT16, NW>, smem, attr_set)) return MOE_ERR_CUDA;
  // CTAs per token tile: a power of two <= 8 that leaves every CTA at least one chunk, grown while
  // the grid stays within two CTAs per SM (measured: 256 CTAs beat 128 and 512 at 2048 and 4096 tokens)
  const int nchunks = (s->H + kGateKC - 1) / kGateKC;
  const int tiles = (s->T + TM - 1) / TM;
  int ks = 1;
  while (ks * 2 <= 8 && ks * 2 <= nchunks && tiles * ks * 2 <= 296) ks *= 2;
  const cudaError_t err = launch_dependent(
      moe_gate_kernel<NT16, NW>, dim3((unsigned)tiles, (unsigned)ks, 1), dim3(32 * NW), smem, stream, (unsigned)ks,
      reinterpret_cast<const __nv_bfloat16*>(x), reinterpret_cast<const __nv_bfloat16*>(W_gate), gate_bias, (int)s->T,
      (int)s->H, (int)s->N, (int)s->K_orig, w_stride, scores, topk_idx, topk_score, zero_ptr, zero_n);
  return err == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

// The tcgen05 kernel.  KS: enough CTAs per 128-token tile that each holds at most kUGateMaxStages blocks of H and
// the grid is about one CTA per SM.  False when the shape does not fit (the caller falls back to mma.sync).
static bool gate_umma_fits(const moe_shape* s, int* ks_out) {
  if (s->T < 1024 || (s->N != 64 && s->N != 128)) return false;
  const int nblocks = (s->H + kUGateBK - 1) / kUGateBK;
  const int stage = kUGateXBytes + (s->N / 64) * kUGateWBoxBytes;
  const int max_stages = (200 * 1024) / stage < kUGateMaxStages ? (200 * 1024) / stage : kUGateMaxStages;
  const int tiles = (s->T + kUGateTM - 1) / kUGateTM;
  int ks = 1;
  while ((nblocks + ks - 1) / ks > max_stages && ks < 8) ks *= 2;
  if ((nblocks + ks - 1) / ks > max_stages) return false;
  while (ks * 2 <= 8 && ks * 2 <= nblocks && tiles * ks * 2 <= 160) ks *= 2;   // about one CTA per SM
  *ks_out = ks;
  return true;
}

template <int NB64>
static moe_status gate_launch_umma(const moe_shape* s, int ks, const uint16_t* x, const uint16_t* W_gate,
                                   const float* gate_bias, float* scores, int32_t* topk_idx, float* topk_score,
                                   int32_t* zero_ptr, int zero_n, int32_t* dev_status, cudaStream_t stream) {
  constexpr int NP = 64 * NB64;
  const int nblocks = (s->H + kUGateBK - 1) / kUGateBK;
  const int per_cta = (nblocks + ks - 1) / ks;
  const size_t stage = (size_t)kUGateXBytes + (size_t)NB64 * kUGateWBoxBytes;
  size_t smem = per_cta * stage;
  const size_t red = (size_t)kUGateTM * (NP + 1) * 4;   // the partial tile, and as much again for the summed logits
  if (smem < 2 * red) smem = 2 * red;
  smem += 1024;   // the stages start on a 1024-byte boundary (swizzle pattern)
  CUtensorMap tm_x, tm_w;
  if (!make_tmap(&tm_x, x, (uint64_t)s->H, (uint64_t)s->T, 0, (uint64_t)s->H, 0, kUGateTM) ||
      !make_tmap(&tm_w, W_gate, (uint64_t)s->N, (uint64_t)s->H, 0, (uint64_t)s->N, 0, kUGateBK))
    return MOE_ERR_CUDA;
  static PerDeviceOnce attr_set;
  if (!ensure_dynamic_smem(moe_gate_umma_kernel<NB64>, 202 * 1024, attr_set)) return MOE_ERR_CUDA;
  const int tiles = (s->T + kUGateTM - 1) / kUGateTM;
  const cudaError_t err = launch_dependent(
      moe_gate_umma_kernel<NB64>, dim3((unsigned)tiles, (unsigned)ks, 1), dim3(256), smem, stream, (unsigned)ks, tm_x, tm_w,
      gate_bias, (int)s->T, (int)s->H, (int)s->N, (int)s->K_orig, scores, topk_idx, topk_score, zero_ptr, zero_n,
      dev_status);
  return err == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

template <int NT16>
static moe_status gate_launch_nw(const moe_shape* s, const uint16_t* x, const uint16_t* W_gate, const float* gate_bias,
                                 float* scores, int32_t* topk_idx, float* topk_score, int32_t* zero_ptr, int zero_n,
                                 int32_t* dev_status, cudaStream_t stream) {
  if constexpr (NT16 == 4 || NT16 == 8) {
    int ks = 1;
    if (gate_umma_fits(s, &ks))
      return gate_launch_umma<NT16 / 4>(s, ks, x, W_gate, gate_bias, scores, topk_idx, topk_score, zero_ptr, zero_n,
                                        dev_status, stream);
  }
  if (s->T >= 2048)
    return gate_launch_t<NT16, 4>(s, x, W_gate, gate_bias, scores, topk_idx, topk_score, zero_ptr, zero_n, stream);
  return gate_launch_t<NT16, 2>(s, x, W_gate, gate_bias, scores, topk_idx, topk_score, zero_ptr, zero_n, stream);
}

// zero_ptr / zero_n: device ints the launch also clears (nullptr: none); dev_status: optional status word
moe_status launch_moe_gate(const moe_shape* s, const uint16_t* x, const uint16_t* W_gate, const float* gate_bias,
                           float* scores, int32_t* topk_idx, float* topk_score, int32_t* zero_ptr, int zero_n,
                           int32_t* dev_status, cudaStream_t stream) {
  const int nt16 = (s->N + 15) / 16;
  switch (nt16) {
    case 1: return gate_launch_nw<1>(s, x, W_gate, gate_bias, scores, topk_idx, topk_score, zero_ptr, zero_n, dev_status,
                                     stream);
    case 2: return gate_launch_nw<2>(s, x, W_gate, gate_bias, scores, topk_idx, topk_score, zero_ptr, zero_n, dev_status,
                                     stream);
    case 3: return gate_launch_nw<3>(s, x, W_gate, gate_bias, scores, topk_idx, topk_score, zero_ptr, zero_n, dev_status,
                                     stream);
    case 4: return gate_launch_nw<4>(s, x, W_gate, gate_bias, scores, topk_idx, topk_score, zero_ptr, zero_n, dev_status,
                                     stream);
    case 5: return gate_launch_nw<5>(s, x, W_gate, gate_bias, scores, topk_idx, topk_score, zero_ptr, zero_n, dev_status,
                                     stream);
    case 6: return gate_launch_nw<6>(s, x, W_gate, gate_bias, scores, topk_idx, topk_score, zero_ptr, zero_n, dev_status,
                                     stream);
    case 7: return gate_launch_nw<7>(s, x, W_gate, gate_bias, scores, topk_idx, topk_score, zero_ptr, zero_n, dev_status,
                                     stream);
    case 8: return gate_launch_nw<8>(s, x, W_gate, gate_bias, scores, topk_idx, topk_score, zero_ptr, zero_n, dev_status,
                                     stream);
    default: return MOE_ERR_ARG;
  }
}
