// Grouped SwiGLU expert GEMMs on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA.
//
// "Each activated expert corresponds to one feed-forward execution" (Sec. 3.1): for the rows of
// expert e (a contiguous run of the permuted list)
//     GEMM-1   h = silu(X W1_e^T) * (X W3_e^T)       [rows, I]   (SwiGLU fused in the epilogue)
//     GEMM-2   y = h W2_e^T                          [rows, H]
//
// The number of rows an expert receives is data dependent and, under a reduced budget, small and
// ragged (3 per expert at decode, 30-250 in the layer stack).  The tensor-core instruction has a
// fixed M of 128 but an N of any multiple of 16 up to 256, so the kernels compute the TRANSPOSED
// product: the UMMA "A" operand is a tile of 128 weight rows, the "B" operand is a tile of the
// expert's tokens whose width N is the expert's row count rounded up to 16.  No tensor-core time
// is spent on padding rows, and a token tile occupies only as much shared memory as it has rows.
//     D[128 weight rows, N tokens] = W_tile[128, K] . X_tile[N, K]^T      (both operands K-major)
// GEMM-1's weight tile interleaves 16 rows of W1 with the matching 16 rows of W3 (one 5-d TMA
// box), so an accumulator holds gate and up values of 64 h columns in neighbouring lanes of the
// same warp and the SwiGLU needs only a lane exchange.
//
// One persistent kernel per GEMM: grid = number of SMs, every CTA walks the tile list
// tile = blockIdx.x, += gridDim.x.  The list is built on the device from expert_offsets: groups in
// order (routed experts, then the shared experts as one group over all T rows); inside a group
// weight blocks outermost and token tiles innermost, so CTAs that run concurrently share a weight
// block through L2 and every weight byte leaves HBM once.
//
// CTA = 6 warps: one thread of warp 0 issues TMA loads into a ring of variable-size stages
// (16 KB of weights + 4 KB per 32 tokens, between 4 and 11 stages in flight); one thread of warp 1
// issues tcgen05.mma (M=128, N=16..256, K=16) into one of two 256-column TMEM accumulators;
// warps 2-5 read the finished accumulator with tcgen05.ld, apply the epilogue and store bf16
// while the next tile's main loop runs.  Every mbarrier wait is bounded (see common.cuh).
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"

namespace allocmoe {

constexpr int kWM = 128;                 // weight rows per tile (UMMA M)
constexpr int kBK = 64;                  // K per stage: 64 bf16 = one 128-byte swizzle row
constexpr int kMaxTok = 256;             // tokens per tile (UMMA N) at most
constexpr int kTokBox = 32;              // token rows per TMA box unit
constexpr int kFfnThreads = 192;
constexpr uint32_t kWBytes = kWM * kBK * 2;           // 16 KB
constexpr uint32_t kTokBoxBytes = kTokBox * kBK * 2;  // 4 KB
constexpr uint32_t kRingBytes = 220 * 1024;           // a multiple of the 4 KB stage granule
constexpr uint32_t kSlots = 16;          // barrier pairs (power of two); at most 11 stages fit the ring
constexpr int kTmemCols = 512;           // two accumulators of 256 columns
constexpr int kMaxGroups = 130;          // up to 128 routed experts + the shared group
constexpr int kGemm1Cols = 64;           // h columns per GEMM-1 tile (64 W1 rows + 64 W3 rows)

struct FfnGemmParams {
  const int32_t* expert_offsets;    // device [n_experts+1]; unused when n_experts == 0
  int n_experts;                    // routed groups
  int shared_rows;                  // T when the shared group is present, else 0
  int shared_sub;                   // S
  int n_per_sub;                    // output columns per (sub-)expert: I for GEMM-1, H for GEMM-2
  int k_per_sub;                    // K per (sub-)expert: H for GEMM-1, I for GEMM-2
  int tok_cap;                      // token rows per tile at most (multiple of 16, <= 256)
  __nv_bfloat16* out_routed;        // GEMM-1: h [rows, I]; GEMM-2: y_perm [rows, H]
  __nv_bfloat16* out_shared;        // GEMM-1: h_sh [T, S*I]; GEMM-2: y_shared [T, H]
  long long ld_out_routed, ld_out_shared;
  int32_t* dev_status;
};

// Tensor maps of one GEMM: weights and tokens of the routed experts [0] and of the shared group
// [1]; the token matrices have one map per box height (32, 64, 128, 256 rows).
struct FfnMaps {
  CUtensorMap w[2];
  CUtensorMap x[2][4];
};

struct FfnSmemCtl {
  uint64_t full[kSlots];
  uint64_t empty[kSlots];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  volatile int abort_flag;
  int n_groups;
  int total_tiles;
  uint32_t ent_v[kSlots];           // producer's record of where each live stage starts (ring position)
  int tile_start[kMaxGroups + 1];   // first tile of each group
  int row_start[kMaxGroups];        // first row of each group in its token / output matrix
  int row_count[kMaxGroups];
  int tok_tiles[kMaxGroups];        // token tiles per weight block
  int tile_rows[kMaxGroups];        // rows per token tile (multiple of 16)
};

struct TileCoord {
  int group, wb, m0, nvalid;
  bool shared;
  DEV int n_mma() const { return (nvalid + 15) & ~15; }
  DEV int n_box() const { return (nvalid + kTokBox - 1) / kTokBox; }   // 1..8 units of 32 token rows
  DEV uint32_t stage_bytes() const { return kWBytes + (uint32_t)n_box() * kTokBoxBytes; }
};

// Weight blocks per group.  GEMM-1: 64 h columns per block, the shared group has S sub-experts'
// worth; GEMM-2: 128 y columns per block.
template <bool kSwiGLU>
DEV int weight_blocks(const FfnGemmParams& p, bool shared) {
  if (kSwiGLU) return (p.n_per_sub / kGemm1Cols) * (shared ? p.shared_sub : 1);
  return (p.n_per_sub + kWM - 1) / kWM;
}

struct TileWalker {
  const FfnSmemCtl* c;
  int n_experts;
  int g;
  DEV TileWalker(const FfnSmemCtl* ctl, int n_exp) : c(ctl), n_experts(n_exp), g(0) {}
  DEV TileCoord at(int tile) {   // tiles must be asked for in ascending order, tile < total_tiles
    while (tile >= c->tile_start[g + 1]) ++g;
    TileCoord tc;
    tc.group = g;
    tc.shared = (g >= n_experts);
    const int local = tile - c->tile_start[g];
    const int tt = c->tok_tiles[g];
    tc.wb = local / tt;
    const int ti = local - tc.wb * tt;
    const int r0 = ti * c->tile_rows[g];
    tc.m0 = c->row_start[g] + r0;
    tc.nvalid = min(c->tile_rows[g], c->row_count[g] - r0);
    return tc;
  }
};

// The stage ring.  Stages of different sizes (a tile with few tokens needs less room) are carved
// out of one circular buffer in issue order: a stage starts where the previous one ended, or at
// offset 0 when it would run past the end.  Producer and MMA issuer walk the same tile list, so
// both derive every stage's offset, barrier slot (stage number mod kSlots) and phase on their
// own.  The producer also keeps a running position `vpos` that counts every byte passed, skipped
// ends included: a live stage that starts more than one ring length before the end of a new
// stage is exactly a stage the new one would overwrite, and since stages are consumed in issue
// order only the oldest live stage has to be looked at.

// kSwiGLU: true = GEMM-1, false = GEMM-2.
template <bool kSwiGLU>
__global__ void __launch_bounds__(kFfnThreads, 1)
ffn_gemm_kernel(const FfnGemmParams p, const __grid_constant__ FfnMaps maps) {
  extern __shared__ unsigned char smem_dyn[];
  // stages need 1024-byte alignment for the 128-byte swizzle
  unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  FfnSmemCtl* ctl = reinterpret_cast<FfnSmemCtl*>(ring + kRingBytes);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // ---------------- setup: group table, barriers, TMEM
  const int n_groups = p.n_experts + (p.shared_rows > 0 ? 1 : 0);
  for (int gi = tid; gi < n_groups; gi += kFfnThreads) {
    int lo = 0, rows = p.shared_rows;
    if (gi < p.n_experts) {
      lo = p.expert_offsets[gi];
      rows = max(p.expert_offsets[gi + 1] - lo, 0);
    }
    // even split into the fewest tiles of at most tok_cap rows, tile height a multiple of 16
    int tt = (rows + p.tok_cap - 1) / p.tok_cap;
    int tr = 16;
    if (rows > 0) {
      tr = (((rows + tt - 1) / tt) + 15) & ~15;
      tt = (rows + tr - 1) / tr;
    }
    ctl->row_start[gi] = lo;
    ctl->row_count[gi] = rows;
    ctl->tok_tiles[gi] = max(tt, 1);
    ctl->tile_rows[gi] = tr;
  }
  if (tid == 0) {
    for (uint32_t s = 0; s < kSlots; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tmem_full[a], 1); mbar_init(&ctl->tmem_empty[a], 4); }
    mbar_init(&ctl->drain, 1);
    ctl->abort_flag = 0;
    fence_barrier_init();
    for (int i = 0; i < 2; ++i) {
      prefetch_tensormap(&maps.w[i]);
      for (int c = 0; c < 4; ++c) prefetch_tensormap(&maps.x[i][c]);
    }
  }
  __syncthreads();
  if (tid == 0) {
    int acc = 0;
    for (int gi = 0; gi < n_groups; ++gi) {
      ctl->tile_start[gi] = acc;
      if (ctl->row_count[gi] > 0) acc += ctl->tok_tiles[gi] * weight_blocks<kSwiGLU>(p, gi >= p.n_experts);
    }
    ctl->tile_start[n_groups] = acc;
    ctl->total_tiles = acc;
    ctl->n_groups = n_groups;
  }
  if (warp == 1) {
    tmem_alloc(&ctl->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = ctl->tmem_base;
  const int total_tiles = ctl->total_tiles;
  const int kb_routed = p.k_per_sub / kBK;
  const int kb_shared = kSwiGLU ? kb_routed : kb_routed * p.shared_sub;
  const int wb_per_sub = p.n_per_sub / kGemm1Cols;   // GEMM-1 only
  volatile int* abort_flag = &ctl->abort_flag;

  if (warp == 0) {
    // ======================= TMA producer =======================
    if (lane == 0) {
      TileWalker w(ctl, p.n_experts);
      uint32_t head = 0, vpos = 0;      // ring offset and running position of the next stage
      uint32_t e = 0, tail = 0;         // stages issued; oldest stage not yet known to be consumed
      uint32_t tail_v = 0;              // running position at which stage `tail` starts
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const TileCoord tc = w.at(tile);
        const CUtensorMap* tmW = &maps.w[tc.shared ? 1 : 0];
        const CUtensorMap* tmX = maps.x[tc.shared ? 1 : 0];
        const int nkb = tc.shared ? kb_shared : kb_routed;
        const uint32_t bytes = tc.stage_bytes();
        const int nbox = tc.n_box();
        // weight coordinates of this tile: (sub-)expert and row block inside it
        int e_w = tc.group, blk = tc.wb;
        if (tc.shared) {
          if (kSwiGLU) { e_w = tc.wb / wb_per_sub; blk = tc.wb - e_w * wb_per_sub; }
          else { e_w = 0; }
        }
        for (int kb = 0; kb < nkb; ++kb) {
          if (head + bytes > kRingBytes) {
            vpos += kRingBytes - head;
            head = 0;
          }
          const uint32_t vend = vpos + bytes;
          // consumed first: every live stage the new one overlaps, and the previous user of this
          // barrier slot (differences of running positions are taken modulo 2^32)
          while (tail != e && ((int32_t)(tail_v + kRingBytes - vend) < 0 || e - tail >= kSlots)) {
            if (!(ok = mbar_wait_bounded(&ctl->empty[tail & (kSlots - 1)], (tail / kSlots) & 1u, abort_flag, p.dev_status)))
              break;
            ++tail;
            tail_v = ctl->ent_v[tail & (kSlots - 1)];   // meaningful only while tail != e
          }
          if (!ok) break;
          const uint32_t slot = e & (kSlots - 1);
          ctl->ent_v[slot] = vpos;
          if (tail == e) tail_v = vpos;
          unsigned char* sw = ring + head;
          unsigned char* sx = sw + kWBytes;
          uint64_t* bar = &ctl->full[slot];
          mbar_expect_tx(bar, bytes);
          if (kSwiGLU) {
            tma_load_5d(sw, tmW, bar, kb * kBK, 0, 0, blk * 4, e_w);
          } else {
            int e_k = e_w, k_col = kb * kBK;
            if (tc.shared) { e_k = kb / kb_routed; k_col = (kb - e_k * kb_routed) * kBK; }
            tma_load_3d(sw, tmW, bar, k_col, blk * kWM, e_k);
          }
          // token rows: the binary digits of nbox pick one box each of 256, 128, 64, 32 rows
          int done = 0;
#pragma unroll
          for (int c = 3; c >= 0; --c) {
            if (nbox - done >= (1 << c)) {
              tma_load_2d(sx + done * kTokBoxBytes, tmX + c, bar, kb * kBK, tc.m0 + done * kTokBox);
              done += 1 << c;
            }
          }
          head += bytes;
          vpos = vend;
          ++e;
        }
      }
      // drain: every load this thread issued must have landed before the CTA may exit
      for (uint32_t q = tail; q != e; ++q) mbar_wait_drain(&ctl->full[q & (kSlots - 1)], (q / kSlots) & 1u);
    }
  } else if (warp == 1) {
    // ======================= MMA issuer =======================
    if (lane == 0) {
      TileWalker w(ctl, p.n_experts);
      uint32_t head = 0, e = 0;
      uint32_t tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
        const TileCoord tc = w.at(tile);
        const int nkb = tc.shared ? kb_shared : kb_routed;
        const uint32_t bytes = tc.stage_bytes();
        const uint32_t idesc = umma_idesc_bf16(kWM, tc.n_mma());
        const uint32_t a = tcount & 1u, aph = (tcount >> 1) & 1u;
        if (!(ok = mbar_wait_bounded(&ctl->tmem_empty[a], aph ^ 1u, abort_flag, p.dev_status))) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + a * kMaxTok;
        for (int kb = 0; kb < nkb; ++kb) {
          if (head + bytes > kRingBytes) head = 0;
          const uint32_t slot = e & (kSlots - 1);
          if (!(ok = mbar_wait_bounded(&ctl->full[slot], (e / kSlots) & 1u, abort_flag, p.dev_status))) break;
          tc_fence_after_sync();
          const uint32_t sw = smem_u32(ring + head);
          const uint64_t dw = umma_desc_sw128(sw), dx = umma_desc_sw128(sw + kWBytes);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            umma_bf16(d_tmem, dw + (uint64_t)(k * 2), dx + (uint64_t)(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit(&ctl->empty[slot]);   // frees the stage once these MMAs have read it
          head += bytes;
          ++e;
        }
        if (ok) umma_commit(&ctl->tmem_full[a]);
      }
      // drain: all MMAs complete before TMEM is freed
      umma_commit(&ctl->drain);
      mbar_wait_drain(&ctl->drain, 0u);
    }
  } else {
    // ======================= epilogue (warps 2..5) =======================
    TileWalker w(ctl, p.n_experts);
    const int q = warp & 3;                  // TMEM lane quarter this warp may read
    const bool odd = (lane & 1) != 0;
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      const TileCoord tc = w.at(tile);
      const uint32_t a = tcount & 1u, aph = (tcount >> 1) & 1u;
      if (!(ok = mbar_wait_bounded_warp(&ctl->tmem_full[a], aph, abort_flag, p.dev_status))) break;
      tc_fence_after_sync();
      __nv_bfloat16* out = tc.shared ? p.out_shared : p.out_routed;
      const long long ld = tc.shared ? p.ld_out_shared : p.ld_out_routed;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * kMaxTok;
      const int nchunks = (tc.nvalid + 31) / 32;
      if (kSwiGLU) {
        // lanes 0-15 of the warp hold the gate rows of h columns col0 + 16q + (0..15), lanes 16-31
        // the up rows of the same columns.  After the exchange lane l < 16 owns tokens 0-15 of the
        // 32-token chunk for its column and lane l+16 owns tokens 16-31.
        const bool hi = lane >= 16;
        // first h column of the tile: wb = sub * (I/64) + block, so wb * 64 = sub * I + block * 64
        const int col_pair = tc.wb * kGemm1Cols + 16 * q + (lane & 14);
#pragma unroll 1
        for (int c = 0; c < nchunks; ++c) {
          uint32_t v[32];
          tmem_ld_32x32(taddr + c * 32, v);
          tmem_ld_wait();
          float hv[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float mine_lo = __uint_as_float(v[i]), mine_hi = __uint_as_float(v[16 + i]);
            const float recv = __shfl_xor_sync(0xffffffffu, hi ? mine_lo : mine_hi, 16);
            const float g = hi ? recv : mine_lo;
            const float u = hi ? mine_hi : recv;
            hv[i] = g * u / (1.f + __expf(-g));
          }
          // pair neighbouring columns: the even lane stores tokens 0-7 of its 16, the odd lane 8-15
          const int tl0 = c * 32 + (hi ? 16 : 0) + (odd ? 8 : 0);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float recv = __shfl_xor_sync(0xffffffffu, odd ? hv[i] : hv[8 + i], 1);
            const uint32_t packed = odd ? pack_bf16x2(recv, hv[8 + i]) : pack_bf16x2(hv[i], recv);
            const int tl = tl0 + i;
            if (tl < tc.nvalid)
              *reinterpret_cast<uint32_t*>(out + (long long)(tc.m0 + tl) * ld + col_pair) = packed;
          }
        }
      } else {
        // lane l holds y column col0 + 32q + l for the chunk's 32 tokens
        const int col_pair = tc.wb * kWM + 32 * q + (lane & 30);
        const bool col_ok = col_pair < p.n_per_sub;
#pragma unroll 1
        for (int c = 0; c < nchunks; ++c) {
          uint32_t v[32];
          tmem_ld_32x32(taddr + c * 32, v);
          tmem_ld_wait();
          const int tl0 = c * 32 + (odd ? 16 : 0);
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float mine_lo = __uint_as_float(v[i]), mine_hi = __uint_as_float(v[16 + i]);
            const float recv = __shfl_xor_sync(0xffffffffu, odd ? mine_lo : mine_hi, 1);
            const uint32_t packed = odd ? pack_bf16x2(recv, mine_hi) : pack_bf16x2(mine_lo, recv);
            const int tl = tl0 + i;
            if (col_ok && tl < tc.nvalid)
              *reinterpret_cast<uint32_t*>(out + (long long)(tc.m0 + tl) * ld + col_pair) = packed;
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->tmem_empty[a]);
    }
  }

  // ---------------- teardown
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace allocmoe

using namespace allocmoe;

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor of `rank` dimensions (dims[0] contiguous; strides in elements for dims 1..rank-1),
// 128-byte swizzle, out-of-range elements read as zero.
static bool make_tmap(CUtensorMap* tm, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_elems,
                      const uint32_t* box) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], es[5];
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) st[i] = strides_elems[i] * 2;
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Token matrix [rows, K], K contiguous with row stride ld: four maps with boxes of 32, 64, 128 and
// 256 rows x 64 columns.
static bool make_tmap_tokens(CUtensorMap* tm4, const void* base, uint64_t K, uint64_t rows, uint64_t ld) {
  const uint64_t dims[2] = {K, rows}, st[1] = {ld};
  bool ok = true;
  for (int c = 0; c < 4; ++c) {
    const uint32_t box[2] = {(uint32_t)kBK, (uint32_t)(kTokBox << c)};
    ok &= make_tmap(&tm4[c], base, 2, dims, st, box);
  }
  return ok;
}

// W13 [E, 2I, H]: one box = for each of 4 consecutive 16-row blocks, 16 rows of W1 then the same
// 16 rows of W3 (128 rows x 64 columns).  Dimensions (H, 16, 2, I/16, E).
static bool make_tmap_w13(CUtensorMap* tm, const void* base, uint64_t H, uint64_t I, uint64_t E) {
  const uint64_t dims[5] = {H, 16, 2, I / 16, E};
  const uint64_t st[4] = {H, I * H, 16 * H, 2 * I * H};
  const uint32_t box[5] = {(uint32_t)kBK, 16, 2, 4, 1};
  return make_tmap(tm, base, 5, dims, st, box);
}

// W2 [E, H, I]: boxes of 128 rows x 64 columns of one expert.
static bool make_tmap_w2(CUtensorMap* tm, const void* base, uint64_t H, uint64_t I, uint64_t E) {
  const uint64_t dims[3] = {I, H, E};
  const uint64_t st[2] = {I, H * I};
  const uint32_t box[3] = {(uint32_t)kBK, (uint32_t)kWM, 1};
  return make_tmap(tm, base, 3, dims, st, box);
}

static int g_num_sms = 0;
static int num_sms() {
  if (g_num_sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (g_num_sms <= 0) g_num_sms = 148;
  }
  return g_num_sms;
}

constexpr size_t kFfnSmemBytes = (size_t)kRingBytes + sizeof(FfnSmemCtl) + 1024;
static_assert(kFfnSmemBytes <= 232448, "ring + control block exceed the 227 KB a CTA may use");

template <bool kSwiGLU>
static moe_status launch_gemm(const FfnGemmParams& p, const FfnMaps& maps, cudaStream_t stream) {
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(ffn_gemm_kernel<kSwiGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kFfnSmemBytes) != cudaSuccess)
      return MOE_ERR_CUDA;
    attr_done = true;
  }
  ffn_gemm_kernel<kSwiGLU><<<num_sms(), kFfnThreads, kFfnSmemBytes, stream>>>(p, maps);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

// Token rows per tile at most.  256 gives the tensor cores their widest instruction; when experts
// receive few rows the tiles are small anyway and the cap does not bind.
static int token_tile_cap() {
  static int cap = 0;
  if (cap == 0) {
    cap = kMaxTok;
    const char* e = getenv("ALLOCMOE_TOKEN_TILE");   // tuning knob: 16..256, multiple of 16
    if (e != nullptr) {
      const int v = atoi(e);
      if (v >= 16 && v <= kMaxTok && v % 16 == 0) cap = v;
    }
  }
  return cap;
}

// Routed and/or shared experts in one pair of launches.
//   routed part present iff budget > 0 && x_perm != nullptr; shared part iff S > 0 && x_shared != nullptr.
moe_status launch_ffn(const moe_shape* s, const uint16_t* x_perm, const int32_t* expert_offsets, int64_t budget,
                      const uint16_t* W13, const uint16_t* W2, uint16_t* h, uint16_t* y_perm, const uint16_t* x_shared,
                      const uint16_t* Wsh13, const uint16_t* Wsh2, uint16_t* h_sh, uint16_t* y_shared,
                      int32_t* dev_status, cudaStream_t stream, cudaEvent_t between) {
  const bool routed = (budget > 0 && x_perm != nullptr);
  const bool shared = (s->S > 0 && x_shared != nullptr);
  if (!routed && !shared) return MOE_OK;
  const uint64_t H = s->H, I = s->I;
  FfnMaps m1, m2;   // GEMM-1, GEMM-2
  bool ok = true;
  if (routed) {
    ok &= make_tmap_w13(&m1.w[0], W13, H, I, (uint64_t)s->N);
    ok &= make_tmap_tokens(m1.x[0], x_perm, H, (uint64_t)budget, H);
    ok &= make_tmap_w2(&m2.w[0], W2, H, I, (uint64_t)s->N);
    ok &= make_tmap_tokens(m2.x[0], h, I, (uint64_t)budget, I);
  }
  if (shared) {
    const uint64_t S = s->S;
    ok &= make_tmap_w13(&m1.w[1], Wsh13, H, I, S);
    ok &= make_tmap_tokens(m1.x[1], x_shared, H, (uint64_t)s->T, H);
    ok &= make_tmap_w2(&m2.w[1], Wsh2, H, I, S);
    ok &= make_tmap_tokens(m2.x[1], h_sh, S * I, (uint64_t)s->T, S * I);
  }
  if (!ok) return MOE_ERR_CUDA;
  if (!(routed && shared)) {   // an absent part is never addressed; give its maps valid contents all the same
    const int have = routed ? 0 : 1, miss = routed ? 1 : 0;
    for (FfnMaps* m : {&m1, &m2}) {
      m->w[miss] = m->w[have];
      for (int c = 0; c < 4; ++c) m->x[miss][c] = m->x[have][c];
    }
  }

  FfnGemmParams p{};
  p.expert_offsets = expert_offsets;
  p.n_experts = routed ? s->N : 0;
  p.shared_rows = shared ? s->T : 0;
  p.shared_sub = s->S;
  p.tok_cap = token_tile_cap();
  p.dev_status = dev_status;
  // GEMM-1
  p.n_per_sub = s->I;
  p.k_per_sub = s->H;
  p.out_routed = reinterpret_cast<__nv_bfloat16*>(h);
  p.out_shared = reinterpret_cast<__nv_bfloat16*>(h_sh);
  p.ld_out_routed = s->I;
  p.ld_out_shared = (long long)s->S * s->I;
  moe_status st = launch_gemm<true>(p, m1, stream);
  if (st != MOE_OK) return st;
  if (between != nullptr) cudaEventRecord(between, stream);
  // GEMM-2
  p.n_per_sub = s->H;
  p.k_per_sub = s->I;
  p.out_routed = reinterpret_cast<__nv_bfloat16*>(y_perm);
  p.out_shared = reinterpret_cast<__nv_bfloat16*>(y_shared);
  p.ld_out_routed = s->H;
  p.ld_out_shared = s->H;
  return launch_gemm<false>(p, m2, stream);
}
