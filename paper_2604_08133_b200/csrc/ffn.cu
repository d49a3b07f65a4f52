// Grouped SwiGLU expert GEMMs on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA.
//
// One expert feed-forward execution per kept (token, expert) pair (Sec. 3.1): for the rows of
// expert e (a contiguous run of the permuted list)
//     GEMM-1   h = silu(X W1_e^T) * (X W3_e^T)       [rows, I]   (SwiGLU fused in the epilogue)
//     GEMM-2   y = h W2_e^T                          [rows, H]
// Both are C = A B^T with A [rows, K] and B [n, K] K-contiguous, i.e. both operands K-major.
//
// One persistent kernel per GEMM: grid = number of SMs, every CTA walks the tile list
// tile = blockIdx.x, += gridDim.x (TileSched).  The list is built on the device from expert_offsets
// (row counts are data dependent): groups in order, inside a group column blocks outermost and
// 128-row blocks innermost, so CTAs that run concurrently share a weight tile through L2.
// A "group" is the shared experts (first; all T rows; their S sub-experts are extra column blocks
// in GEMM-1 and extra K blocks in GEMM-2, which makes those the longest tiles) or a routed expert.
//
// CTA = 6 warps: warp 0 lane 0 issues TMA loads (A 128x64, B 256x64 or 128x64 bf16, 128-byte
// swizzle) into a ring of 4 (6) stages; warp 1 lane 0 issues tcgen05.mma (M=128, N=256 or 128,
// K=16) into one of two TMEM accumulators; warps 2-5 read the finished accumulator with
// tcgen05.ld, apply the epilogue and store bf16 rows (row-masked at the ragged end of an expert's
// run) while the next tile's main loop runs.  Every wait is bounded (see common.cuh).
// Where expert runs are short (FfnGemmParams::gather_rows) the A rows do not come as one 128-row box:
// the 32 lanes of warp 0 fetch four rows each with tile::gather4 loads -- for GEMM-1 straight from x
// through perm_token, so no permuted copy of x exists -- and skip the rows past the run's end.
//
// Two variants of the kernel: one CTA per 128-row tile (ffn_gemm_kernel) and a CTA pair per 256-row
// tile (ffn_gemm_pair_kernel, tcgen05 cta_group::2); launch_ffn picks by shape.  GEMM-2 is launched
// as a programmatic dependent that does not wait for the whole of GEMM-1: per block of token rows
// GEMM-1's epilogue counts finished tiles of h and GEMM-2's producer loads a block once its count is
// complete, so GEMM-2 fills the SMs that GEMM-1's last round of tiles leaves idle.
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"
#include "ffn.h"

namespace allocmoe {

constexpr int kBM = 128;            // rows per tile (UMMA M)
constexpr int kBK = 64;             // K per stage: 64 bf16 = one 128-byte swizzle row
constexpr int kAccCols = 256;       // TMEM columns reserved per accumulator
constexpr int kMaxStages = 6;
constexpr int kFfnThreads = 192;
constexpr int kABytes = kBM * kBK * 2;        // 16 KB
constexpr int kTmemCols = 512;      // two accumulators of 256 columns

// The B tile (weight rows = UMMA N) is 256 rows (4 stages of 48 KB) or 128 rows (6 stages of 32 KB).
template <int kN>
struct TileCfg {
  static constexpr int kBBytes = kN * kBK * 2;             // 32 or 16 KB
  static constexpr int kStageBytes = kABytes + kBBytes;    // 48 or 32 KB
  static constexpr int kStages = kN == 256 ? 4 : 6;
  static constexpr size_t kSmemBytes = (size_t)kStages * kStageBytes;
};
constexpr int kMaxGroups = 130;     // up to 128 routed experts + the shared group

struct FfnGemmParams {
  const int32_t* expert_offsets;    // device [n_experts+1]; unused when n_experts == 0
  int n_experts;                    // routed groups
  int routed_rows;                  // rows of the routed A / output matrices (the budget)
  int shared_rows;                  // T when the shared group is present, else 0
  int shared_sub;                   // S
  int n_per_sub;                    // output columns per (sub-)expert: I for GEMM-1, H for GEMM-2
  int k_per_sub;                    // K per (sub-)expert: H for GEMM-1, I for GEMM-2
  int up_row_offset;                // GEMM-1: row of W3 inside an expert's W13 (= I)
  __nv_bfloat16* out_routed;        // GEMM-1: h [rows, I]; GEMM-2: y_perm [rows, H]
  __nv_bfloat16* out_shared;        // GEMM-1: h_sh [T, S*I]; GEMM-2: y_shared [T, H]
  long long ld_out_routed, ld_out_shared;
  int32_t* dev_status;
  // GEMM-2 may start while GEMM-1 is still running: per block of token rows, GEMM-1 counts the tiles
  // of h it has finished (done[block], once per epilogue warp) and GEMM-2 loads a block's rows once
  // the count reaches dep_need_* (GEMM-1's tiles per block x epilogue warps).  nullptr = no tracking.
  // Invariant: a GEMM-2 launch that was handed `done` does not complete before the GEMM-1 launch ahead of it
  // in the stream has (it executes griddepcontrol.wait in its teardown at the latest, also when a bounded
  // wait gave up), so whatever follows GEMM-2 in the stream may reuse h, `done` and the workspace.
  int32_t* done;
  int done_capacity;                // counters behind `done`; offsets that need more (inconsistent input) switch tracking off
  int dep_need_routed, dep_need_shared;
  long long wait_limit_clk;         // limit of every bounded wait of the launch, in SM clocks (kWaitLimitClk)
  // gather_rows > 0: the routed A tensor map has a box one row high and the producer warp fetches a
  // tile's rows four per TMA instruction, only those that hold rows of the expert's run.  GEMM-1 can
  // then read the routed tokens' rows straight from x instead of a permuted copy: row m of the routed
  // A matrix is x[gather_idx[m]] (gather_idx = perm_token, gather_rows entries); with gather_idx ==
  // nullptr row m is row m (GEMM-2 on h).  gather_rows == 0: A rows come as one 128-row box.
  const int32_t* gather_idx;
  int gather_rows;
  int gather_src_rows;              // rows of the matrix the indices point into; indices are clamped to it
};

// Token rows a producer lane fetches per stage when A is gathered: lane l owns rows 4l..4l+3 of the tile.
struct GatherRows {
  int r[4];
  bool issue;          // this lane's four rows hold at least one row of the expert's run
  uint32_t a_bytes;    // bytes of A all lanes together bring in per stage
};
// Rows past the end of the run inside a fetched group of four take the index of the list's last valid
// entry; groups wholly past the end are not fetched at all (their rows of the accumulator are never
// stored), which at decode sizes leaves half a KB of A per stage instead of 16 KB.
DEV GatherRows gather_rows_of_tile(const FfnGemmParams& p, int a_row, int m_end, int lane, int tile_rows) {
  GatherRows g;
  const int valid = min(max(m_end - a_row, 0), tile_rows);
  g.issue = 4 * lane < valid;
  g.a_bytes = (uint32_t)((valid + 3) / 4) * 512u;
#pragma unroll
  for (int i = 0; i < 4; ++i) g.r[i] = 0;
  if (g.issue) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int m = min(a_row + 4 * lane + i, p.gather_rows - 1);
      // clamped: a routing step that reported an error may leave anything in the list
      g.r[i] = p.gather_idx != nullptr ? clamp_index(__ldg(p.gather_idx + m), 0, p.gather_src_rows - 1, p.dev_status) : m;
    }
  }
  return g;
}

struct FfnSmemCtl {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  volatile int abort_flag;
  int n_groups;
  int total_tiles;
  int track_done;                   // the row-block counters are in use (FfnGemmParams::done, done_capacity)
  int shared_tiles;                 // tiles of the shared group: they come first in the tile numbering
  int tile_start[kMaxGroups + 1];   // first tile of each routed group; [n_experts] = total_tiles
  int row_start[kMaxGroups];        // first row of each group in its A / output matrix
  int row_count[kMaxGroups];
  int mblock_start[kMaxGroups + 1]; // first row block of each group in the numbering of `done`
};

struct TileCoord {
  int group, m0, m_end, nb;
  int dep_id;       // index of the tile's row block in `done`
  bool shared;
};

// kSwiGLU: true = GEMM-1 (B tile = kN/2 W1 rows + kN/2 W3 rows, kN/2 output columns),
//          false = GEMM-2 (B tile = kN W2 rows, kN output columns).
template <bool kSwiGLU, int kN, int kTileM>
struct TileWalker {
  const FfnSmemCtl* c;
  int nb_routed, nb_shared;
  int g;
  DEV TileWalker(const FfnSmemCtl* ctl, const FfnGemmParams& p) : c(ctl), g(0) {
    constexpr int cols = kSwiGLU ? kN / 2 : kN;
    nb_routed = (p.n_per_sub + cols - 1) / cols;
    nb_shared = kSwiGLU ? nb_routed * p.shared_sub : nb_routed;
  }
  // tile ids handed to one walker never decrease
  DEV TileCoord at(int tile, const FfnGemmParams& p) {
    TileCoord tc;
    tc.shared = tile < c->shared_tiles;
    if (!tc.shared)
      while (tile >= c->tile_start[g + 1]) ++g;   // tile < total_tiles, tile_start is non-decreasing
    const int gi = tc.shared ? p.n_experts : g;
    tc.group = gi;
    const int local = tc.shared ? tile : tile - c->tile_start[gi];
    const int mblocks = (c->row_count[gi] + kTileM - 1) / kTileM;
    tc.nb = local / mblocks;
    const int mb = local % mblocks;
    tc.dep_id = c->mblock_start[gi] + mb;
    tc.m0 = c->row_start[gi] + mb * kTileM;
    tc.m_end = c->row_start[gi] + c->row_count[gi];
    return tc;
  }
};

// Which tiles a CTA (or CTA pair) works on, in order.  Normally tile c, c + G, c + 2G, ...  The shared
// group's tiles come first in the numbering, and in GEMM-2 each of them runs S times as long as a
// routed tile (K = S*I).  Handed out round-robin, the CTAs that got one would finish S - 1 tile
// times after the others, alone on the memory system; so while the shared tiles fit one round
// (n_sh <= G) the CTAs that hold one sit out the next w - 1 rounds of routed tiles (w = S).
struct TileSched {
  int c, G, n_sh, w;
  bool skip;
  DEV TileSched(int cta, int n_ctas, int shared_tiles, int weight)
      : c(cta), G(n_ctas), n_sh(shared_tiles), w(weight), skip(shared_tiles <= n_ctas && weight > 1) {}
  DEV int tile(int k) const {      // the CTA's k-th tile; increases with k; >= total_tiles ends the walk
    if (!skip) return c + k * G;
    const int free = G - n_sh;     // CTAs without a shared tile
    if (c < n_sh) return k == 0 ? c : n_sh + w * free + c + (k - 1) * G;
    return k < w ? c + k * free : n_sh + w * free + c + (k - w) * G;
  }
};

// One warp: first tile and first row block of every group from the groups' row counts (the shared group's tiles
// and row blocks are numbered first, the routed groups follow in order; every routed group has nb_routed column
// blocks).  Lane l takes a run of consecutive experts, a warp scan joins the runs.
template <int kTileM>
DEV void build_tile_table(FfnSmemCtl* ctl, const FfnGemmParams& p, int nb_routed, int nb_shared, int n_groups) {
  const int lane = threadIdx.x & 31;
  const int sh_mblocks = p.shared_rows > 0 ? (p.shared_rows + kTileM - 1) / kTileM : 0;
  const int sh_tiles = sh_mblocks * nb_shared;
  const int per = (p.n_experts + 31) / 32;
  const int g0 = min(lane * per, p.n_experts), g1 = min(g0 + per, p.n_experts);
  int mb = 0;
  for (int g = g0; g < g1; ++g) mb += (ctl->row_count[g] + kTileM - 1) / kTileM;
  int incl = mb;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  int before = incl - mb;   // routed row blocks of lower experts
  for (int g = g0; g < g1; ++g) {
    ctl->mblock_start[g] = sh_mblocks + before;
    ctl->tile_start[g] = sh_tiles + before * nb_routed;
    before += (ctl->row_count[g] + kTileM - 1) / kTileM;
  }
  const int routed_mblocks = __shfl_sync(0xffffffffu, incl, 31);
  if (lane == 0) {
    const int total = sh_tiles + routed_mblocks * nb_routed;
    ctl->shared_tiles = sh_tiles;
    ctl->mblock_start[p.n_experts] = 0;
    ctl->tile_start[p.n_experts] = total;
    ctl->total_tiles = total;
    ctl->n_groups = n_groups;
    ctl->track_done = (p.done != nullptr && sh_mblocks + routed_mblocks <= p.done_capacity) ? 1 : 0;
  }
}

template <bool kSwiGLU, int kN>
__global__ void __launch_bounds__(kFfnThreads, 1)
ffn_gemm_kernel(const FfnGemmParams p, const __grid_constant__ CUtensorMap tmA_routed,
                const __grid_constant__ CUtensorMap tmB_routed, const __grid_constant__ CUtensorMap tmA_shared,
                const __grid_constant__ CUtensorMap tmB_shared) {
  extern __shared__ unsigned char smem_dyn[];
  // tiles need 1024-byte alignment for the 128-byte swizzle
  unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  FfnSmemCtl* ctl = reinterpret_cast<FfnSmemCtl*>(tiles + TileCfg<kN>::kSmemBytes);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int kStages = TileCfg<kN>::kStages, kStageBytes = TileCfg<kN>::kStageBytes, kBBytes = TileCfg<kN>::kBBytes;
  constexpr int kOutCols = kSwiGLU ? kN / 2 : kN;

  // ---------------- setup: barriers, TMEM (no global memory yet), then the group table
  const int n_groups = p.n_experts + (p.shared_rows > 0 ? 1 : 0);
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tmem_full[a], 1); mbar_init(&ctl->tmem_empty[a], 4); }
    mbar_init(&ctl->drain, 1);
    ctl->abort_flag = 0;
    fence_barrier_init();
    prefetch_tensormap(&tmA_routed);
    prefetch_tensormap(&tmB_routed);
    prefetch_tensormap(&tmA_shared);
    prefetch_tensormap(&tmB_shared);
  }
  if (warp == 1) {
    tmem_alloc(&ctl->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  // GEMM-1 waits for everything before it and only then lets GEMM-2 start, so a GEMM-2 CTA that finds
  // an SM free while GEMM-1 is in its last round sees complete routing data; GEMM-2 itself does not
  // wait for the whole of GEMM-1 but for the row blocks of h it needs (p.done).
  if (kSwiGLU || p.done == nullptr) pdl_wait();
  pdl_launch_dependents();   // expert_offsets and the operands come from earlier kernels of the stream
  for (int gi = tid; gi < n_groups; gi += kFfnThreads) {
    if (gi < p.n_experts) {
      // clamped to the routed matrices' rows: a routing step that reported an error may leave anything here
      const int lo = clamp_index(p.expert_offsets[gi], 0, p.routed_rows, p.dev_status);
      const int hi = clamp_index(p.expert_offsets[gi + 1], lo, p.routed_rows, p.dev_status);
      ctl->row_start[gi] = lo;
      ctl->row_count[gi] = hi - lo;
    } else {
      ctl->row_start[gi] = 0;
      ctl->row_count[gi] = p.shared_rows;
    }
  }
  __syncthreads();
  if (warp == 2) {
    TileWalker<kSwiGLU, kN, kBM> w(ctl, p);
    build_tile_table<kBM>(ctl, p, w.nb_routed, w.nb_shared, n_groups);
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = ctl->tmem_base;
  const int total_tiles = ctl->total_tiles;
  const bool track = ctl->track_done != 0;
  if (!kSwiGLU && p.done != nullptr && !track) pdl_wait();   // no counters to go by: wait for all of GEMM-1
  const TileSched sched((int)blockIdx.x, (int)gridDim.x, ctl->shared_tiles, kSwiGLU ? 1 : p.shared_sub);
  const int kb_routed = p.k_per_sub / kBK;
  const int kb_shared = kSwiGLU ? kb_routed : kb_routed * p.shared_sub;
  volatile int* abort_flag = &ctl->abort_flag;

  if (warp == 0) {
    // ======================= TMA producer =======================
    // Lane 0 issues the box loads.  With gathered A rows (FfnGemmParams::gather_rows) the whole warp runs
    // the loop and every lane fetches its four rows of a routed tile per stage.
    const bool gather = p.gather_rows > 0;
    if (lane == 0 || gather) {
      TileWalker<kSwiGLU, kN, kBM> w(ctl, p);
      uint32_t it = 0;
      bool ok = true;
      for (int k = 0; ok; ++k) {
        const int tile = sched.tile(k);
        if (tile >= total_tiles) break;
        const TileCoord tc = w.at(tile, p);
        const CUtensorMap* tmA = tc.shared ? &tmA_shared : &tmA_routed;
        const CUtensorMap* tmB = tc.shared ? &tmB_shared : &tmB_routed;
        const int nkb = tc.shared ? kb_shared : kb_routed;
        // expert coordinate and row inside the expert's weight matrix for this column block
        int e_n = tc.group, n_row = tc.nb * kOutCols;
        if (tc.shared) {
          if (kSwiGLU) { e_n = tc.nb / w.nb_routed; n_row = (tc.nb % w.nb_routed) * kOutCols; }
          else { e_n = 0; }
        }
        const bool gtile = gather && !tc.shared;
        GatherRows gr{};
        if (gtile) gr = gather_rows_of_tile(p, tc.m0, tc.m_end, lane, kBM);
        if (!kSwiGLU && track) {   // the block's rows of h are complete?
          if (lane == 0)
            ok = flag_wait_bounded(p.done + tc.dep_id, tc.shared ? p.dep_need_shared : p.dep_need_routed, abort_flag,
                                   p.dev_status, p.wait_limit_clk);
          if (gather) {
            __syncwarp();
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
          }
          if (!ok) break;
          fence_proxy_async_global();
        }
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          ok = gather ? mbar_wait_bounded_warp(&ctl->empty[s], ph ^ 1u, abort_flag, p.dev_status, p.wait_limit_clk)
                      : mbar_wait_bounded(&ctl->empty[s], ph ^ 1u, abort_flag, p.dev_status, p.wait_limit_clk);
          if (!ok) break;
          unsigned char* sa = tiles + s * kStageBytes;
          unsigned char* sb = sa + kABytes;
          if (lane == 0) {
            mbar_expect_tx(&ctl->full[s], gtile ? gr.a_bytes + kBBytes : kStageBytes);
            if (!gtile) tma_load_2d(sa, tmA, &ctl->full[s], kb * kBK, tc.m0);
            int e_k = e_n, k_col = kb * kBK;
            if (tc.shared && !kSwiGLU) { e_k = kb / kb_routed; k_col = (kb % kb_routed) * kBK; }
            if (kSwiGLU) {
              tma_load_3d(sb, tmB, &ctl->full[s], k_col, n_row, e_k);
              tma_load_3d(sb + kBBytes / 2, tmB, &ctl->full[s], k_col, p.up_row_offset + n_row, e_k);
            } else {
              tma_load_3d(sb, tmB, &ctl->full[s], k_col, n_row, e_k);
            }
          }
          if (gtile) {
            __syncwarp();   // the stage's byte count is announced before any lane's rows can land
            if (gr.issue) tma_gather4_2d(sa + lane * 512, tmA, &ctl->full[s], kb * kBK, gr.r[0], gr.r[1], gr.r[2], gr.r[3]);
          }
        }
      }
      // drain: every load this warp issued must have landed before the CTA may exit
      if (lane == 0) {
        const uint32_t issued = it;
        for (uint32_t q = (issued > (uint32_t)kStages ? issued - kStages : 0u); q < issued; ++q)
          mbar_wait_drain(&ctl->full[q % kStages], (q / kStages) & 1u);
      }
    }
  } else if (warp == 1) {
    // ======================= MMA issuer =======================
    if (lane == 0) {
      TileWalker<kSwiGLU, kN, kBM> w(ctl, p);
      constexpr uint32_t idesc = umma_idesc_bf16(kBM, kN);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int k = 0; ok; ++k, ++tcount) {
        const int tile = sched.tile(k);
        if (tile >= total_tiles) break;
        const TileCoord tc = w.at(tile, p);
        const int nkb = tc.shared ? kb_shared : kb_routed;
        const uint32_t a = tcount & 1u, aph = (tcount >> 1) & 1u;
        if (!(ok = mbar_wait_bounded(&ctl->tmem_empty[a], aph ^ 1u, abort_flag, p.dev_status, p.wait_limit_clk))) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + a * kAccCols;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!(ok = mbar_wait_bounded(&ctl->full[s], ph, abort_flag, p.dev_status, p.wait_limit_clk))) break;
          tc_fence_after_sync();
          const uint32_t sa = smem_u32(tiles + s * kStageBytes);
          const uint64_t da = umma_desc_sw128(sa), db = umma_desc_sw128(sa + kABytes);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            umma_bf16(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit(&ctl->empty[s]);      // frees the stage once these MMAs have read it
        }
        if (ok) umma_commit(&ctl->tmem_full[a]);
      }
      // drain: all MMAs complete before TMEM is freed
      umma_commit(&ctl->drain);
      mbar_wait_drain(&ctl->drain, 0u);
    }
  } else {
    // ======================= epilogue (warps 2..5) =======================
    TileWalker<kSwiGLU, kN, kBM> w(ctl, p);
    const int q = warp & 3;                  // TMEM lane quarter this warp may read
    uint32_t tcount = 0;
    bool ok = true;
    for (int k = 0; ok; ++k, ++tcount) {
      const int tile = sched.tile(k);
      if (tile >= total_tiles) break;
      const TileCoord tc = w.at(tile, p);
      const uint32_t a = tcount & 1u, aph = (tcount >> 1) & 1u;
      if (!(ok = mbar_wait_bounded_warp(&ctl->tmem_full[a], aph, abort_flag, p.dev_status, p.wait_limit_clk))) break;
      tc_fence_after_sync();
      const int row = tc.m0 + q * 32 + lane;
      const bool row_ok = row < tc.m_end;
      const int n_total = tc.shared ? (kSwiGLU ? p.n_per_sub * p.shared_sub : p.n_per_sub) : p.n_per_sub;
      int col0 = tc.nb * kOutCols;           // first output column of the tile
      int col_limit = n_total;
      if (kSwiGLU && tc.shared) {            // column block nb of sub-expert s -> column s*I + ...
        const int s = tc.nb / w.nb_routed;
        col0 = s * p.n_per_sub + (tc.nb % w.nb_routed) * kOutCols;
        col_limit = (s + 1) * p.n_per_sub;
      }
      __nv_bfloat16* out = tc.shared ? p.out_shared : p.out_routed;
      const long long ld = tc.shared ? p.ld_out_shared : p.ld_out_routed;
      __nv_bfloat16* out_row = out + (long long)row * ld;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * kAccCols;
      // a warp whose 32 rows all lie past the end of the expert's run has nothing to store: at
      // decode sizes (a few rows per expert) that is three warps of four
      const int n_chunks = (tc.m0 + q * 32 < tc.m_end) ? kOutCols / 32 : 0;
#pragma unroll 1
      for (int c = 0; c < n_chunks; ++c) {
        uint32_t packed[16];
        if (kSwiGLU) {
          uint32_t g[32], u[32];
          tmem_ld_32x32(taddr + c * 32, g);
          tmem_ld_32x32(taddr + kN / 2 + c * 32, u);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float g0 = __uint_as_float(g[2 * i]), g1 = __uint_as_float(g[2 * i + 1]);
            const float h0 = __fdividef(g0 * __uint_as_float(u[2 * i]), 1.f + __expf(-g0));
            const float h1 = __fdividef(g1 * __uint_as_float(u[2 * i + 1]), 1.f + __expf(-g1));
            packed[i] = pack_bf16x2(h0, h1);
          }
        } else {
          uint32_t v[32];
          tmem_ld_32x32(taddr + c * 32, v);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) packed[i] = pack_bf16x2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
        }
        const int col = col0 + c * 32;
        if (row_ok) {
          if (col + 32 <= col_limit) {
            uint4* dst = reinterpret_cast<uint4*>(out_row + col);
#pragma unroll
            for (int i = 0; i < 4; ++i) dst[i] = make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
          } else {
            for (int i = 0; i < 32; ++i)
              if (col + i < col_limit) {
                const uint32_t w2 = packed[i >> 1];
                reinterpret_cast<uint16_t*>(out_row)[col + i] = (uint16_t)((i & 1) ? (w2 >> 16) : (w2 & 0xFFFFu));
              }
          }
        }
      }
      if (kSwiGLU && track) {   // publish this warp's quarter of the tile (FfnGemmParams::done)
        __threadfence();
        __syncwarp();
        if (lane == 0) {
          fence_proxy_async_global();
          flag_add_release(p.done + tc.dep_id, 1);
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->tmem_empty[a]);
    }
  }

  // ---------------- teardown
  // GEMM-2 with row-block tracking has not waited for the whole of GEMM-1 yet.  It does so here, on the abort
  // path too, so that its completion implies GEMM-1's (FfnGemmParams::done); in the normal case GEMM-1 has
  // finished long before and the wait is free.
  if (!kSwiGLU && p.done != nullptr) pdl_wait();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}


// ------------------------------------------------------------------------------------------------
// The same GEMM on CTA pairs (cta_group::2).  A cluster of two CTAs on the two SMs of a TPC works on
// a tile of 256 rows x 256 weight rows: each CTA loads its own 128 rows of A and HALF of the B tile
// (for GEMM-1 the leader takes the 128 W1 rows, its peer the 128 W3 rows), the leader's MMA thread
// issues tcgen05.mma with M = 256 and both tensor cores read the two halves of B from both shared
// memories.  Per 128x256x64 block of MACs an SM now moves 32 KB from L2 instead of 48 KB and reads
// 8 KB instead of 12 KB of operands per MMA from shared memory -- the two paths that bound the
// one-CTA kernel on compute-heavy shapes -- and the ring holds 6 stages.
//
// Barriers: `full` lives in the leader and counts two arrivals (each CTA's producer announces its
// own 32 KB); `empty` and `tmem_full` exist in both CTAs and are signalled by multicast commits;
// `tmem_empty` lives in the leader and counts the 8 epilogue warps of the pair.  No load uses
// cluster multicast.
constexpr int kPairStages = 6;
constexpr int kPairStageBytes = 2 * kABytes;          // 16 KB of A + 16 KB of B per CTA
constexpr int kPairM = 2 * kBM;

template <bool kSwiGLU>
__global__ void __launch_bounds__(kFfnThreads, 1)
ffn_gemm_pair_kernel(const FfnGemmParams p, const __grid_constant__ CUtensorMap tmA_routed,
                     const __grid_constant__ CUtensorMap tmB_routed, const __grid_constant__ CUtensorMap tmA_shared,
                     const __grid_constant__ CUtensorMap tmB_shared) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  FfnSmemCtl* ctl = reinterpret_cast<FfnSmemCtl*>(tiles + kPairStages * kPairStageBytes);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int kN = 256;
  constexpr int kOutCols = kSwiGLU ? kN / 2 : kN;
  const uint32_t rank = cluster_cta_rank();          // 0 = leader
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  // ---------------- setup: barriers, TMEM (no global memory yet), then the group table
  const int n_groups = p.n_experts + (p.shared_rows > 0 ? 1 : 0);
  if (tid == 0) {
    for (int s = 0; s < kPairStages; ++s) { mbar_init(&ctl->full[s], 2); mbar_init(&ctl->empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&ctl->tmem_full[a], 1); mbar_init(&ctl->tmem_empty[a], 8); }
    mbar_init(&ctl->drain, 1);
    ctl->abort_flag = 0;
    fence_barrier_init();
    prefetch_tensormap(&tmA_routed);
    prefetch_tensormap(&tmB_routed);
    prefetch_tensormap(&tmA_shared);
    prefetch_tensormap(&tmB_shared);
  }
  if (warp == 1) {
    tmem_alloc_pair(&ctl->tmem_base, kTmemCols);
    tmem_relinquish_pair();
  }
  // GEMM-1 waits for everything before it and only then lets GEMM-2 start, so a GEMM-2 CTA that finds
  // an SM free while GEMM-1 is in its last round sees complete routing data; GEMM-2 itself does not
  // wait for the whole of GEMM-1 but for the row blocks of h it needs (p.done).
  if (kSwiGLU || p.done == nullptr) pdl_wait();
  pdl_launch_dependents();
  for (int gi = tid; gi < n_groups; gi += kFfnThreads) {
    if (gi < p.n_experts) {
      // clamped to the routed matrices' rows: a routing step that reported an error may leave anything here
      const int lo = clamp_index(p.expert_offsets[gi], 0, p.routed_rows, p.dev_status);
      const int hi = clamp_index(p.expert_offsets[gi + 1], lo, p.routed_rows, p.dev_status);
      ctl->row_start[gi] = lo;
      ctl->row_count[gi] = hi - lo;
    } else {
      ctl->row_start[gi] = 0;
      ctl->row_count[gi] = p.shared_rows;
    }
  }
  __syncthreads();
  if (warp == 2) {
    TileWalker<kSwiGLU, kN, kPairM> w(ctl, p);
    build_tile_table<kPairM>(ctl, p, w.nb_routed, w.nb_shared, n_groups);
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();          // both CTAs' barriers are initialised before either signals the other
  tc_fence_after_sync();
  const uint32_t tmem_base = ctl->tmem_base;
  const int total_tiles = ctl->total_tiles;
  const bool track = ctl->track_done != 0;
  if (!kSwiGLU && p.done != nullptr && !track) pdl_wait();   // no counters to go by: wait for all of GEMM-1
  const TileSched sched(pair_id, n_pairs, ctl->shared_tiles, kSwiGLU ? 1 : p.shared_sub);
  const int kb_routed = p.k_per_sub / kBK;
  const int kb_shared = kSwiGLU ? kb_routed : kb_routed * p.shared_sub;
  volatile int* abort_flag = &ctl->abort_flag;

  if (warp == 0) {
    // ======================= TMA producer (both CTAs) =======================
    const bool gather = p.gather_rows > 0;   // see the one-CTA kernel
    if (lane == 0 || gather) {
      TileWalker<kSwiGLU, kN, kPairM> w(ctl, p);
      uint32_t it = 0;
      bool ok = true;
      for (int k = 0; ok; ++k) {
        const int tile = sched.tile(k);
        if (tile >= total_tiles) break;
        const TileCoord tc = w.at(tile, p);
        const CUtensorMap* tmA = tc.shared ? &tmA_shared : &tmA_routed;
        const CUtensorMap* tmB = tc.shared ? &tmB_shared : &tmB_routed;
        const int nkb = tc.shared ? kb_shared : kb_routed;
        int e_n = tc.group, n_row = tc.nb * kOutCols;
        if (tc.shared) {
          if (kSwiGLU) { e_n = tc.nb / w.nb_routed; n_row = (tc.nb % w.nb_routed) * kOutCols; }
          else { e_n = 0; }
        }
        // this CTA's half of the B tile: GEMM-1 W1 rows (leader) or W3 rows (peer); GEMM-2 rows +128*rank
        const int b_row = kSwiGLU ? (rank == 0 ? n_row : p.up_row_offset + n_row) : n_row + (int)rank * (kN / 2);
        const int a_row = tc.m0 + (int)rank * kBM;
        const bool gtile = gather && !tc.shared;
        GatherRows gr{};
        if (gtile) gr = gather_rows_of_tile(p, a_row, tc.m_end, lane, kBM);
        if (!kSwiGLU && track) {   // the block's rows of h are complete?
          if (lane == 0)
            ok = flag_wait_bounded(p.done + tc.dep_id, tc.shared ? p.dep_need_shared : p.dep_need_routed, abort_flag,
                                   p.dev_status, p.wait_limit_clk);
          if (gather) {
            __syncwarp();
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
          }
          if (!ok) break;
          fence_proxy_async_global();
        }
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % kPairStages;
          const uint32_t ph = (it / kPairStages) & 1u;
          ok = gather ? mbar_wait_bounded_warp(&ctl->empty[s], ph ^ 1u, abort_flag, p.dev_status, p.wait_limit_clk)
                      : mbar_wait_bounded(&ctl->empty[s], ph ^ 1u, abort_flag, p.dev_status, p.wait_limit_clk);
          if (!ok) break;
          unsigned char* sa = tiles + s * kPairStageBytes;
          unsigned char* sb = sa + kABytes;
          const uint32_t bar = cluster_addr_of(&ctl->full[s], 0);
          if (lane == 0) {
            mbar_expect_tx_cluster(bar, gtile ? gr.a_bytes + kABytes : kPairStageBytes);
            if (!gtile) tma_load_2d_pair(sa, tmA, bar, kb * kBK, a_row);
            int e_k = e_n, k_col = kb * kBK;
            if (tc.shared && !kSwiGLU) { e_k = kb / kb_routed; k_col = (kb % kb_routed) * kBK; }
            tma_load_3d_pair(sb, tmB, bar, k_col, b_row, e_k);
          }
          if (gtile) {
            __syncwarp();   // the stage's byte count is announced before any lane's rows can land
            if (gr.issue) tma_gather4_2d_pair(sa + lane * 512, tmA, bar, kb * kBK, gr.r[0], gr.r[1], gr.r[2], gr.r[3]);
          }
        }
      }
      // drain: the last loads have landed once the leader's barriers of the last stages completed;
      // the peer learns it through the multicast `empty` that follows.  Wait for what was issued.
      if (lane == 0) {
        const uint32_t issued = it;
        if (rank == 0) {
          for (uint32_t q = (issued > (uint32_t)kPairStages ? issued - kPairStages : 0u); q < issued; ++q)
            mbar_wait_drain(&ctl->full[q % kPairStages], (q / kPairStages) & 1u);
        } else {
          for (uint32_t q = (issued > (uint32_t)kPairStages ? issued - kPairStages : 0u); q < issued; ++q)
            mbar_wait_drain(&ctl->empty[q % kPairStages], (q / kPairStages) & 1u);
        }
      }
    }
  } else if (warp == 1) {
    // ======================= MMA issuer (leader only) =======================
    if (lane == 0 && rank == 0) {
      TileWalker<kSwiGLU, kN, kPairM> w(ctl, p);
      constexpr uint32_t idesc = umma_idesc_bf16(kPairM, kN);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int k = 0; ok; ++k, ++tcount) {
        const int tile = sched.tile(k);
        if (tile >= total_tiles) break;
        const TileCoord tc = w.at(tile, p);
        const int nkb = tc.shared ? kb_shared : kb_routed;
        const uint32_t a = tcount & 1u, aph = (tcount >> 1) & 1u;
        if (!(ok = mbar_wait_bounded(&ctl->tmem_empty[a], aph ^ 1u, abort_flag, p.dev_status, p.wait_limit_clk))) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + a * kAccCols;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % kPairStages;
          const uint32_t ph = (it / kPairStages) & 1u;
          if (!(ok = mbar_wait_bounded(&ctl->full[s], ph, abort_flag, p.dev_status, p.wait_limit_clk))) break;
          tc_fence_after_sync();
          const uint32_t sa = smem_u32(tiles + s * kPairStageBytes);
          const uint64_t da = umma_desc_sw128(sa), db = umma_desc_sw128(sa + kABytes);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            umma_bf16_pair(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit_pair(&ctl->empty[s], 3);      // frees the stage in both CTAs
        }
        if (ok) umma_commit_pair(&ctl->tmem_full[a], 3);
      }
      // drain: all MMAs complete before TMEM is freed
      umma_commit_pair(&ctl->drain, 1);
      mbar_wait_drain(&ctl->drain, 0u);
    }
  } else {
    // ======================= epilogue (warps 2..5 of both CTAs) =======================
    TileWalker<kSwiGLU, kN, kPairM> w(ctl, p);
    const int q = warp & 3;
    uint32_t tcount = 0;
    bool ok = true;
    for (int k = 0; ok; ++k, ++tcount) {
      const int tile = sched.tile(k);
      if (tile >= total_tiles) break;
      const TileCoord tc = w.at(tile, p);
      const uint32_t a = tcount & 1u, aph = (tcount >> 1) & 1u;
      if (!(ok = mbar_wait_bounded_warp(&ctl->tmem_full[a], aph, abort_flag, p.dev_status, p.wait_limit_clk))) break;
      tc_fence_after_sync();
      const int row0 = tc.m0 + (int)rank * kBM + q * 32;
      const int row = row0 + lane;
      const bool row_ok = row < tc.m_end;
      const int n_total = tc.shared ? (kSwiGLU ? p.n_per_sub * p.shared_sub : p.n_per_sub) : p.n_per_sub;
      int col0 = tc.nb * kOutCols;
      int col_limit = n_total;
      if (kSwiGLU && tc.shared) {
        const int s = tc.nb / w.nb_routed;
        col0 = s * p.n_per_sub + (tc.nb % w.nb_routed) * kOutCols;
        col_limit = (s + 1) * p.n_per_sub;
      }
      __nv_bfloat16* out = tc.shared ? p.out_shared : p.out_routed;
      const long long ld = tc.shared ? p.ld_out_shared : p.ld_out_routed;
      __nv_bfloat16* out_row = out + (long long)row * ld;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * kAccCols;
      const int n_chunks = (row0 < tc.m_end) ? kOutCols / 32 : 0;
#pragma unroll 1
      for (int c = 0; c < n_chunks; ++c) {
        uint32_t packed[16];
        if (kSwiGLU) {
          uint32_t g[32], u[32];
          tmem_ld_32x32(taddr + c * 32, g);
          tmem_ld_32x32(taddr + kN / 2 + c * 32, u);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float g0 = __uint_as_float(g[2 * i]), g1 = __uint_as_float(g[2 * i + 1]);
            const float h0 = __fdividef(g0 * __uint_as_float(u[2 * i]), 1.f + __expf(-g0));
            const float h1 = __fdividef(g1 * __uint_as_float(u[2 * i + 1]), 1.f + __expf(-g1));
            packed[i] = pack_bf16x2(h0, h1);
          }
        } else {
          uint32_t v[32];
          tmem_ld_32x32(taddr + c * 32, v);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) packed[i] = pack_bf16x2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
        }
        const int col = col0 + c * 32;
        if (row_ok) {
          if (col + 32 <= col_limit) {
            uint4* dst = reinterpret_cast<uint4*>(out_row + col);
#pragma unroll
            for (int i = 0; i < 4; ++i) dst[i] = make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
          } else {
            for (int i = 0; i < 32; ++i)
              if (col + i < col_limit) {
                const uint32_t w2 = packed[i >> 1];
                reinterpret_cast<uint16_t*>(out_row)[col + i] = (uint16_t)((i & 1) ? (w2 >> 16) : (w2 & 0xFFFFu));
              }
          }
        }
      }
      if (kSwiGLU && track) {   // publish this warp's quarter of the tile (FfnGemmParams::done)
        __threadfence();
        __syncwarp();
        if (lane == 0) {
          fence_proxy_async_global();
          flag_add_release(p.done + tc.dep_id, 1);
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(cluster_addr_of(&ctl->tmem_empty[a], 0));
    }
  }

  // ---------------- teardown: neither CTA leaves (or frees TMEM) while its peer may still touch it
  if (!kSwiGLU && p.done != nullptr) pdl_wait();   // GEMM-2's completion implies GEMM-1's (see the one-CTA kernel)
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

}  // namespace allocmoe

using namespace allocmoe;

// ------------------------------------------------------------------ host side
#include "tmap.h"

// SM count of the current device (the persistent kernels' grid), looked up once per device.
static PerDeviceInt g_num_sms;
static int num_sms() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  int n = g_num_sms.get(dev);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    g_num_sms.set(dev, n);
  }
  return n;
}


template <bool kSwiGLU, int kN>
static moe_status launch_gemm(const FfnGemmParams& p, const CUtensorMap& ar, const CUtensorMap& br,
                              const CUtensorMap& as, const CUtensorMap& bs, cudaStream_t stream) {
  constexpr size_t smem = TileCfg<kN>::kSmemBytes + sizeof(FfnSmemCtl) + 1024;
  static_assert(smem <= 232448, "ring + control block exceed the 227 KB a CTA may use");
  static PerDeviceOnce attr_set;
  if (!ensure_dynamic_smem(ffn_gemm_kernel<kSwiGLU, kN>, smem, attr_set)) return MOE_ERR_CUDA;
  return launch_dependent(ffn_gemm_kernel<kSwiGLU, kN>, dim3((unsigned)num_sms()), dim3(kFfnThreads), smem, stream, 1, p,
                          ar, br, as, bs) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

template <bool kSwiGLU>
static moe_status launch_gemm_pair(const FfnGemmParams& p, const CUtensorMap& ar, const CUtensorMap& br,
                                   const CUtensorMap& as, const CUtensorMap& bs, cudaStream_t stream) {
  constexpr size_t smem = (size_t)kPairStages * kPairStageBytes + sizeof(FfnSmemCtl) + 1024;
  static_assert(smem <= 232448, "ring + control block exceed the 227 KB a CTA may use");
  static PerDeviceOnce attr_set;
  if (!ensure_dynamic_smem(ffn_gemm_pair_kernel<kSwiGLU>, smem, attr_set)) return MOE_ERR_CUDA;
  const unsigned grid = (unsigned)(num_sms() & ~1);
  return launch_dependent_cluster(ffn_gemm_pair_kernel<kSwiGLU>, dim3(grid), dim3(kFfnThreads), smem, stream,
                                  dim3(2, 1, 1), p, ar, br, as, bs) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

// CTA pairs or single CTAs.  Measured on B200: pairs win (7 % of the layer) where the routed experts
// receive between 128 and 256 rows on average -- one 256-row pair tile then covers an expert that
// needs two single-CTA tiles, the second mostly padding; they lose at decode sizes (the HBM-bound
// stream runs with half as many weight bytes per stage) and on very large experts under the
// power cap.  ALLOCMOE_PAIR = 0 / 1 forces the choice.
static bool use_pairs(const moe_shape* s, int64_t routed_rows) {
  static int forced = -2;
  if (forced == -2) {
    forced = -1;
    const char* e = getenv("ALLOCMOE_PAIR");
    if (e != nullptr) forced = atoi(e) != 0 ? 1 : 0;
  }
  if (forced >= 0) return forced == 1;
  return routed_rows > 128ll * s->N && routed_rows <= 256ll * s->N;
}

// Weight rows per tile.  256 everywhere: the 128-row variant (twice as many, half as long tiles, 6
// stages) was measured slower on every workload -- each tile re-reads its 16 KB token stage from
// L2 twice as often -- and is kept only behind the knob.
static int pick_tile_n(const moe_shape*, int64_t, bool) {
  static int forced = -1;
  if (forced < 0) {
    forced = 0;
    const char* e = getenv("ALLOCMOE_TILE_N");   // tuning knob: 128 or 256
    if (e != nullptr && (atoi(e) == 128 || atoi(e) == 256)) forced = atoi(e);
  }
  return forced ? forced : 256;
}

// Ints of row-block counters a call needs: one per 128-row block of every group at most.
size_t ffn_done_ints(const moe_shape* s, int64_t budget) {
  return (size_t)(budget / kBM + s->N + (s->S > 0 ? s->T / kBM + 1 : 0) + 4);
}

// Fetching A rows four per TMA instruction costs the producer one instruction per four rows and
// stage where a box load costs one per stage: measured, it pays while an expert's run is short (the
// weight stream leaves the TMA unit idle and most of a 128-row box would be padding) and loses
// badly on full tiles (prefill step 0.46 -> 0.72 ms).  Used up to ALLOCMOE_GATHER (default 32) rows
// per routed expert on average; 0 = never.
bool ffn_gathers(const moe_shape* s, int64_t budget) {
  static int limit = -1;
  if (limit < 0) {
    limit = 32;
    const char* e = getenv("ALLOCMOE_GATHER");
    if (e != nullptr && atoi(e) >= 0) limit = atoi(e);
  }
  return budget > 0 && budget <= (int64_t)limit * s->N;
}

// Routed and/or shared experts in one pair of launches (FfnArgs in ffn.h).
//   routed part present iff budget > 0 && a_routed != nullptr; shared part iff S > 0 && x_shared != nullptr.
//   gather_idx != nullptr: a_routed is x [T, H] itself and routed row m is x[gather_idx[m]] (perm_token);
//   callers pass it only where ffn_gathers() holds.
//   done_is_clear: an earlier kernel of the stream has zeroed `done` (else a memset is enqueued here).
moe_status launch_ffn(const FfnArgs& a) {
  const moe_shape* s = a.s;
  const int64_t budget = a.budget;
  const bool routed = (budget > 0 && a.a_routed != nullptr);
  const bool shared = (s->S > 0 && a.x_shared != nullptr);
  if (!routed && !shared) return MOE_OK;
  const int64_t expected = !routed ? 0 : (a.budget_hint > 0 && a.budget_hint < budget ? a.budget_hint : budget);
  const uint64_t H = s->H, I = s->I;
  CUtensorMap a1r, b1r, a1s, b1s, a2r, b2r, a2s, b2s;
  const bool pairs = use_pairs(s, expected);
  const int tile_n = pairs ? 256 : pick_tile_n(s, expected, shared);
  const uint32_t kUmmaN = (uint32_t)tile_n;
  const uint32_t b2_box = pairs ? kUmmaN / 2 : kUmmaN;   // a pair's CTA loads half of the B tile
  const bool by_rows = routed && (a.gather_idx != nullptr || ffn_gathers(s, expected));
  bool ok = true;
  if (routed) {
    if (a.gather_idx != nullptr) ok &= make_tmap(&a1r, a.a_routed, H, (uint64_t)s->T, 0, H, 0, 1);
    else ok &= make_tmap(&a1r, a.a_routed, H, (uint64_t)budget, 0, H, 0, by_rows ? 1 : kBM);
    ok &= make_tmap(&b1r, a.W13, H, 2 * I, (uint64_t)s->N, H, 2 * I * H, kUmmaN / 2);
    ok &= make_tmap(&a2r, a.h, I, (uint64_t)budget, 0, I, 0, by_rows ? 1 : kBM);
    ok &= make_tmap(&b2r, a.W2, I, H, (uint64_t)s->N, I, H * I, b2_box);
  }
  if (shared) {
    const uint64_t S = s->S;
    ok &= make_tmap(&a1s, a.x_shared, H, (uint64_t)s->T, 0, H, 0, kBM);
    ok &= make_tmap(&b1s, a.Wsh13, H, 2 * I, S, H, 2 * I * H, kUmmaN / 2);
    ok &= make_tmap(&a2s, a.h_sh, S * I, (uint64_t)s->T, 0, S * I, 0, kBM);
    ok &= make_tmap(&b2s, a.Wsh2, I, H, S, I, H * I, b2_box);
  }
  if (!ok) return MOE_ERR_CUDA;
  if (!routed) { a1r = a1s; b1r = b1s; a2r = a2s; b2r = b2s; }
  if (!shared) { a1s = a1r; b1s = b1r; a2s = a2r; b2s = b2r; }

  FfnGemmParams p{};
  p.expert_offsets = a.expert_offsets;
  p.n_experts = routed ? s->N : 0;
  p.routed_rows = routed ? (int)budget : 0;
  p.shared_rows = shared ? s->T : 0;
  p.shared_sub = s->S;
  p.dev_status = a.dev_status;
  p.wait_limit_clk = a.wait_limit_clk > 0 ? a.wait_limit_clk : kWaitLimitClk;
  // row-block completion counters for the GEMM-1 -> GEMM-2 hand-over
  p.done = a.done;
  if (a.done != nullptr) {
    const int nb1 = (int)((s->I + kUmmaN / 2 - 1) / (kUmmaN / 2));      // GEMM-1 column blocks per (sub-)expert
    const int per_tile = 4 * (pairs ? 2 : 1);                           // every epilogue warp counts once
    p.dep_need_routed = nb1 * per_tile;
    p.dep_need_shared = nb1 * s->S * per_tile;
    p.done_capacity = (int)ffn_done_ints(s, routed ? budget : 0);
    if (!a.done_is_clear &&
        cudaMemsetAsync(a.done, 0, ffn_done_ints(s, routed ? budget : 0) * sizeof(int32_t), a.stream) != cudaSuccess)
      return MOE_ERR_CUDA;
  }
  // GEMM-1
  p.gather_idx = routed ? a.gather_idx : nullptr;
  p.gather_rows = by_rows ? (int)budget : 0;
  p.gather_src_rows = (int)s->T;
  p.n_per_sub = s->I;
  p.k_per_sub = s->H;
  p.up_row_offset = s->I;
  p.out_routed = reinterpret_cast<__nv_bfloat16*>(a.h);
  p.out_shared = reinterpret_cast<__nv_bfloat16*>(a.h_sh);
  p.ld_out_routed = s->I;
  p.ld_out_shared = (long long)s->S * s->I;
  if (!a.gemm2_only) {
    moe_status st = pairs           ? launch_gemm_pair<true>(p, a1r, b1r, a1s, b1s, a.stream)
                    : tile_n == 128 ? launch_gemm<true, 128>(p, a1r, b1r, a1s, b1s, a.stream)
                                    : launch_gemm<true, 256>(p, a1r, b1r, a1s, b1s, a.stream);
    if (st != MOE_OK) return st;
  }
  if (a.between != nullptr) cudaEventRecord(a.between, a.stream);
  // GEMM-2
  p.gather_idx = nullptr;
  p.gather_rows = by_rows ? (int)budget : 0;
  p.gather_src_rows = (int)budget;
  p.n_per_sub = s->H;
  p.k_per_sub = s->I;
  p.up_row_offset = 0;
  p.out_routed = reinterpret_cast<__nv_bfloat16*>(a.y_perm);
  p.out_shared = reinterpret_cast<__nv_bfloat16*>(a.y_shared);
  p.ld_out_routed = s->H;
  p.ld_out_shared = s->H;
  if (pairs) return launch_gemm_pair<false>(p, a2r, b2r, a2s, b2s, a.stream);
  return tile_n == 128 ? launch_gemm<false, 128>(p, a2r, b2r, a2s, b2s, a.stream)
                       : launch_gemm<false, 256>(p, a2r, b2r, a2s, b2s, a.stream);
}
