// Shared device helpers of the sm_100a kernels: PTX wrappers (mbarrier, TMA, tcgen05),
// bounded waits, small block-wide primitives.  Nothing here is used by the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "allocmoe.h"
#include "device_once.h"

#define DEV __device__ __forceinline__

namespace allocmoe {

// ------------------------------------------------------------------ status word
DEV void set_dev_status(int32_t* dev_status, moe_status s) {
  if (dev_status != nullptr) atomicOr(dev_status, 1 << (int)s);
}

// Values that index global memory and come from device data (expert_offsets, perm_token) are clamped to their
// valid range before use, so that a list left behind by a routing step that reported an error cannot lead
// outside the caller's buffers.  The checked build (-DALLOCMOE_CHECKED, `build.py --checked`) also reports every
// value that needed clamping as MOE_ERR_ARG in the status word, which turns silent corruption upstream into an
// error the caller sees.
DEV int clamp_index(int v, int lo, int hi, int32_t* dev_status) {
#ifdef ALLOCMOE_CHECKED
  if (v < lo || v > hi) set_dev_status(dev_status, MOE_ERR_ARG);
#else
  (void)dev_status;
#endif
  return min(max(v, lo), hi);
}

DEV uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ------------------------------------------------------------------ programmatic dependent launch
// Every kernel of the library is launched so that it may become resident while the previous
// kernel of the stream is still running (launch_dependent below).  A kernel therefore does its
// set-up that touches no global memory, calls pdl_prologue_done(), and only then reads or writes
// global memory: the wait returns once every earlier kernel of the stream has completed and its
// writes are visible.  Launched without the attribute, both instructions do nothing.
DEV void pdl_prologue_done() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may start its own set-up
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Default limit of the bounded waits below, in SM clocks: about 0.5 s at 1.9 GHz.  Kernels take the
// limit as a launch parameter (FfnGemmParams::wait_limit_clk) so that a test can make a wait run out
// within milliseconds; every product launch passes this value.
constexpr long long kWaitLimitClk = 1000ll * 1000ll * 1000ll;
DEV void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
DEV void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ------------------------------------------------------------------ flags between kernels / CTAs
// A tile of h written with ordinary stores by GEMM-1's epilogue is read by GEMM-2's TMA loads
// (the async proxy), possibly while GEMM-1 is still running on other SMs.  Writer: stores,
// __threadfence, barrier among the storing warps, then one thread fence_proxy_async_global +
// flag_add_release.  Reader: flag_load_acquire until the count is reached, fence_proxy_async_global,
// then the TMA loads.
DEV void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
DEV void flag_add_release(int32_t* flag, int v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(flag), "r"(v) : "memory");
}
DEV int flag_load_acquire(const int32_t* flag) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
  return v;
}
// Bounded wait for *flag >= need (same limit and abort protocol as the mbarrier waits).
DEV bool flag_wait_bounded(const int32_t* flag, int need, volatile int* abort_flag, int32_t* dev_status,
                           long long limit_clk) {
  if (flag_load_acquire(flag) >= need) return true;
  long long t0 = 0;
  uint32_t spins = 0;
  while (true) {
    __nanosleep(64);
    if (flag_load_acquire(flag) >= need) return true;
    if ((++spins & 63u) == 0u) {
      if (*abort_flag) return false;
      const long long now = clock64();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > limit_clk) {
        *abort_flag = 1;
        set_dev_status(dev_status, MOE_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

// ------------------------------------------------------------------ mbarrier
DEV void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
DEV void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
DEV void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
DEV bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Every wait in these kernels is bounded.  A wait that exceeds its limit (limit_clk) raises the CTA's
// abort flag and MOE_ERR_TIMEOUT in the caller's status word; every other wait of the CTA
// then returns false at its next poll, the roles leave their loops and the CTA tears down
// normally (drains its own copies, frees TMEM, returns).  Time is the SM's own cycle counter,
// looked at only every 64th poll, so a wait that succeeds quickly never pays for it.
constexpr long long kDrainLimitClk = 40ll * 1000ll * 1000ll;    // teardown waits: about 20 ms

DEV bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* dev_status,
                           long long limit_clk) {
  if (mbar_try_wait(bar, parity)) return true;
  long long t0 = 0;
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 63u) == 0u) {
      if (*abort_flag) return false;
      const long long now = clock64();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > limit_clk) {
        *abort_flag = 1;
        set_dev_status(dev_status, MOE_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

// The same wait for a whole warp whose lanes all need the result: lane 0 polls, with a short
// sleep between polls, and the outcome is broadcast, so that 128 epilogue threads do not all
// poll the same barrier word.
DEV bool mbar_wait_bounded_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* dev_status,
                                long long limit_clk) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) {
    if (!mbar_try_wait(bar, parity)) {
      long long t0 = 0;
      uint32_t spins = 0;
      while (true) {
        __nanosleep(40);
        if (mbar_try_wait(bar, parity)) break;
        if ((++spins & 63u) == 0u) {
          if (*abort_flag) { ok = 0; break; }
          const long long now = clock64();
          if (t0 == 0) {
            t0 = now;
          } else if (now - t0 > limit_clk) {
            *abort_flag = 1;
            set_dev_status(dev_status, MOE_ERR_TIMEOUT);
            ok = 0;
            break;
          }
        }
      }
    }
  }
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// Teardown wait: ignores the abort flag, has its own short limit.
DEV bool mbar_wait_drain(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (clock64() - t0 < kDrainLimitClk) {
    if (mbar_try_wait(bar, parity)) return true;
  }
  return false;
}

DEV void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

// ------------------------------------------------------------------ TMA (no multicast anywhere)
DEV void prefetch_tensormap(const void* tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)tmap) : "memory");
}
DEV void tma_load_2d(void* smem_dst, const void* tmap, uint64_t* bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)tmap), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}
DEV void tma_load_3d(void* smem_dst, const void* tmap, uint64_t* bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)tmap), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

// Four rows of a 2-D tensor picked by row index (the map's box is 64 columns x 1 row): 4 x 128 bytes,
// stored as four consecutive rows of the 128-byte-swizzled tile that smem_dst lies in.
DEV void tma_gather4_2d(void* smem_dst, const void* tmap, uint64_t* bar, int c0, int r0, int r1, int r2, int r3) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)tmap), "r"(smem_u32(bar)), "r"(c0), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
      : "memory");
}

// Orders this thread's earlier generic-proxy accesses to shared memory (ldmatrix reads of a ring slot, made
// visible to it by a barrier) before async-proxy writes it issues afterwards (the TMA load that refills the slot).
DEV void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ------------------------------------------------------------------ tcgen05 / TMEM
DEV void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {   // whole warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(ncols) : "memory");
}
DEV void tmem_relinquish() {                                     // whole warp
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
DEV void tmem_dealloc(uint32_t taddr, uint32_t ncols) {          // whole warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
DEV void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
DEV void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T ; kind::f16 covers bf16 inputs with fp32 accumulation.
DEV void umma_bf16(uint32_t d_tmem, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on `bar` once every MMA this thread issued so far has completed.
DEV void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp gets lane (base_lane + i).
DEV void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
DEV void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile stored as rows of 128 bytes with the
// 128-byte swizzle (what TMA writes with SWIZZLE_128B): 8-row groups are 1024 bytes apart
// (stride byte offset), the leading byte offset is unused for swizzled K-major tiles (1),
// descriptor version 1 (Blackwell), layout type 2 (SWIZZLE_128B).  The tile base must be
// 1024-byte aligned.  Stepping 16 elements along K adds 32 bytes to the start address.
DEV uint64_t umma_desc_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor, kind::f16: fp32 accumulator (bits 4-5 = 1), A and B bf16 (bits 7-9 and
// 10-12 = 1), both K-major (bits 15, 16 = 0), N >> 3 at bit 17, M >> 4 at bit 24.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------ CTA pairs (cta_group::2)
// Two CTAs of a cluster on the two SMs of a TPC issue ONE tcgen05.mma of M = 256: each CTA holds
// 128 rows of A, half of the B tile's rows and its 128 rows of the accumulator.  The pair's even
// CTA (the leader) issues the MMAs and owns the "stage full" barriers; both CTAs load their own
// parts and signal the leader's barrier; commits are multicast to both CTAs' barriers.
DEV uint32_t cluster_addr_of(const void* smem_ptr, uint32_t cta_rank) {   // this variable in CTA cta_rank
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(smem_ptr)), "r"(cta_rank));
  return r;
}
DEV void mbar_expect_tx_cluster(uint32_t bar_cluster_addr, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(bar_cluster_addr), "r"(bytes) : "memory");
}
DEV void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
// Loads into this CTA's shared memory, completion counted on a barrier that may live in the peer.
DEV void tma_load_2d_pair(void* smem_dst, const void* tmap, uint32_t bar_cluster_addr, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)tmap), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
      : "memory");
}
DEV void tma_load_3d_pair(void* smem_dst, const void* tmap, uint32_t bar_cluster_addr, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)tmap), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
DEV void tma_gather4_2d_pair(void* smem_dst, const void* tmap, uint32_t bar_cluster_addr, int c0, int r0, int r1, int r2,
                             int r3) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes.cta_group::2"
      " [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)tmap), "r"(bar_cluster_addr), "r"(c0), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
      : "memory");
}
DEV void tmem_alloc_pair(uint32_t* smem_result, uint32_t ncols) {   // the same warp of both CTAs
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(ncols) : "memory");
}
DEV void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
DEV void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem of both CTAs] (+)= A * B^T, M = 256 over the pair; issued by one thread of the leader.
DEV void umma_bf16_pair(uint32_t d_tmem, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  const uint32_t z = 0u;   // no output lane disabled
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(z)
      : "memory");
}
// Arrives on the barrier at this offset in every CTA of cta_mask once the MMAs issued so far are done.
DEV void umma_commit_pair(uint64_t* bar, uint16_t cta_mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"(cta_mask) : "memory");
}
DEV void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");   // not .aligned: the role warps arrive diverged
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
DEV uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}

// ------------------------------------------------------------------ cp.async (Ampere-style, 16 B)
DEV void cp_async_16(void* smem_dst, const void* gsrc, bool valid) {
  const int sz = valid ? 16 : 0;   // src-size 0: the 16 bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(sz) : "memory");
}
DEV void cp_async_8(void* smem_dst, const void* gsrc, bool valid) {
  const int sz = valid ? 8 : 0;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(sz) : "memory");
}
DEV void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
DEV void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// ------------------------------------------------------------------ misc
DEV float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }
DEV uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Exclusive scan of one int per thread over the block (blockDim.x <= 1024, multiple of 32).
// `warp_sums` is 33 ints of shared memory; returns the exclusive prefix, *total gets the sum.
DEV int block_exclusive_scan(int v, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  int incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  __syncthreads();   // protects warp_sums against a previous use
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = lane < nwarps ? warp_sums[lane] : 0;
    int wi = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int o = __shfl_up_sync(0xffffffffu, wi, d);
      if (lane >= d) wi += o;
    }
    warp_sums[lane] = wi - w;
    if (lane == 31) warp_sums[32] = wi;
  }
  __syncthreads();
  *total = warp_sums[32];
  return warp_sums[warp] + incl - v;
}

}  // namespace allocmoe

// Host side.  Lets `kernel` use `bytes` of dynamic shared memory on the current device; the attribute is
// per device, so `once` remembers the devices it has been set on.
template <typename Kernel>
inline bool ensure_dynamic_smem(Kernel kernel, size_t bytes, allocmoe::PerDeviceOnce& once) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  if (once.done(dev)) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return false;
  once.mark(dev);
  return true;
}

// Host side: launch with the programmatic-stream-serialization attribute (and, when cluster_y > 1,
// a thread-block cluster).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                            cudaStream_t stream, dim3 cluster, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster.x * cluster.y * cluster.z > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster.x;
    attr[n].val.clusterDim.y = cluster.y;
    attr[n].val.clusterDim.z = cluster.z;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = (unsigned)n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    unsigned cluster_y, Args... args) {
  return launch_dependent_cluster(kernel, grid, block, smem, stream, dim3(1, cluster_y, 1), args...);
}
