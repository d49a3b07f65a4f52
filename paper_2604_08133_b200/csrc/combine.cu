// moe_combine: Eq. 2 over the kept pairs.
//   out[t] = sum_{j < n_sel[t]} topk_score[t,j] * y_perm[pair_pos[t,j]]  (+ y_shared[t]) (+ x[t])
// fp32 FMAs in ascending j, one rounding to bf16.  One CTA per token, 16 bytes (8 bf16) per
// thread per step: every global access is a coalesced 128-bit load or store.
#include "common.cuh"

namespace allocmoe {

DEV void fma8(float (&acc)[8], const uint4& v, float w) {
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    acc[2 * q] = fmaf(w, bf16_bits_to_float(u[q] & 0xFFFFu), acc[2 * q]);
    acc[2 * q + 1] = fmaf(w, bf16_bits_to_float(u[q] >> 16), acc[2 * q + 1]);
  }
}

__global__ void __launch_bounds__(256, 5)
combine_kernel(const uint4* __restrict__ y_perm, const int32_t* __restrict__ pair_pos,
               const float* __restrict__ topk_score, const int32_t* __restrict__ n_sel,
               const uint4* __restrict__ y_shared, const uint4* __restrict__ x_res, int K_orig, int row_vec,
               long long budget_rows, uint4* __restrict__ out) {
  __shared__ int s_pos[16];
  __shared__ float s_w[16];
  __shared__ int s_n;
  const int t = blockIdx.x;
  pdl_prologue_done();
  if (threadIdx.x < 16) {
    // the count, the position and the weight of column j do not depend on each other: one round trip
    const int j = threadIdx.x;
    const int n = min(max(__ldg(n_sel + t), 0), K_orig);
    int pos = -1;
    float w = 0.f;
    if (j < K_orig) {
      pos = __ldg(pair_pos + (long long)t * K_orig + j);
      w = __ldg(topk_score + (long long)t * K_orig + j);
    }
    if (j >= n || pos < 0 || pos >= budget_rows) { pos = -1; w = 0.f; }
    if (j == 0) s_n = n;
    s_pos[j] = pos;
    s_w[j] = w;
  }
  __syncthreads();
  const int n = s_n;
  for (int c = threadIdx.x; c < row_vec; c += blockDim.x) {
    // the token's own rows first, then the expert rows four loads at a time, FMAs in ascending j
    uint4 vs = make_uint4(0, 0, 0, 0), vr = make_uint4(0, 0, 0, 0);
    if (y_shared != nullptr) vs = __ldg(y_shared + (long long)t * row_vec + c);
    if (x_res != nullptr) vr = __ldg(x_res + (long long)t * row_vec + c);
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int jb = 0; jb < n; jb += 4) {
      uint4 v[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int pos = s_pos[jb + q < 16 ? jb + q : 15];
        v[q] = make_uint4(0, 0, 0, 0);
        if (jb + q < n && pos >= 0) v[q] = __ldg(y_perm + (long long)pos * row_vec + c);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (jb + q < n) fma8(acc, v[q], s_w[jb + q < 16 ? jb + q : 15]);
    }
    if (y_shared != nullptr) fma8(acc, vs, 1.f);
    if (x_res != nullptr) fma8(acc, vr, 1.f);
    uint4 o;
    o.x = pack_bf16x2(acc[0], acc[1]);
    o.y = pack_bf16x2(acc[2], acc[3]);
    o.z = pack_bf16x2(acc[4], acc[5]);
    o.w = pack_bf16x2(acc[6], acc[7]);
    out[(long long)t * row_vec + c] = o;
  }
}

// Pre-norm of the layer stack: out[t] = x[t] * rsqrt(mean(x[t]^2) + eps).  One CTA per token; the
// sum of squares is reduced in a fixed order (lanes by shuffle, warps in index order).
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const uint4* __restrict__ x, int row_vec, int H, uint4* __restrict__ out) {
  __shared__ float warp_part[8];
  __shared__ float s_scale;
  const int t = blockIdx.x;
  pdl_prologue_done();
  float ss = 0.f;
  for (int c = threadIdx.x; c < row_vec; c += blockDim.x) {
    const uint4 v = __ldg(x + (long long)t * row_vec + c);
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float a = bf16_bits_to_float(u[q] & 0xFFFFu), b = bf16_bits_to_float(u[q] >> 16);
      ss = fmaf(a, a, ss);
      ss = fmaf(b, b, ss);
    }
  }
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int w = 0; w < 8; ++w) tot += warp_part[w];
    s_scale = rsqrtf(tot / (float)H + 1e-6f);
  }
  __syncthreads();
  const float sc = s_scale;
  for (int c = threadIdx.x; c < row_vec; c += blockDim.x) {
    const uint4 v = __ldg(x + (long long)t * row_vec + c);
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
      o[q] = pack_bf16x2(bf16_bits_to_float(u[q] & 0xFFFFu) * sc, bf16_bits_to_float(u[q] >> 16) * sc);
    out[(long long)t * row_vec + c] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

}  // namespace allocmoe

using namespace allocmoe;

moe_status launch_rmsnorm(const moe_shape* s, const uint16_t* x, uint16_t* out, cudaStream_t stream) {
  return launch_dependent(rmsnorm_kernel, dim3((unsigned)s->T), dim3(256), 0, stream, 1, reinterpret_cast<const uint4*>(x),
                          s->H / 8, s->H, reinterpret_cast<uint4*>(out)) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

moe_status launch_moe_combine(const moe_shape* s, const uint16_t* y_perm, const int32_t* pair_pos,
                              const float* topk_score, const int32_t* n_sel, const uint16_t* y_shared,
                              const uint16_t* x_res, long long budget_rows, uint16_t* out, cudaStream_t stream) {
  return launch_dependent(combine_kernel, dim3((unsigned)s->T), dim3(256), 0, stream, 1,
                          reinterpret_cast<const uint4*>(y_perm), pair_pos, topk_score, n_sel,
                          reinterpret_cast<const uint4*>(y_shared), reinterpret_cast<const uint4*>(x_res), (int)s->K_orig,
                          s->H / 8, budget_rows, reinterpret_cast<uint4*>(out)) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}
