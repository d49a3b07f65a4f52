// Host interface of the expert-GEMM launcher (ffn.cu), used by the C-ABI entry points (api.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "allocmoe.h"

// One call = expert GEMM-1 (+ SwiGLU) and GEMM-2 for the routed experts and / or the shared experts.
struct FfnArgs {
  const moe_shape* s = nullptr;
  // routed experts (absent when a_routed == nullptr or budget == 0)
  const uint16_t* a_routed = nullptr;      // x_perm [budget, H]; or x [T, H] when gather_idx is given
  const int32_t* gather_idx = nullptr;     // perm_token [budget]: routed row m is x[gather_idx[m]]
  const int32_t* expert_offsets = nullptr; // device [N+1]
  int64_t budget = 0;                      // rows of the routed matrices: an upper bound of expert_offsets[N]
  int64_t budget_hint = 0;                 // expected list length when it is below `budget`; only picks the tile variant
  const uint16_t* W13 = nullptr;
  const uint16_t* W2 = nullptr;
  uint16_t* h = nullptr;                   // [budget, I] scratch
  uint16_t* y_perm = nullptr;              // [budget, H]
  // shared experts (absent when x_shared == nullptr or S == 0)
  const uint16_t* x_shared = nullptr;
  const uint16_t* Wsh13 = nullptr;
  const uint16_t* Wsh2 = nullptr;
  uint16_t* h_sh = nullptr;                // [T, S*I] scratch
  uint16_t* y_shared = nullptr;            // [T, H]
  int32_t* dev_status = nullptr;
  int32_t* done = nullptr;                 // row-block counters of the GEMM-1 -> GEMM-2 hand-over (ffn_done_ints)
  bool done_is_clear = false;              // an earlier kernel of the stream has zeroed them
  long long wait_limit_clk = 0;            // limit of the kernels' bounded waits in SM clocks; 0 = the default
  bool gemm2_only = false;                 // self-test only: GEMM-1 is not launched, so GEMM-2's waits run out
  cudaStream_t stream = nullptr;
  cudaEvent_t between = nullptr;           // recorded between the two GEMMs when set
};

moe_status launch_ffn(const FfnArgs& args);
size_t ffn_done_ints(const moe_shape* s, int64_t budget);
bool ffn_gathers(const moe_shape* s, int64_t budget);
