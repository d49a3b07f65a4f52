// alloc_l_solve: Alloc-L's layer-level allocation (Sec. 3.2, Eq. 3-6), host side.
//
// Choose K_i in 1..K_orig for each of L layers so that sum_i S[i, K_i] is smallest under
// sum_i K_i <= B: a grouped knapsack, one group per layer, solved exactly by
//     DP[i, b] = min over 1 <= k <= min(K_orig, b) of DP[i-1, b-k] + S[i, k],
//     DP[-1, 0] = 0, DP[-1, b > 0] = +inf,
// the answer being the best DP[L-1, b] over b <= B, recovered by backtracking: O(L * B * K_orig)
// time, O(L * B) bytes for the choices.  It runs once, off line, before serving; nothing here
// touches the GPU.  Ties go to the smaller k, then to the smaller total b, so the result is unique.
#include <cstdint>
#include <limits>
#include <new>
#include <vector>

#include "allocmoe.h"

extern "C" moe_status alloc_l_solve(const double* S, int32_t L, int32_t K_orig, int64_t B, int32_t* K_out,
                                    double* cost_out) {
  if (S == nullptr || K_out == nullptr || L < 1 || K_orig < 1 || K_orig > 255) return MOE_ERR_ARG;
  if (B < (int64_t)L) return MOE_ERR_BUDGET;                 // Eq. 5 cannot hold with one expert per layer
  const int64_t cap = (int64_t)L * K_orig;                   // more budget than this is never used
  const int64_t Bc = B < cap ? B : cap;
  if ((Bc + 1) * (int64_t)L > (int64_t)1 << 31) return MOE_ERR_ARG;
  const double inf = std::numeric_limits<double>::infinity();
  try {
    std::vector<double> prev((size_t)Bc + 1, inf), cur((size_t)Bc + 1, inf);
    std::vector<uint8_t> choice((size_t)L * (size_t)(Bc + 1), 0);
    prev[0] = 0.0;
    for (int32_t i = 0; i < L; ++i) {
      const double* Si = S + (size_t)i * K_orig;
      uint8_t* ch = choice.data() + (size_t)i * (size_t)(Bc + 1);
      for (int64_t b = 0; b <= Bc; ++b) {
        double best = inf;
        uint8_t arg = 0;
        const int64_t kmax = b < K_orig ? b : K_orig;
        for (int64_t k = 1; k <= kmax; ++k) {
          const double v = prev[(size_t)(b - k)] + Si[k - 1];
          if (v < best) { best = v; arg = (uint8_t)k; }      // strict: the smaller k keeps a tie
        }
        cur[(size_t)b] = best;
        ch[b] = arg;
      }
      prev.swap(cur);
    }
    int64_t bb = -1;
    double best = inf;
    for (int64_t b = 0; b <= Bc; ++b)
      if (prev[(size_t)b] < best) { best = prev[(size_t)b]; bb = b; }
    if (bb < 0) return MOE_ERR_NONFINITE;                    // every total is +inf or NaN: S is not finite
    for (int32_t i = L - 1; i >= 0; --i) {
      const int32_t k = choice[(size_t)i * (size_t)(Bc + 1) + (size_t)bb];
      if (k < 1) return MOE_ERR_NONFINITE;
      K_out[i] = k;
      bb -= k;
    }
    if (cost_out != nullptr) *cost_out = best;
  } catch (const std::bad_alloc&) {
    return MOE_ERR_WORKSPACE;
  }
  return MOE_OK;
}
