// Host-side argument checks shared by every entry point (see moe_shape in allocmoe.h).
#pragma once

#include <stdint.h>

#include "allocmoe.h"

namespace allocmoe {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline bool shape_ok(const moe_shape* s) {
  if (s == nullptr) return false;
  if (s->flags != 0) return false;
  if (s->T < 1 || s->H < 64 || s->I < 64 || s->N < 8 || s->S < 0) return false;
  if (s->H % 64 != 0 || s->I % 64 != 0 || s->N % 4 != 0 || s->N > 128) return false;
  if (s->K_orig < 1 || s->K_orig > 16 || s->K_orig > s->N) return false;
  if (s->K_base < 0 || s->K_base > s->K_orig) return false;
  if ((long long)s->T * s->K_orig >= (1ll << 31)) return false;
  return true;
}

}  // namespace allocmoe
