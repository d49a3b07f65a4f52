// Host-side builder of TMA tensor maps (cuTensorMapEncodeTiled through the runtime's driver entry point),
// shared by the expert GEMMs and the gate.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

// bf16 tensor [d2][d1][d0] (d0 contiguous; d2 == 0: two-dimensional), box {64, box1, 1}, 128-byte swizzle,
// out-of-range elements read as zero.  Strides in elements.  False when the driver refuses the map.
bool make_tmap(CUtensorMap* tm, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_elems,
               uint64_t stride2_elems, uint32_t box1);
