// Host-side construction of TMA tensor maps (driver entry point fetched through the runtime, so
// the library does not link libcuda).
#pragma once

#include <cuda.h>
#include "common.cuh"

namespace focus {

// 4-D bf16 tensor map, innermost dimension first; strides in bytes for dimensions 1..3; the box is
// box0 x box1 x 1 x 1 elements, 128-byte swizzle, out-of-bounds elements read as zero.
int make_tmap_bf16_4d(CUtensorMap* out, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t d3,
                      uint64_t s1_bytes, uint64_t s2_bytes, uint64_t s3_bytes, uint32_t box0, uint32_t box1);

// tensor map of a [batch, H, n, D] bf16 focus_tensor with a 64 x rows (columns x rows) box
int make_tmap_qkv(CUtensorMap* out, const focus_tensor& t, int batch, int H, int n, int D, int rows = 128);

}  // namespace focus
