// Host-side construction of the TMA tensor maps the tcgen05 kernels use.
#pragma once

#include <cuda.h>
#include <stdint.h>

namespace ssn {

// Row-major bf16 matrix [rows x cols], leading dimension ld, fetched in boxes of box_rows x 64
// columns into the 128-byte swizzled layout.  False when no map can be made (no driver entry
// point, unaligned base or pitch, too many rows).
bool make_sw128_map(CUtensorMap *map, const void *base, int64_t rows, int64_t cols, int64_t ld,
                    int box_rows);

// Row-major bf16 tensor [n2][n1][cols] (row pitch ld, slab pitch ld2, in elements), fetched in
// boxes of 64 columns x box1 x box2 into the 128-byte swizzled layout.
bool make_sw128_map3(CUtensorMap *map, const void *base, int64_t cols, int64_t n1, int64_t n2, int64_t ld,
                     int64_t ld2, int box1, int box2);

}  // namespace ssn
