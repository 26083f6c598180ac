// Host-side helpers shared by the tensor-core kernels' launchers: TMA tensor maps of the operands (encoded once per
// buffer and shape, then found again), the SM count of the current device, and the optional event pairs around
// kernel launches.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace dsmoe {

constexpr int kTileK = 64;     // reduction elements per operand tile: 128 bytes of bf16, the swizzle span

// Tensor maps of one packed weight tensor [E, n, k] with boxes of 16, 32, 64, 128 and 256 rows: a tile of
// any width (a multiple of 16 rows) is fetched with at most five copies, largest first.
struct BMaps {
    CUtensorMap m[5];
};

// ... and, for the small-T up-projection whose tile widths are arbitrary multiples of 16, one map per height
// 16, 32, ..., 256, so that a tile (or each of its two parts) is a single copy.
struct BMaps16 {
    CUtensorMap m[16];
};


typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_fn();

int sm_count();     // of the current device (148 when there is none: host-only sizing)

// bf16 [rows, cols] row-major, box {64 cols, box_rows}, 128-byte swizzle
dsmoe_status cached_map_2d(const CUtensorMap** out, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows);
// packed weights [E][k / 64][n][64]
dsmoe_status cached_bmaps(const BMaps** out, const void* ptr, uint64_t E, uint64_t n, uint64_t k);
dsmoe_status cached_bmaps16(const BMaps16** out, const void* ptr, uint64_t E, uint64_t n, uint64_t k);
// weights in their natural layout [E][n][k], k contiguous
dsmoe_status cached_bmaps_plain(const BMaps** out, const void* ptr, uint64_t E, uint64_t n, uint64_t k);

// Event pair around a launch when the timing ring is on and has room: *slot = its index, or -1.
dsmoe_status timing_begin(cudaStream_t s, int* slot);
dsmoe_status timing_end(cudaStream_t s, int slot);

}  // namespace dsmoe
