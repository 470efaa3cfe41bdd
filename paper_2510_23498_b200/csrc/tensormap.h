// Host-side construction (and caching) of the TMA tensor maps the tensor-core kernels read their operands through.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace mpode {

// Tensor map of a row-major [rows, cols] 16-bit matrix with row stride ld (elements): box = [box_rows, 64 columns],
// 128-byte swizzle, out-of-range elements read as zero.  Returns false if the driver entry point is unavailable or
// the encode call rejects the shape (the caller then takes the CUDA-core path).
bool get_tensor_map(const void* ptr, long long rows, long long cols, long long ld, int box_rows, mpode_dtype dt,
                    CUtensorMap* out);

// The same for a stack of `slots` such matrices `slot_stride` elements apart: a 3-D map with coordinates
// (column, row, slot) and box [1, box_rows, 64].
bool get_tensor_map_3d(const void* ptr, long long slots, long long rows, long long cols, long long slot_stride,
                       long long ld, int box_rows, mpode_dtype dt, CUtensorMap* out);

// NHWC image tensor [B][H][W][C] (C a multiple of 64 channels of a 16-bit format) seen as a 4-D map with coordinates
// (channel, x, y, image) and box [64 channels][W][box_h rows][1 image]: W * box_h pixels land as consecutive 128-byte
// rows; coordinates outside the image (the zero padding of a convolution) read as zero.
bool get_tensor_map_nhwc(const void* ptr, int B, int H, int W, int C, int box_h, mpode_dtype dt, CUtensorMap* out);

constexpr int kMaxDevices = 64;
int current_device();     // index of the current CUDA device (0 when there is none)
int sm_count();           // SM count of the current device

}  // namespace mpode
