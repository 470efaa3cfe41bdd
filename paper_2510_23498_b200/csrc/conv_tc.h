// 3x3 convolutions with 64 channels in and out on the tensor cores with resident weights and one halo block per horizontal
// stencil offset (see conv_tc.cu): forward (position-class bias, activation, rounding) and input gradient (activation
// derivative from the stored layer output, rounding, overflow flag).
#pragma once
#include "common.cuh"

namespace mpode {

// true when the contraction is such a convolution (GemmArgs in the implicit-convolution form, conv_on = 1)
bool conv_halo_eligible(mpode_dtype dt, const GemmArgs& g);
// launches it; returns false (nothing launched) if the tensor maps could not be built
bool launch_conv_halo(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* launches);

// Weight gradient of such a convolution, dW[cout][tap][cin] = sum over pixels of dZ[p][cout] * X[p + tap offset][cin], from one
// image block and three shifted dZ blocks per 64 pixels (see conv_tc.cu): slices of the pixels, then a fixed-order sum into
// out[(cout * 9 + tap) * ct + cin] = beta * out + sign * dW.  `partial`: fp32 scratch of conv_wgrad_halo_scratch_bytes.
bool conv_wgrad_halo_eligible(mpode_dtype dt, int B, int H, int W, int C, const void* dz, const void* x, const float* partial,
                              size_t partial_bytes, const unsigned* err);
size_t conv_wgrad_halo_scratch_bytes(int B, int H, int W);
// `indicator`: the position-class table of one image (launch_conv_class_indicator); `class_part`: scratch of
// (conv_wgrad_halo_slices + 1) * 9 * 64 floats for the per-slice sums of dZ per position class and their total; `counter`: a device
// word that is zero between calls (the reduction's last-block election).  From the class sums the same reduction writes
// bias_out[cout] = beta * bias_out + sign * sum dZ and, when ct > 64, the gradient of the appended time channel's weights
// (out[(cout * 9 + tap) * ct + ct - 1], tau times the sum over the pixels where the tap is inside the image).
int conv_wgrad_halo_slices(int B, int H, int W);
bool launch_conv_wgrad_halo(mpode_dtype dt, const void* dz, const void* x, const void* indicator, int B, int H, int W, int ct, float* out,
                            float* bias_out, float tau, float beta, float* partial, float* class_part, unsigned* counter, unsigned* err,
                            cudaStream_t st, long long* launches, float sign = 1.f);

}  // namespace mpode
