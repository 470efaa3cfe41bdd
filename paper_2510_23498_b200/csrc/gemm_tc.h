// Tensor-core (tcgen05 / TMEM / TMA) path of the velocity-layer contractions.
#pragma once
#include "common.cuh"

namespace mpode {

// true when the contraction can run on the tensor-core kernels (16-bit formats, K-major operands, aligned shapes)
bool tc_eligible(mpode_dtype dt, const GemmArgs& g);
// launches it; returns false (nothing launched) if the tensor maps could not be built
bool launch_gemm_tc(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* launches);

// Weight-gradient contractions (reduction over the batch rows): eligibility, launch (kernel + fixed-order reduction
// of the slice partial sums into `out` with beta), and the fp32 scratch `g.partial` must provide.
bool wgrad_tc_eligible(mpode_dtype dt, const GemmArgs& g);
bool launch_wgrad_tc(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* launches);
size_t wgrad_tc_scratch_bytes(int M, int N, int K);

// 3x3 convolution weight gradient dW[cout][tap][cin] = sum over pixels of dZ[p][cout] * X[p + tap offset][cin] for an NHWC
// image with C a multiple of 64 channels: computed transposed ((tap, cin) rows, cout columns) over slices of the pixels, then summed
// in a fixed order into out[(cout * 9 + tap) * ct + cin] (ct = channels per tap of the destination layout).
bool conv_wgrad_tc_eligible(mpode_dtype dt, int B, int H, int W, int C, const void* dz, const void* x, const float* partial,
                            size_t partial_bytes, const unsigned* err);
size_t conv_wgrad_tc_scratch_bytes(int B, int H, int W, int C);
// out = beta * out + sign * dW
bool launch_conv_wgrad_tc(mpode_dtype dt, const void* dz, const void* x, int B, int H, int W, int C, int ct, float* out, float beta,
                          float* partial, unsigned* err, cudaStream_t st, long long* launches, float sign = 1.f);

}  // namespace mpode
