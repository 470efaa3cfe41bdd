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

}  // namespace mpode
