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

}  // namespace mpode
