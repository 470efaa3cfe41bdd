// Chooses the kernel for one contraction: the tensor-core path where the shape and format allow it, otherwise
// the general CUDA-core kernel.  Optionally brackets each launch with CUDA events (measurement hook).
#include "common.cuh"
#include "conv_tc.h"
#include "gemm_tc.h"
#include "profiler.h"

namespace mpode {

thread_local Profiler* tl_profiler = nullptr;
thread_local PathCounters* tl_counters = nullptr;

// returns which kernel ran: 0 the CUDA-core kernel, 1 the general tensor-core kernel, 2 the 64-channel convolution kernel
int launch_contraction(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* L) {
    Profiler* pr = tl_profiler;
    int klass = g.epi == EPI_FWD ? 0 : (g.epi == EPI_WGRAD ? 2 : 1);
    if (pr && pr->enabled) pr->begin(klass, 2.0 * g.M * g.N * (double)g.K, st);
    bool done = false, halo = false;
    if (g.epi == EPI_WGRAD) done = wgrad_tc_eligible(dt, g) && launch_wgrad_tc(dt, g, st, L);
    else {
        done = halo = conv_halo_eligible(dt, g) && launch_conv_halo(dt, g, st, L);
        if (!done) done = tc_eligible(dt, g) && launch_gemm_tc(dt, g, st, L);
    }
    if (tl_counters) ++(done ? tl_counters->tc : tl_counters->simt);
    if (!done) {
        GemmArgs s = g;
        if (s.epi == EPI_WGRAD && s.split_k <= 1) s.partial = nullptr;
        launch_gemm_simt(dt, s, st, L);
    }
    if (pr && pr->enabled) pr->end(st);
    return halo ? 2 : (done ? 1 : 0);
}

}  // namespace mpode
