// Kernels of the hypernetwork flow with the exact trace (Sec. 6.1, the two-dimensional experiments): see hyper_cnf.cu.
#pragma once
#include "common.cuh"

namespace mpode {

constexpr int HYPER_MAX_D = 8;

size_t hyper_param_count(int h, int w, int d);       // A1, c1, A2, c2, A3, c3
size_t hyper_stage_floats(int h, int w, int d);      // h1, h2, the w weight sets and the products U_j . W_j of one stage time
int hyper_blocks(int B);                             // blocks of the per-sample kernels = partial sums of the weight-set cotangents

// k = [v; -tr] for one stage: `hyp` (hyper_stage_floats) receives the hypernetwork's rounded layers, A (low [w][B]) the units
void launch_hyper_forward(mpode_dtype dt, const float* theta, float tau16, int h, int w, int d, float* hyp, const void* Y, void* A, void* k,
                          void* k_l, int B, cudaStream_t st, long long* launches);
// psi and dg = (beta != 0 ? beta * dg : 0) + dtheta of one stage from its cotangent (kappa low [B, d], kappa_l low [B]);
// part: hyper_blocks(B) * w * (2 d + 2) floats of scratch; non-finite low-format values raise *flag (flag may be null)
void launch_hyper_vjp(mpode_dtype dt, const float* theta, float tau16, int h, int w, int d, const float* hyp, const void* Y, const void* A,
                      const void* kappa, const void* kappa_l, void* psi, float* part, float* dg, float beta, int B, unsigned* flag,
                      cudaStream_t st, long long* launches);

}  // namespace mpode
