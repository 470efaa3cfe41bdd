// Kernels of the hypernetwork flow with the exact trace (Sec. 6.1, the two-dimensional experiments): see hyper_cnf.cu.
#pragma once
#include "common.cuh"

namespace mpode {

constexpr int HYPER_MAX_D = 8;

size_t hyper_param_count(int h, int w, int d);       // A1, c1, A2, c2, A3, c3
size_t hyper_stage_floats(int h, int w, int d);      // h1, h2, the w weight sets and the products U_j . W_j of one stage time
size_t hyper_scratch_floats(int w, int d);           // the batch sums of the weight-set cotangents
bool hyper_shape_ok(int h, int w, int d);            // the weight sets of one stage time fit the kernels' shared memory

// k = [v; -tr] for one stage: `hyp` (hyper_stage_floats) receives the hypernetwork's rounded layers, A (low [w][B]) the units
void launch_hyper_forward(mpode_dtype dt, const float* theta, float tau16, int h, int w, int d, float* hyp, const void* Y, void* A, void* k,
                          void* k_l, int B, cudaStream_t st, long long* launches);
// psi and dg = (beta != 0 ? beta * dg : 0) + dtheta of one stage from its cotangent (kappa low [B, d], kappa_l low [B]).
// Sb: low [w][B] scratch for the unit cotangents; sums: hyper_scratch_floats; counter: a device word that is zero between calls;
// non-finite low-format values raise *flag (flag may be null)
void launch_hyper_vjp(mpode_dtype dt, const float* theta, float tau16, int h, int w, int d, const float* hyp, const void* Y, const void* A,
                      void* Sb, const void* kappa, const void* kappa_l, void* psi, float* sums, float* dg, float beta, int B, unsigned* flag,
                      unsigned* counter, cudaStream_t st, long long* launches);

}  // namespace mpode
