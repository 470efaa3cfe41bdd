// Kernels of the hypernetwork flow with the exact trace (Sec. 6.1, the two-dimensional experiments): see hyper_cnf.cu.
#pragma once
#include "common.cuh"
#include "rk_fused.h"

namespace mpode {

constexpr int HYPER_MAX_D = 8;

size_t hyper_param_count(int h, int w, int d);       // A1, c1, A2, c2, A3, c3
size_t hyper_stage_floats(int h, int w, int d);      // h1, h2, the w weight sets and the products U_j . W_j of one stage time
size_t hyper_scratch_floats(int w, int d);           // the batch sums of the weight-set cotangents
size_t hyper_step_scratch_floats(int h, int w, int d);   // whole-step product: those sums, the parts of the h2 cotangent, the stage gradients
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

// All stages of one Runge-Kutta step in one launch each way (the samples are independent of each other through a step).
// The hypernetwork is evaluated for every stage time of the solve beforehand: launch_hyper_table fills table[count] (each
// hyper_stage_floats) from the device array taus[count] of rounded stage times.
// Per stage: hyp (hyper_stage_floats, an entry of that table), units A (low [w][B]), k (low [B, d]), kl (low [B]), the stage input y (low [B, d]; stage 0
// reads the step's state instead), psi (low [B, d]), the unit cotangents sb (low [w][B]), the stage cotangent kap / kapl.
struct HyperStagePtrs {
    float* hyp[RK_MAX_STAGES];
    void *A[RK_MAX_STAGES], *k[RK_MAX_STAGES], *kl[RK_MAX_STAGES], *y[RK_MAX_STAGES], *psi[RK_MAX_STAGES], *sb[RK_MAX_STAGES],
        *kap[RK_MAX_STAGES], *kapl[RK_MAX_STAGES];
};
bool hyper_step_shape_ok(int h, int w, int d, int stages);      // the weight sets of all stage times fit shared memory
// Y_j = Q16(ybar + sum_{l<j} (h a_jl) k_l) and k_j = f(tau_j, Y_j) for every stage (Alg. 1, increment)
void launch_hyper_table(mpode_dtype dt, const float* theta, const float* taus, int count, int h, int w, int d, float* table, cudaStream_t st,
                        long long* launches);
void launch_hyper_step_forward(mpode_dtype dt, const RkStepScalars& sc, int stages, int h, int w, int d,
                               const HyperStagePtrs& ptr, const void* ybar, int B, cudaStream_t st, long long* launches);
// kappa_j = Q16(b_j v + sum_{l>j} (h a_lj) psi_l), psi_j and dg = sum_j dtheta_j (added last stage first) from the seed v (low
// [B, d]) and v_l (low [B]).  scratch: hyper_step_scratch_floats; counters: `stages` device words that are zero between calls.
void launch_hyper_step_vjp(mpode_dtype dt, const float* theta, const RkStepScalars& sc, int stages, int h, int w, int d,
                           const HyperStagePtrs& ptr, const void* ybar, const void* v, const void* v_l, float* scratch, float* dg, int B,
                           unsigned* flag, unsigned* counters, cudaStream_t st, long long* launches);

}  // namespace mpode
