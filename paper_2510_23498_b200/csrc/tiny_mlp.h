// Whole-solve kernels for very small dense velocities (state width <= 8, one hidden layer of <= 64 units, batch <= 1024):
// at these sizes the time loop is pure launch latency, so the forward pass of Alg. 1 and the whole backward pass of
// Alg. 2 (recompute, vector-Jacobian products, finiteness test, halving / doubling of the adjoint scale, fp32 updates)
// each run as ONE launch of a single CTA with one thread per sample and the rounded weights in shared memory.
#pragma once
#include "common.cuh"
#include "rk_fused.h"

namespace mpode {

constexpr int TINY_MAX_D = 8;
constexpr int TINY_MAX_H = 64;
constexpr int TINY_MAX_B = 1024;
constexpr int TINY_MAX_P = 640;

struct TinyParams {
    int B, d, h, stages, n_steps;
    int act, time, bias;
    int poly;                           // 1: the scalar velocity f = -(theta_1 t^2 + theta_2 t + theta_3) y of Example 1 (d = 1, 3 parameters,
                                        // every arithmetic operation rounded to the low format) instead of the MLP
    const float* theta;                 // fp32 [p]: W1 [h][d (+1)], b1 [h], W2 [d][h], b2 [d]
    const RkStepScalars* scal;          // device [n_steps]
    void* traj;                         // low [(n_steps + 1)][B][d]
    int round_increment;
    // forward
    const float* y0; float* yT;
    // backward
    const float* dLdyT; float* a; float* g; int accumulate;
    int scaling, k_max, growth_rule, pbits, e0, e0_from_norm;
    int* log_exp; int* log_attempts; int* log_doubled;   // device [n_steps]
    int* status;                        // device [4]: 0 = MPODE status, 1 = first failed step, 2 = retries, 3 = overflow seen
    const float* cot;                   // device fp32 [n_steps][B][d] running-cost cotangents, or null
    float* tprime;                      // device fp32 [n_steps + 1], zero at launch: receives dL/dt; null = not wanted
};

bool tiny_mlp_supported(int B, int d, int h, int n_layers, int p);
void launch_tiny_forward(mpode_dtype dt, const TinyParams& p, cudaStream_t st, long long* launches);
void launch_tiny_backward(mpode_dtype dt, const TinyParams& p, cudaStream_t st, long long* launches);

}  // namespace mpode
