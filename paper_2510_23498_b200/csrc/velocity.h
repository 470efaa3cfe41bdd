// Host-side description of a built-in velocity network: where its buffers live in the caller's workspace and
// which kernels evaluate it (forward, the increment of Alg. 1) and its vector-Jacobian product (Eq. (vjp)).
#pragma once
#include <stddef.h>

#include <vector>

#include "common.cuh"
#include "rk_fused.h"

namespace mpode {

// Scale policy and outputs of a whole backward pass done in one launch (very small velocities).
struct WholeBackward {
    const float* theta = nullptr; const float* dLdyT = nullptr; float* a = nullptr; float* g = nullptr;
    int accumulate = 0, scaling = 0, k_max = 10, growth_rule = 0, pbits = 8, e0 = 0, e0_from_norm = 0;
    // host results
    int status = 0, first_failed_step = -1, retries = 0;
    int* exp_used = nullptr; int* attempts = nullptr; unsigned char* doubled = nullptr;   // host arrays or null
    const float* cot = nullptr;     // device fp32 [n_steps][B, D] running-cost cotangents, or null
    float* dt_host = nullptr;       // host [n_steps + 1]: receives dL/dt, or null
};

// What the fused Runge-Kutta kernels need to know about one solve (filled by the host driver).
struct FusedSolve {
    int n_steps = 0, stages = 0, round_increment = 0;
    unsigned long long wait_ns = 2000000000ull; // limit of every device-side wait
    int starve = 0;                             // test of the bounded waits: the forward program's second phase waits for a
                                                // count that is never reached
    const void* traj = nullptr;                 // low [(n_steps+1), B, d]
    float* y = nullptr;                         // fp32 running state [B, D]
    std::vector<RkStepScalars> scalars;         // one entry per step
    double a[16] = {0};                         // tableau, row-major stages x stages
};

// Offsets (bytes) into the caller-provided workspace; every slice is 256-byte aligned.
struct Layout {
    size_t total = 0;
    size_t scal = 0;          // 64 words, zeroed by every forward pass: [0] non-finite flag (u32), [1] ||a||_inf (f32), [2] error word of the
                              // bounded waits, [8..10] scale state (log2 S, failed step, bad input), [12..14] its copy when no mapped
                              // host words exist, [16] last-block counter of the convolution weight-gradient reduction,
                              // [17] that of the hypernetwork flow's cotangent sums, [20..23] those of its whole-step product, [24..55] those of the column sums
    size_t kbuf[4] = {0};     // stage derivatives k_j, low [B, d]
    size_t klbuf[4] = {0};    // CNF: log-density component of k_j, low [B]
    size_t ybuf[4] = {0};     // stage inputs Y_j, low [B, d] (CNF: [2B, d], second half = probe)
    size_t psi[4] = {0};      // stage input cotangents psi_j, low [B, d]
    size_t v = 0, vl = 0;     // seed Q16(S a): state part low [B, d], CNF log-density part low [B]
    size_t kappa = 0, kappal = 0;
    size_t dg = 0;            // per-step parameter gradient, fp32 [p]
    size_t slog = 0;          // dynamic scaling: the device-side scale log, int exponent [max_steps], int attempts [max_steps], byte doubled [max_steps]
    // time-grid gradient (policy.time_gradient): t' fp32 [max_steps + 1]; scratch floats: partial sums of Phi^T a [148], of the
    // <psi_j, k_l> terms [148], dtau_j [4], c_j [4], {Phi^T a, dt, dh} [4]
    bool time_gradient = false;
    size_t tprime = 0, tdots = 0;
    size_t take(size_t bytes) {
        size_t o = total;
        total += (bytes + 255) & ~(size_t)255;
        return o;
    }
};

// kappa_{j-1} = Q16(bv * v + c * psi_j): the previous stage's cotangent when the tableau couples it to stage j alone
struct KappaNext { void* out = nullptr; const void* v = nullptr; float bv = 0.f, c = 0.f; };

class Velocity {
public:
    virtual ~Velocity() {}
    virtual size_t param_count() const = 0;
    // reserve the common and the velocity-specific workspace slices
    virtual void plan(Layout& lay) = 0;
    // Q16(theta) into the workspace (and any per-pass constants such as the probe in low format)
    virtual void prepare(cudaStream_t st, void* ws, const float* theta, const signed char* probe, long long* L) = 0;
    // k_j = f(tau_j, Y_j): reads the stage input, writes kbuf[j] (and klbuf[j]); keeps the layer outputs of stage j
    virtual void forward(cudaStream_t st, void* ws, int j, const void* yin, float tau16, long long* L) = 0;
    // (psi_j, dtheta_j) = VJP of stage j with the cotangent in the kappa buffer; dg = beta * dg + dtheta_j
    virtual void vjp(cudaStream_t st, void* ws, int j, const void* yin, float tau16, void* psi_out, float* dg,
                     float beta, unsigned* flag, long long* L) = 0;
    // Velocities that can write the previous stage's cotangent from the epilogue that produces psi_j: the driver asks with
    // can_write_next_kappa(), hands the request over before vjp(), and vjp() then writes `out` whatever kernel it ends up taking.
    virtual bool can_write_next_kappa() const { return false; }
    virtual void set_next_kappa(const KappaNext&) {}
    // whether the velocity can return the cotangent of its stage times (time-grid gradient), written to dtau[j] by vjp / fused_vjp
    virtual bool supports_time_gradient() const { return false; }
    // velocities whose parameters are piecewise constant in time are told which step the following calls belong to
    virtual void set_step(int step, int n_steps) {}
    // true when stage 0 cannot read the trajectory slice in place (it needs the input in its own buffer)
    virtual bool needs_input_copy() const { return false; }
    virtual size_t kappa_offset(const Layout& lay) const { return lay.kappa; }
    // called after prepare(), once per pass: whatever depends on the solve's time grid and on the parameters alone
    virtual void prepare_solve(cudaStream_t st, void* ws, const FusedSolve& fs, long long* L) {}
    // Velocities that act on each sample by itself may take a whole step at a time: step_forward forms every stage input
    // Y_j = Q16(ybar + sum_{l<j} (h a_jl) k_l) and stage derivative (kbuf, klbuf; the stage inputs of stages > 0 into ybuf);
    // step_vjp forms every stage cotangent from the seed in the layout's v / vl buffers, writes psi_j into the layout's psi
    // buffers and the step's parameter gradient into dg.  false = not available, the caller then goes stage by stage.
    virtual bool step_forward(cudaStream_t st, void* ws, const void* ybar, const RkStepScalars& sc, int stages, long long* L) { return false; }
    virtual bool step_vjp(cudaStream_t st, void* ws, const void* ybar, const RkStepScalars& sc, int stages, float* dg, unsigned* flag,
                          long long* L) { return false; }
    // Whole forward time loop (all steps, stages and layers) in one persistent launch; false = not available for this
    // velocity / format / shape, the caller then runs the layer-by-layer path.
    virtual bool fused_forward(cudaStream_t st, void* ws, const FusedSolve& fs, long long* L) { return false; }
    // Very small velocities: the whole forward pass (Alg. 1) or backward pass (Alg. 2, including the scale decisions) in one
    // launch; false = not available.  whole_backward synchronises the stream to read back the status and the scale log.
    virtual bool whole_forward(cudaStream_t st, void* ws, const FusedSolve& fs, const float* theta, const float* y0, float* yT,
                               long long* L) { return false; }
    virtual bool whole_backward(cudaStream_t st, void* ws, const FusedSolve& fs, WholeBackward& wb, long long* L) { return false; }
    // Fused backward: begin() prepares the phase tables of one solve (false = not available); then per step one
    // recompute launch (keeps every layer output of every stage) and, per attempt, one launch for all stage
    // vector-Jacobian products and weight gradients.  fused_vjp reads the seed from the layout's v buffer, writes
    // psi_j into the layout's psi buffers and the step's parameter gradient into dg.
    virtual bool fused_backward_begin(cudaStream_t st, void* ws, const FusedSolve& fs, long long* L) { return false; }
    virtual void fused_recompute(cudaStream_t st, void* ws, const FusedSolve& fs, int step, long long* L) {}
    // out = (beta ? beta * out : 0) + coef * (parameter gradient of the step): the step gradient itself, or the update
    // g <- g + (h / S) dg when no finiteness decision stands between the two
    // With `st_finish` != null the reductions that follow the fused launch run on that stream, after `after_kernel` (recorded
    // on `st` right behind the launch).
    virtual void fused_vjp(cudaStream_t st, void* ws, const FusedSolve& fs, int step, float* out, float beta, float coef,
                           unsigned* flag, long long* L, cudaEvent_t after_kernel = nullptr, cudaStream_t st_finish = nullptr) {}
    // where the seed kernel writes the last stage's cotangent kappa_s = Q16(b_s v) for fused_vjp
    virtual void* fused_kappa_last(void* ws) const { return nullptr; }
};

Velocity* make_velocity(const mpode_velocity_desc& desc, int batch, mpode_dtype low, int max_steps);

}  // namespace mpode
