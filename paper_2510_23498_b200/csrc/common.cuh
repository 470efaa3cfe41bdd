// Shared device helpers: the low-precision type traits (Q16 of Sec. 2), activation functions and the
// internal launch interface between the host driver and the kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mpode.h"

namespace mpode {

// ---------------------------------------------------------------- low-format traits (round to nearest even)
template <typename T> struct Low;
template <> struct Low<float> {
    static __host__ __device__ __forceinline__ float to_f(float x) { return x; }
    static __host__ __device__ __forceinline__ float from_f(float x) { return x; }
    static __device__ __forceinline__ bool nonfinite(float x) {
        return (__float_as_uint(x) & 0x7F800000u) == 0x7F800000u;
    }
};
template <> struct Low<__half> {
    static __host__ __device__ __forceinline__ float to_f(__half x) { return __half2float(x); }
    static __host__ __device__ __forceinline__ __half from_f(float x) { return __float2half_rn(x); }
    static __device__ __forceinline__ bool nonfinite(__half x) {
        return (__half_as_ushort(x) & 0x7C00u) == 0x7C00u;
    }
};
template <> struct Low<__nv_bfloat16> {
    static __host__ __device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
    static __host__ __device__ __forceinline__ __nv_bfloat16 from_f(float x) { return __float2bfloat16_rn(x); }
    static __device__ __forceinline__ bool nonfinite(__nv_bfloat16 x) {
        return (__bfloat16_as_ushort(x) & 0x7F80u) == 0x7F80u;
    }
};

// Q16 applied to a host scalar (stage times), returned as float.
inline float round_scalar_to_low(float x, mpode_dtype dt) {
    switch (dt) {
        case MPODE_BF16: return __bfloat162float(__float2bfloat16_rn(x));
        case MPODE_F16: return __half2float(__float2half_rn(x));
        default: return x;
    }
}
inline size_t low_size(mpode_dtype dt) { return dt == MPODE_F32 ? 4 : 2; }

// ---------------------------------------------------------------- activations
// softplus(x) = max(x, 0) + log1p(exp(-|x|)); derivatives are written in terms of the stored output H.
__device__ __forceinline__ float act_fwd(int act, float z) {
    switch (act) {
        case MPODE_ACT_TANH: return tanhf(z);
        case MPODE_ACT_SOFTPLUS: return fmaxf(z, 0.f) + log1pf(expf(-fabsf(z)));
        case MPODE_ACT_RELU: return fmaxf(z, 0.f);
        default: return z;
    }
}
__device__ __forceinline__ float act_deriv_from_output(int act, float h) {
    switch (act) {
        case MPODE_ACT_TANH: return 1.f - h * h;
        case MPODE_ACT_SOFTPLUS: return -expm1f(-h);
        case MPODE_ACT_RELU: return h > 0.f ? 1.f : 0.f;
        default: return 1.f;
    }
}

// One flag word per attempt (Alg. 2, finiteness test): any thread that produced a non-finite low-precision value ORs 1
// into it; the OR is taken per warp first so that at most one atomic per warp is issued.
__device__ __forceinline__ void warp_flag_or(unsigned* flag, bool bad) {
    // every lane of the warp must call this (kernels accumulate `bad` in a register and call it once at the end)
    unsigned any = __ballot_sync(0xffffffffu, bad);
    if (flag != nullptr && any != 0u && (threadIdx.x & 31) == 0) atomicOr(flag, 1u);
}

// ---------------------------------------------------------------- dense / implicit-conv contraction (SIMT path)
enum Epilogue : int {
    EPI_FWD = 0,     // out = Q16(act(acc + bias + tau * wt))          (low-format output)
    EPI_DGRAD = 1,   // out = Q16(act'(hprev) * acc), raises the flag   (low-format output)
    EPI_WGRAD = 2,   // out32 = beta * out32 + acc                      (fp32 output)
    EPI_RAW32 = 3    // out32 = acc
};

struct GemmArgs {
    // C(m, n) = sum_k A(m, k) * B(n, k); element (i, k) of an operand sits at ptr[i * rs + k * ks].
    const void* A; long long a_rs, a_ks;
    const void* B; long long b_rs, b_ks;
    int M, N, K;
    // Implicit 3x3 convolution view of one operand (0 = off, 1 = A, 2 = B): the operand's "row" index runs over
    // NHWC pixels (b, y, x) and its "k" index over (tap, channel) with `conv_ct` channels per tap; channels
    // >= conv_cd read the constant conv_tau inside the image (the appended time channel); everything is 0 in
    // the zero-padding halo.  The operand pointer is the NHWC tensor with conv_cd channels.
    int conv_on, conv_h, conv_w, conv_cd, conv_ct;
    float conv_tau;
    // EPI_FWD on the tensor-core convolution path: fp32 table [9][N] of bias + tau * (time-channel weights of the taps that
    // fall inside the image), one row per position class 3 * (0 top, 1 middle, 2 bottom) + (0 left, 1 middle, 2 right)
    const float* conv_tbias;
    int epi;
    void* out; long long ldo;
    void* out2; int m_split;        // rows >= m_split are written to out2 (row m - m_split) without bias/activation
    const void* bias;               // low format [N] or null
    const void* wt; float tau;      // time column of the first layer, low format [N] or null
    int act;
    const void* hprev; long long ldh;
    float beta;
    unsigned* flag;
    unsigned* err;                  // device word that a kernel sets when a bounded wait gives up
    int split_k; float* partial;    // EPI_WGRAD only: split the K loop over gridDim.z, partial sums in `partial`
    // EPI_DGRAD without hprev, kernels that take it only (conv_tc.cu): beside out = psi also kap_out = Q16(kap_bv * v + kap_c * psi),
    // the cotangent of the previous stage (Eq. (vjp) through the tableau), non-finite values flagged; v, kap_out: low format [M, N]
    void* kap_out; const void* kap_v; float kap_bv, kap_c;
    // Continuous normalizing flow with a trace estimate (Sec. 6.1), tensor-core kernel only: the operand rows are m_split primal
    // rows followed by their m_split tangent rows, and a tile holds 64 primal rows and the tangent rows of the same samples.
    //   1 (with EPI_FWD): out = H = Q16(act(acc + bias)) for the primal rows, out2 = U = Q16(acc) for the tangent rows, and when
    //     pair_out is given also G = Q16(act'(H) * U) (row = sample);
    //   2 (with EPI_DGRAD): the accumulators are hbar (primal) and gbar (tangent); with s = act'(H) from hprev and U from uprev
    //     (both [m_split, N], leading dimension ldh): out = Q16(s hbar + s (1 - s) U gbar), out2 = Q16(s gbar), non-finite flagged.
    int cnf_pair; void* pair_out; const void* uprev;
};

void launch_gemm_simt(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* launches);

// ---------------------------------------------------------------- elementwise / reduction kernels
struct Terms {                      // up to 4 low-format arrays with fp32 coefficients
    const void* p[4];
    float c[4];
    int n;
};

void launch_quantize_matrix(mpode_dtype dt, const float* src, long long src_ld, int rows, int cols, void* dst,
                            void* dst_t, cudaStream_t st, long long* launches);
void launch_quantize_conv_weights(mpode_dtype dt, const float* src, int cout, int cin_total, int cin_keep, void* dst,
                                  void* dst_flip_t, cudaStream_t st, long long* launches, float sign = 1.f);
// Instance normalisation of an NHWC tensor [B][HW][C] per (image, channel) plane (Sec. 6.3): Z = Q16((S - mean) rstd), and its
// vector-Jacobian product followed by the activation derivative, dU = Q16(act'(S) Q16(rstd (dZ - mean(dZ) - Z mean(dZ Z))))
void launch_instnorm_fwd(mpode_dtype dt, const void* S, void* Z, float* rstd, int B, int HW, int C, float eps, cudaStream_t st,
                         long long* launches);
void launch_instnorm_bwd(mpode_dtype dt, const void* dZ, const void* Z, const void* S, const float* rstd, void* dU, int B, int HW, int C,
                         int act, int norm, unsigned* flag, cudaStream_t st, long long* launches);
// out[(cout * 9 + tap) * ct + cin] = (beta ? out : 0) + sum_z partial[z][tap * C + cin][cout]
void launch_conv_wgrad_reduce(const float* partial, int S, int C, int ct, float* out, float beta, cudaStream_t st, long long* launches,
                              float sign = 1.f);
// Gradients that are sums of a cotangent dZ[p][cout] over pixels (C a multiple of 8 with 128 % (C / 8) == 0):
// bias_out[cout] (+)= sum over all pixels; wt_out[(cout * 9 + tap) * ct + ct - 1] (+)= tau * (sum over the pixels whose tap
// neighbour lies inside the image), the weights of an appended time channel.  Either output may be null.
// `scratch` holds 9 C floats for each of 8 x 148 blocks plus 9 C more; the requested format must be 16-bit.
void launch_conv_class_grads(mpode_dtype dt, const void* dz, int B, int H, int W, int C, int ct, float tau, float* scratch,
                             float* wt_out, float* bias_out, float beta, cudaStream_t st, long long* launches);
// From the [9][C] class sums `cs` of a cotangent (shared memory, all threads of the block call this): the bias gradient (sum over
// all classes) and, for a layer with an appended time channel, the gradient of that channel's weights per tap (tau times the sum
// over the classes in which the tap is inside the image); out = beta * out + value.
__device__ __forceinline__ void conv_class_finish(const float* cs, int C, int ct, float tau, float* __restrict__ wt_out,
                                                  float* __restrict__ bias_out, float beta) {
    if (wt_out != nullptr) {
        for (int i = threadIdx.x; i < 9 * C; i += blockDim.x) {
            const int tap = i / C, co = i - tap * C, dy = tap / 3 - 1, dx = tap % 3 - 1;
            float s = 0.f;
            for (int cls = 0; cls < 9; ++cls) {
                const int ry = cls / 3, rx = cls - ry * 3;
                if ((ry == 0 && dy < 0) || (ry == 2 && dy > 0) || (rx == 0 && dx < 0) || (rx == 2 && dx > 0)) continue;
                s += cs[cls * C + co];
            }
            float* o = wt_out + ((long long)co * 9 + tap) * ct + ct - 1;
            *o = (beta != 0.f ? *o : 0.f) + tau * s;
        }
    }
    if (bias_out != nullptr) {
        for (int co = threadIdx.x; co < C; co += blockDim.x) {
            float s = 0.f;
            for (int cls = 0; cls < 9; ++cls) s += cs[cls * C + co];
            bias_out[co] = (beta != 0.f ? bias_out[co] : 0.f) + s;
        }
    }
}
// the position-class indicator table of one image, [H * W][64] in the low format (see elementwise.cu)
void launch_conv_class_indicator(mpode_dtype dt, int H, int W, void* out, cudaStream_t st, long long* launches);
void launch_conv_class_bias(mpode_dtype dt, const void* b, const void* w, int cin_total, float tau, int C, float* out,
                            cudaStream_t st, long long* launches);
void launch_init_state(mpode_dtype dt, const float* y0, float* y, void* traj0, int B, int d, int D, cudaStream_t st,
                       long long* launches);
void launch_stage_input(mpode_dtype dt, const void* base, const Terms& t, void* out, long long n, cudaStream_t st,
                        long long* launches);
void launch_final_combine(mpode_dtype dt, float* y, const Terms& t, void* traj_next, int B, int d, int D,
                          int round_increment, float h, cudaStream_t st, long long* launches);
void launch_column_combine(mpode_dtype dt, float* y, int D, int col, const Terms& t, int B, int round_increment,
                           float h, cudaStream_t st, long long* launches);
void launch_copy_amax(const float* src, float* dst, long long n, float* amax, unsigned* flag, cudaStream_t st,
                      long long* launches);
// v = Q16(2^e a); optionally also kappa_last = Q16(b_last * v), the cotangent of the last stage.  With `e_dev` the exponent is
// read from the device (dynamic scaling); the commits below then take coef = h and apply 2^-e themselves.
void launch_seed(mpode_dtype dt, const float* a, int e, void* v, void* v_l, int B, int d, int D, unsigned* flag,
                 cudaStream_t st, long long* launches, void* kappa_last = nullptr, float b_last = 0.f, const int* e_dev = nullptr);
void launch_kappa(mpode_dtype dt, const void* v, float bj, const Terms& t, void* out, long long n, unsigned* flag,
                  cudaStream_t st, long long* launches);
// the commits do nothing when *skip_if_set != 0 (dynamic scaling: the attempt overflowed and will be repeated)
// `add` (nullable, fp32 [B, D]): a running-cost cotangent w_i dR/dy_i added after the update (Alg. 2, adjoint update)
void launch_commit_a(mpode_dtype dt, float* a, const Terms& psis, float coef, int B, int d, int D, float* amax,
                     cudaStream_t st, long long* launches, const unsigned* skip_if_set = nullptr, const float* add = nullptr,
                     const int* e_dev = nullptr);

// ---------------------------------------------------------------- time-grid gradient (Alg. 2, the two t' updates)
// Inner products over the batch, summed in a fixed order: part[blockIdx] = sum_p coef[p] * <x_p, y_p> over the block's share of
// the rows.  x_p: low format [B, d]; y_p: low format [B, d], or fp32 with row stride ldy (the adjoint a, [B, D]).
constexpr int kDotBlocks = 148;
struct DotPairs {
    const void* x[8]; const void* y[8]; float coef[8]; int y_f32[8]; int ldx[8], ldy[8]; int n;
};
void launch_dot_partial(mpode_dtype dt, const DotPairs& pr, int B, int d, float* part, cudaStream_t st, long long* launches);
// dtau[j] = sum_m wt[m] * (sum over `rows` partial rows of colsum[j][r][m * stride]): the cotangent of a stage time that enters
// through the first layer's time column; `off[j]` is the element offset of stage j's partial rows, terms <= 4
struct StageTimeArgs { const float* colsum; long long off[4]; int terms, rows, M, stride; const void* wt; float* dtau; };
void launch_stage_time_cot(mpode_dtype dt, const StageTimeArgs& a, cudaStream_t st, long long* launches);
// One block: phi = sum part_phi, dh = sum_j c[j] dtau[j] + sum part_dh, dt = sum_j dtau[j]; out[0..2] = {phi, dt, dh}; raises
// *flag when Q16(dt) or Q16(dh) is not finite
void launch_tgrad_reduce(mpode_dtype dt, const float* part_phi, const float* part_dh, const float* dtau, const float* c, int stages,
                         float* out, unsigned* flag, cudaStream_t st, long long* launches);
// t'[i] += coef (dt - dh) - phi, t'[i+1] += coef dh + phi (skipped when *skip_if_set != 0)
void launch_tgrad_update(float* tprime, int i, const float* vals, float coef, const unsigned* skip_if_set, cudaStream_t st,
                         long long* launches, const int* e_dev = nullptr);
void launch_commit_g(float* g, const float* dg, float coef, long long p, cudaStream_t st, long long* launches,
                     const unsigned* skip_if_set = nullptr, const int* e_dev = nullptr);
// Alg. 2's scale state machine on the device: state = {log2 S, first failed step or -1, dL/dy_N not finite}, mirrored into mapped
// host memory.  init: S_0 from ||a||_inf (or the fixed exponent); decide: accept + growth test, or record the failure and halve.
void launch_scale_init(unsigned* flag, const float* amax, int pbits, int e_fixed, int from_norm, int e_min, int e_max, int* state,
                       int* mirror, cudaStream_t st, long long* launches);
void launch_scale_decide(const unsigned* flag, const float* amax, int* state, int* mirror, int step, int k_try, int growth_rule,
                         int pbits, int e_min, int e_max, int* log_exp, int* log_att, unsigned char* log_dbl, cudaStream_t st,
                         long long* launches);
void launch_check_as_low(mpode_dtype dt, const float* x, long long n, unsigned* flag, cudaStream_t st,
                         long long* launches);
void launch_fill(float* x, float v, long long n, cudaStream_t st, long long* launches);
void launch_scale(float* x, float v, long long n, cudaStream_t st, long long* launches);      // x <- v * x
void launch_fill_low(mpode_dtype dt, void* x, float v, long long n, cudaStream_t st, long long* launches);   // low-format array
// column sums of a low-format [M, N] matrix, deterministic two-pass; dst1[n*s1] (+)= sum, dst2[n*s2] (+)= scale2*sum
// returns the number of partial rows it left in `partial` ([rows][N])
constexpr int kColsumCounters = 32;   // column blocks a one-launch column sum can count (words of the caller's `counters`)
int launch_colsum(mpode_dtype dt, const void* x, int M, int N, float* partial, float* dst1, long long s1, float* dst2,
                  long long s2, float scale2, float beta, cudaStream_t st, long long* launches, unsigned* counters = nullptr);
// column sums of a low-format [M, N] matrix per group of 128 rows (the layout the fused backward kernel also writes)
void launch_colsum_groups(mpode_dtype dt, const void* x, int M, int N, float* out, cudaStream_t st, long long* launches);
// out[m * ldo + n] = (beta ? out : 0) + sum_z partial[z][m][n], z in ascending order
void launch_splitk_reduce(const float* partial, int S, int M, int N, float* out, long long ldo, float beta, cudaStream_t st,
                          long long* launches);
// One launch that turns the fused backward kernel's scratch into the step's parameter gradient, layer by layer:
//   dW_l[m][n]  = sum over slices z (ascending) of partial[z][m][n]
//   db_l[m]     = sum over stages j and batch slices r of colpart[col_off[j] + (r * M + m) * 8]    (bias_off >= 0)
//   dw_t[m]     = sum over stages j of tau[j] * (sum over row blocks ...)                           (time_off >= 0)
// and writes out[i] = (beta != 0 ? beta * out[i] : 0) + coef * value: either the step gradient itself (beta 0, coef 1)
// or straight into the running gradient g <- g + (h / S) dg of Alg. 2 (beta 1, coef h / S).
struct GradFinishLayer {
    const float* partial; int splits, M, N;
    long long w_off; int ldo;
    const float* colpart; long long col_off[4]; float tau[4]; int terms, rows;
    long long bias_off, time_off;
};
struct GradFinishArgs {
    GradFinishLayer layer[8];
    int n_layers;
    float* out;
    float beta, coef;
};
void launch_grad_finish(const GradFinishArgs& a, cudaStream_t st, long long* launches);
// CNF helpers (Sec. 6.1 joint state)
void launch_cnf_tangent_act(mpode_dtype dt, int act, const void* H, const void* U, void* G, long long n,
                            cudaStream_t st, long long* launches);
void launch_cnf_trace(mpode_dtype dt, const signed char* eps, const void* U, void* k_l, int B, int d, cudaStream_t st,
                      long long* launches);
void launch_cnf_probe_to_low(mpode_dtype dt, const signed char* eps, void* out, long long n, cudaStream_t st,
                             long long* launches);
void launch_cnf_ubar_last(mpode_dtype dt, const void* kappa_l, const signed char* eps, void* ubar, int B, int d,
                          unsigned* flag, cudaStream_t st, long long* launches);
void launch_cnf_backprop_act(mpode_dtype dt, int act, const void* H, const void* U, const float* hbar,
                             const float* gbar, void* zeta, void* ubar, long long n, unsigned* flag, cudaStream_t st,
                             long long* launches);

}  // namespace mpode
