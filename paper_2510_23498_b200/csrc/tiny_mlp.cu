// Whole-solve kernels for very small dense velocities: see tiny_mlp.h.  Arithmetic and rounding points are those of the
// layer-by-layer path: operands rounded to the low format (Q16), products accumulated in fp32 in ascending index order,
// one rounding per layer output / cotangent, activation derivatives from the rounded stored output.
#include "tiny_mlp.h"

#include <math.h>

namespace mpode {
namespace {

template <typename T> __device__ __forceinline__ float q16(float x) { return Low<T>::to_f(Low<T>::from_f(x)); }
template <typename T> __device__ __forceinline__ bool q_nonfinite(float rounded) { return Low<T>::nonfinite(Low<T>::from_f(rounded)); }

// sum of two low-format values, rounded once (the exact sum fits a double)
template <typename T> __device__ __forceinline__ float q16_sum(float a, float b);
template <> __device__ __forceinline__ float q16_sum<float>(float a, float b) { return (float)((double)a + (double)b); }
template <> __device__ __forceinline__ float q16_sum<__half>(float a, float b) { return __half2float(__double2half((double)a + (double)b)); }
template <> __device__ __forceinline__ float q16_sum<__nv_bfloat16>(float a, float b) {
    return __bfloat162float(__double2bfloat16((double)a + (double)b));
}

struct TinyWeights {     // shared memory: Q16(theta) as floats
    float* W1; float* b1; float* W2; float* b2; int in1;
};

template <typename T>
__device__ void tiny_load_weights(const TinyParams& p, float* sm, TinyWeights& w) {
    const int in1 = p.d + (p.time ? 1 : 0);
    const int n1 = p.h * in1, nb1 = p.bias ? p.h : 0, n2 = p.d * p.h, nb2 = p.bias ? p.d : 0;
    w.in1 = in1;
    w.W1 = sm; w.b1 = sm + n1; w.W2 = w.b1 + p.h; w.b2 = w.W2 + n2;
    const float* th = p.theta;
    if (p.poly) {       // Q16(theta_1..3) at the start of the weight area
        if (threadIdx.x < 3) w.W1[threadIdx.x] = q16<T>(th[threadIdx.x]);
        __syncthreads();
        return;
    }
    for (int i = threadIdx.x; i < n1; i += blockDim.x) w.W1[i] = q16<T>(th[i]);
    for (int i = threadIdx.x; i < p.h; i += blockDim.x) w.b1[i] = nb1 ? q16<T>(th[n1 + i]) : 0.f;
    for (int i = threadIdx.x; i < n2; i += blockDim.x) w.W2[i] = q16<T>(th[n1 + nb1 + i]);
    for (int i = threadIdx.x; i < p.d; i += blockDim.x) w.b2[i] = nb2 ? q16<T>(th[n1 + nb1 + n2 + i]) : 0.f;
    __syncthreads();
}

// k = f(tau, Y): H = Q16(act(W1 [Y; tau] + b1)), k = Q16(W2 H + b2)
template <typename T>
__device__ __forceinline__ void tiny_eval(const TinyParams& p, const TinyWeights& w, float tau16, const float* Y, float* H, float* k) {
    if (p.poly) {       // Example 1, one rounding per operation; lambda and t^2 are kept for the backward pass
        const float t2 = q16<T>(tau16 * tau16);
        const float lam = q16_sum<T>(q16_sum<T>(q16<T>(w.W1[0] * t2), q16<T>(w.W1[1] * tau16)), w.W1[2]);
        H[0] = lam; H[1] = t2;
        k[0] = q16<T>(-lam * Y[0]);
        return;
    }
    for (int n = 0; n < p.h; ++n) {
        float z = 0.f;
        for (int c = 0; c < p.d; ++c) z = fmaf(Y[c], w.W1[n * w.in1 + c], z);
        z += w.b1[n];
        if (p.time) z = fmaf(tau16, w.W1[n * w.in1 + p.d], z);
        H[n] = q16<T>(act_fwd(p.act, z));
    }
    for (int i = 0; i < p.d; ++i) {
        float z = 0.f;
        for (int n = 0; n < p.h; ++n) z = fmaf(H[n], w.W2[i * p.h + n], z);
        k[i] = q16<T>(z + w.b2[i]);
    }
}

// All stages of one step from the stored low-precision state ybar (Alg. 1 increment / Alg. 2 recompute)
template <typename T>
__device__ __forceinline__ void tiny_stages(const TinyParams& p, const TinyWeights& w, const RkStepScalars& sc, const float* ybar,
                                            float (*Y)[TINY_MAX_D], float (*H)[TINY_MAX_H], float (*K)[TINY_MAX_D]) {
    for (int j = 0; j < p.stages; ++j) {
        for (int c = 0; c < p.d; ++c) {
            float acc = ybar[c];
            for (int l = 0; l < j; ++l)
                if (sc.ha[j][l] != 0.f) acc = fmaf(sc.ha[j][l], K[l][c], acc);
            Y[j][c] = j == 0 ? ybar[c] : q16<T>(acc);
        }
        tiny_eval<T>(p, w, sc.tau16[j], Y[j], H[j], K[j]);
    }
}

template <typename T>
__global__ void __launch_bounds__(TINY_MAX_B, 1) tiny_forward_kernel(TinyParams p) {
    extern __shared__ float sm[];
    TinyWeights w;
    tiny_load_weights<T>(p, sm, w);
    const int b = threadIdx.x;
    if (b >= p.B) return;
    T* traj = (T*)p.traj;
    float y[TINY_MAX_D], ybar[TINY_MAX_D];
    float Y[RK_MAX_STAGES][TINY_MAX_D], H[RK_MAX_STAGES][TINY_MAX_H], K[RK_MAX_STAGES][TINY_MAX_D];
    for (int c = 0; c < p.d; ++c) {
        y[c] = p.y0[(long long)b * p.d + c];
        const T q = Low<T>::from_f(y[c]);
        traj[(long long)b * p.d + c] = q;
        ybar[c] = Low<T>::to_f(q);
    }
    for (int i = 0; i < p.n_steps; ++i) {
        const RkStepScalars sc = p.scal[i];
        tiny_stages<T>(p, w, sc, ybar, Y, H, K);
        for (int c = 0; c < p.d; ++c) {
            float acc = 0.f;
            for (int j = 0; j < p.stages; ++j) acc = fmaf(sc.hb[j], K[j][c], acc);
            y[c] += p.round_increment ? sc.h * q16<T>(acc) : acc;
            const T q = Low<T>::from_f(y[c]);
            traj[((long long)(i + 1) * p.B + b) * p.d + c] = q;
            ybar[c] = Low<T>::to_f(q);
        }
    }
    for (int c = 0; c < p.d; ++c) p.yT[(long long)b * p.d + c] = y[c];
}


// ---------------------------------------------------------------------------------------------------- block reductions
__device__ __forceinline__ float block_max(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float m = red[0];
    for (int i = 1; i < (int)(blockDim.x >> 5); ++i) m = fmaxf(m, red[i]);
    return m;
}

// S_N = 2^floor(-log2(u_L m)) in integer arithmetic (u_L = 2^-pbits, m = f 2^E with f in [0.5, 1))
__device__ __forceinline__ int tiny_initial_exponent(float m, int pbits) {
    if (m == 0.f) return 0;
    int E;
    const float f = frexpf(m, &E);
    const int e = pbits - ((f > 0.5f) ? E : E - 1);
    return e < -100 ? -100 : (e > 100 ? 100 : e);
}

template <typename T>
__global__ void __launch_bounds__(TINY_MAX_B, 1) tiny_backward_kernel(TinyParams p) {
    extern __shared__ float sm[];
    TinyWeights w;
    const int in1 = p.d + (p.time ? 1 : 0);
    const int n1 = p.h * in1, nb1 = p.bias ? p.h : 0, n2 = p.d * p.h, nb2 = p.bias ? p.d : 0;
    const int P = p.poly ? 3 : n1 + nb1 + n2 + nb2;
    const bool want_dt = p.tprime != nullptr;
    const int P3 = P + (want_dt ? 3 : 0);      // behind the parameters: dt, dh and Phi^T a of the step, summed over the batch alike
    const int o_b1 = n1, o_w2 = n1 + nb1, o_b2 = n1 + nb1 + n2;
    const int nwarps = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* part = sm + (p.h * in1 + p.h + p.d * p.h + p.d);          // [nwarps][P3] per-warp sums
    float* dgs = part + (size_t)nwarps * P3;                           // [P3] parameter gradient of the step (+ dt, dh, Phi^T a)
    float* red = dgs + P3;                                             // [32]
    tiny_load_weights<T>(p, sm, w);

    const int b = threadIdx.x;
    const bool active = b < p.B;
    const T* traj = (const T*)p.traj;
    const bool dynamic = p.scaling == MPODE_SCALE_DYNAMIC, checked = p.scaling != MPODE_SCALE_NONE;

    float a[TINY_MAX_D];
    bool in_bad = false;
    float amax = 0.f;
    for (int c = 0; c < p.d; ++c) {
        a[c] = active ? p.dLdyT[(long long)b * p.d + c] : 0.f;
        in_bad |= Low<float>::nonfinite(a[c]);
        amax = fmaxf(amax, fabsf(a[c]));
    }
    int e = p.e0;
    if (dynamic) {
        const float m = block_max(amax, red);
        if (__syncthreads_or(in_bad) || !(m <= 3.4028234e38f)) {
            if (threadIdx.x == 0) p.status[0] = MPODE_ERR_NONFINITE_INPUT;
            return;
        }
        if (p.e0_from_norm) e = tiny_initial_exponent(m, p.pbits);
    }
    if (!p.accumulate)
        for (int i = threadIdx.x; i < P; i += blockDim.x) p.g[i] = 0.f;
    __syncthreads();

    float Y[RK_MAX_STAGES][TINY_MAX_D], H[RK_MAX_STAGES][TINY_MAX_H], K[RK_MAX_STAGES][TINY_MAX_D], psi[RK_MAX_STAGES][TINY_MAX_D];
    // per stage: the cotangent of the layer-1 pre-activation and of the stage derivative (the parameter gradients are formed from
    // them after the stage loop, term by term, so that no per-sample gradient vector has to live in local memory)
    float DZ[RK_MAX_STAGES][TINY_MAX_H], KAP[RK_MAX_STAGES][TINY_MAX_D];
    int retries = 0, overflow_seen = 0;
    const int s = p.stages;
    const int k_lim = dynamic ? p.k_max : 1;

    for (int i = p.n_steps - 1; i >= 0; --i) {
        const RkStepScalars sc = p.scal[i];
        float ybar[TINY_MAX_D];
        for (int c = 0; c < p.d; ++c) ybar[c] = active ? Low<T>::to_f(traj[((long long)i * p.B + b) * p.d + c]) : 0.f;
        tiny_stages<T>(p, w, sc, ybar, Y, H, K);                       // recompute the increment
        float phi_a = 0.f;                                             // this sample's share of Phi^T a_{i+1} (adjoint before its update)
        if (want_dt) {
            for (int c = 0; c < p.d; ++c) {
                float ph = 0.f;
                for (int j = 0; j < s; ++j) ph = fmaf(sc.b[j], K[j][c], ph);
                if (p.round_increment) ph = q16<T>(ph);
                phi_a = fmaf(ph, a[c], phi_a);
            }
        }
        int k_try = 0;
        bool accepted = false;
        while (k_try < k_lim) {
            ++k_try;
            bool bad = false;
            float v[TINY_MAX_D];
            for (int c = 0; c < p.d; ++c) { v[c] = q16<T>(ldexpf(a[c], e)); bad |= q_nonfinite<T>(v[c]); }   // Q16(S a)
            float g_dt = 0.f, g_dh = 0.f;                              // this sample's dt and dh (Eq. (vjp))
            float g_p0 = 0.f, g_p1 = 0.f, g_p2 = 0.f;                  // scalar example: its three parameter cotangents
            for (int j = s - 1; j >= 0; --j) {
                float dtau = 0.f;                                      // cotangent of the stage time tau_j, this sample's share
                float kap[TINY_MAX_D];
                for (int c = 0; c < p.d; ++c) {
                    float acc = sc.b[j] * v[c];
                    for (int l = j + 1; l < s; ++l)
                        if (sc.ha[l][j] != 0.f) acc = fmaf(sc.ha[l][j], psi[l][c], acc);
                    kap[c] = q16<T>(acc);
                    bad |= q_nonfinite<T>(kap[c]);
                    KAP[j][c] = kap[c];
                }
                if (p.poly) {   // psi = Q16(-lambda kappa); cotangent of lambda and of the three parameters, each product rounded
                    const float lam = H[j][0], t2 = H[j][1];
                    const float ps = q16<T>(-lam * kap[0]);
                    const float dlam = q16<T>(-Y[j][0] * kap[0]);
                    const float d1 = q16<T>(dlam * t2), d2 = q16<T>(dlam * sc.tau16[j]);
                    bad |= q_nonfinite<T>(ps) | q_nonfinite<T>(dlam) | q_nonfinite<T>(d1) | q_nonfinite<T>(d2);
                    psi[j][0] = ps;
                    g_p0 += d1; g_p1 += d2; g_p2 += dlam;
                    if (want_dt) {      // d lambda / d tau = 2 theta_1 tau + theta_2, operation by operation
                        const float dt2 = q16<T>(dlam * w.W1[0]);
                        const float dts = q16_sum<T>(q16<T>(dt2 * q16<T>(2.f * sc.tau16[j])), q16<T>(dlam * w.W1[1]));
                        bad |= q_nonfinite<T>(dt2) | q_nonfinite<T>(dts);
                        g_dt += dts;
                        float dhs = sc.c[j] * dts;
                        for (int l = 0; l < j; ++l)
                            if (sc.a[j][l] != 0.f) dhs = fmaf(sc.a[j][l], ps * K[l][0], dhs);
                        g_dh += dhs;
                    }
                    continue;
                }
                // last layer: dX = W2^T kappa (dW2 += kappa H^T and db2 += kappa follow after the stage loop)
                for (int c = 0; c < p.d; ++c) psi[j][c] = 0.f;
                for (int n = 0; n < p.h; ++n) {
                    float dx = 0.f;
                    for (int c = 0; c < p.d; ++c) dx = fmaf(kap[c], w.W2[c * p.h + n], dx);
                    const float dz = q16<T>(act_deriv_from_output(p.act, H[j][n]) * dx);
                    bad |= q_nonfinite<T>(dz);
                    DZ[j][n] = dz;
                    for (int c = 0; c < p.d; ++c) psi[j][c] = fmaf(dz, w.W1[n * in1 + c], psi[j][c]);
                    if (p.time) dtau = fmaf(dz, w.W1[n * in1 + p.d], dtau);
                }
                for (int c = 0; c < p.d; ++c) { psi[j][c] = q16<T>(psi[j][c]); bad |= q_nonfinite<T>(psi[j][c]); }
                if (want_dt) {      // tau_j = t_i + c_j h and Y_j = ybar + h sum_l a_jl k_l both depend on the grid
                    g_dt += dtau;
                    float dhs = sc.c[j] * dtau;
                    for (int l = 0; l < j; ++l) {
                        if (sc.a[j][l] == 0.f) continue;
                        float dot = 0.f;
                        for (int c = 0; c < p.d; ++c) dot = fmaf(psi[j][c], K[l][c], dot);
                        dhs = fmaf(sc.a[j][l], dot, dhs);
                    }
                    g_dh += dhs;
                }
            }
            // This sample's share of every parameter's gradient (the stages added last to first, as they were computed), summed
            // over the batch: lanes by shuffles, warps in ascending order below
            auto to_part = [&](int i2, float x) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
                if (lane == 0) part[(size_t)warp * P3 + i2] = x;
            };
            if (p.poly) {
                to_part(0, g_p0); to_part(1, g_p1); to_part(2, g_p2);
            } else {
                for (int n = 0; n < p.h; ++n) {
                    for (int c = 0; c < p.d; ++c) {                    // dW1 = dZ Y^T
                        float x = 0.f;
                        for (int j = s - 1; j >= 0; --j) x = fmaf(DZ[j][n], Y[j][c], x);
                        to_part(n * in1 + c, x);
                    }
                    if (p.time) {                                      // the time column: tau_j dZ
                        float x = 0.f;
                        for (int j = s - 1; j >= 0; --j) x = fmaf(sc.tau16[j], DZ[j][n], x);
                        to_part(n * in1 + p.d, x);
                    }
                    if (nb1) {
                        float x = 0.f;
                        for (int j = s - 1; j >= 0; --j) x += DZ[j][n];
                        to_part(o_b1 + n, x);
                    }
                }
                for (int c = 0; c < p.d; ++c) {                        // dW2 = kappa H^T, db2 = kappa
                    for (int n = 0; n < p.h; ++n) {
                        float x = 0.f;
                        for (int j = s - 1; j >= 0; --j) x = fmaf(KAP[j][c], H[j][n], x);
                        to_part(o_w2 + c * p.h + n, x);
                    }
                    if (nb2) {
                        float x = 0.f;
                        for (int j = s - 1; j >= 0; --j) x += KAP[j][c];
                        to_part(o_b2 + c, x);
                    }
                }
            }
            if (want_dt) { to_part(P, g_dt); to_part(P + 1, g_dh); to_part(P + 2, phi_a); }
            __syncthreads();
            for (int i2 = threadIdx.x; i2 < P3; i2 += blockDim.x) {
                float x = 0.f;
                for (int ww = 0; ww < nwarps; ++ww) x += part[(size_t)ww * P3 + i2];
                dgs[i2] = x;
                if (checked && i2 < P + 2) bad |= q_nonfinite<T>(x);  // are Q16(dg), Q16(dt), Q16(dh) finite?
            }
            const int any_bad = __syncthreads_or(bad && checked);
            if (!checked) { accepted = true; break; }
            if (!dynamic) { overflow_seen |= any_bad; accepted = true; break; }
            if (!any_bad) { accepted = true; break; }
            if (e > -100) --e;                                         // halve and retry
            ++retries;
        }
        if (threadIdx.x == 0) { p.log_exp[i] = e; p.log_attempts[i] = k_try; p.log_doubled[i] = 0; }
        if (!accepted) {
            if (threadIdx.x == 0) { p.status[0] = MPODE_ERR_SCALE_FAILED; p.status[1] = i; p.status[2] = retries; }
            return;
        }
        // high-precision updates with h / S
        const float coef = (float)((double)sc.h * ldexp(1.0, -e));
        float m = 0.f;
        for (int c = 0; c < p.d; ++c) {
            float da = 0.f;
            for (int j = s - 1; j >= 0; --j) da += psi[j][c];
            a[c] = fmaf(coef, da, a[c]);
            if (p.cot != nullptr && active) a[c] += p.cot[((long long)i * p.B + b) * p.d + c];     // w_i dR/dy_i
            m = fmaxf(m, fabsf(a[c]));
        }
        for (int i2 = threadIdx.x; i2 < P; i2 += blockDim.x) p.g[i2] = fmaf(coef, dgs[i2], p.g[i2]);
        if (want_dt && threadIdx.x == 0) {                             // Alg. 2: the two t' updates
            const float dts = dgs[P], dhs = dgs[P + 1], ph = dgs[P + 2];
            p.tprime[i] = p.tprime[i] + coef * (dts - dhs) - ph;
            p.tprime[i + 1] = p.tprime[i + 1] + coef * dhs + ph;
        }
        if (dynamic && k_try == 1) {                                   // growth test
            const float mm = block_max(m, red);
            const double scaled = p.growth_rule == 0 ? ldexp((double)mm, e) : (double)mm;
            if (scaled <= ldexp(1.0, p.pbits - 1) && e < 100) {
                ++e;
                if (threadIdx.x == 0) p.log_doubled[i] = 1;
            }
        }
        __syncthreads();
    }
    if (p.scaling == MPODE_SCALE_NONE_SAFE && overflow_seen) {
        for (int c = 0; c < p.d; ++c) a[c] = INFINITY;
        __syncthreads();
        for (int i2 = threadIdx.x; i2 < P; i2 += blockDim.x) p.g[i2] = INFINITY;
        if (want_dt)
            for (int i2 = threadIdx.x; i2 <= p.n_steps; i2 += blockDim.x) p.tprime[i2] = INFINITY;
        if (threadIdx.x == 0) p.status[0] = MPODE_WARN_NONFINITE_GRAD;
    }
    if (threadIdx.x == 0) p.status[2] = retries;
    if (active)
        for (int c = 0; c < p.d; ++c) p.a[(long long)b * p.d + c] = a[c];
}

size_t tiny_smem_bytes(const TinyParams& p, int threads, bool backward) {
    const int in1 = p.d + (p.time ? 1 : 0);
    size_t fl = (size_t)p.h * in1 + p.h + (size_t)p.d * p.h + p.d;
    if (backward) {
        const int P = (p.poly ? 3 : p.h * in1 + (p.bias ? p.h : 0) + p.d * p.h + (p.bias ? p.d : 0)) + 3;
        fl += (size_t)(threads / 32) * P + P + 32;
    }
    return fl * sizeof(float);
}

}  // namespace

bool tiny_mlp_supported(int B, int d, int h, int n_layers, int p) {
    return n_layers == 2 && d >= 1 && d <= TINY_MAX_D && h >= 1 && h <= TINY_MAX_H && B >= 1 && B <= TINY_MAX_B && p <= TINY_MAX_P;
}

void launch_tiny_forward(mpode_dtype dt, const TinyParams& p, cudaStream_t st, long long* launches) {
    const int threads = ((p.B + 31) / 32) * 32;
    const size_t smem = tiny_smem_bytes(p, threads, false);
    if (dt == MPODE_BF16) tiny_forward_kernel<__nv_bfloat16><<<1, threads, smem, st>>>(p);
    else if (dt == MPODE_F16) tiny_forward_kernel<__half><<<1, threads, smem, st>>>(p);
    else tiny_forward_kernel<float><<<1, threads, smem, st>>>(p);
    if (launches) ++*launches;
}

void launch_tiny_backward(mpode_dtype dt, const TinyParams& p, cudaStream_t st, long long* launches) {
    const int threads = ((p.B + 31) / 32) * 32;
    const size_t smem = tiny_smem_bytes(p, threads, true);
    static bool attr[3] = {false, false, false};
    const int k = dt == MPODE_BF16 ? 1 : (dt == MPODE_F16 ? 2 : 0);
    if (!attr[k]) {
        const int cap = 200 * 1024;
        if (k == 1) cudaFuncSetAttribute(tiny_backward_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap);
        else if (k == 2) cudaFuncSetAttribute(tiny_backward_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap);
        else cudaFuncSetAttribute(tiny_backward_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, cap);
        attr[k] = true;
    }
    if (k == 1) tiny_backward_kernel<__nv_bfloat16><<<1, threads, smem, st>>>(p);
    else if (k == 2) tiny_backward_kernel<__half><<<1, threads, smem, st>>>(p);
    else tiny_backward_kernel<float><<<1, threads, smem, st>>>(p);
    if (launches) ++*launches;
}

}  // namespace mpode
