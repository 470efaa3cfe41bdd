// The two-dimensional flows of Sec. 6.1 with the exact trace: joint state y = [z; l],
//   z' = v(t, z) = (1/w) sum_j U_j(t) tanh(W_j(t) . z + b_j(t)),     l' = -tr(dv/dz) = -(1/w) sum_j (U_j . W_j) (1 - tanh^2(W_j . z + b_j)),
// the w weight sets (W_j, b_j, U_j) produced from t by three fully connected layers of hidden width h (tanh between them).
// State width d <= 8, so nothing here is a tensor-core contraction.  Two sets of kernels.  A whole step at a time (the usual
// path, see the second half of the file): the hypernetwork is evaluated once per pass for every stage time of the solve, one
// launch evaluates all stages of a step, one forms all stage cotangents, one sums the weight-set cotangents over the batch and
// runs the hypernetwork backwards, one adds the stage gradients.  Stage by stage (when the weight sets of all stages do not fit
// shared memory): per stage evaluation one launch in which every block evaluates the hypernetwork for the stage time into its
// shared memory (block 0 keeps a copy for the backward pass) and then the velocity with one thread per sample; the
// vector-Jacobian product is two launches: per-sample unit cotangents and psi, then one block per weight set that sums its
// cotangents over the batch in a fixed order, and the block that finishes last runs the hypernetwork backwards.
// Rounding points (the paper lists none): the hypernetwork's two hidden layers and its output, the products c_j = Q16(U_j . W_j),
// the units a_j = Q16(tanh(.)), the two outputs; in the vector-Jacobian product the unit cotangents, psi, and the batch-summed
// cotangents of the hypernetwork's output and hidden layers.  Sums are fp32 in a fixed order, one rounding per tensor.
#include "hyper_cnf.h"

#include <math.h>

namespace mpode {
namespace {

#define MPODE_DISPATCH_T(dt, T, ...)                                         \
    do {                                                                     \
        if ((dt) == MPODE_BF16) { using T = __nv_bfloat16; __VA_ARGS__; }    \
        else if ((dt) == MPODE_F16) { using T = __half; __VA_ARGS__; }       \
        else { using T = float; __VA_ARGS__; }                               \
    } while (0)

template <typename T> __device__ __forceinline__ float q16(float x) { return Low<T>::to_f(Low<T>::from_f(x)); }
template <typename T> __device__ __forceinline__ bool q_bad(float rounded) { return Low<T>::nonfinite(Low<T>::from_f(rounded)); }

// Layout of the per-stage block of floats `hyp`: h1 [h], h2 [h], o [m] = W [w][d], b [w], U [w][d], then c [w].

// theta: A1 [h][1], c1 [h], A2 [h][h], c2 [h], A3 [m][h], c3 [m]
struct ThetaOffsets { int A1, c1, A2, c2, A3, c3; };
__host__ __device__ inline ThetaOffsets theta_offsets(int h, int m) {
    ThetaOffsets o;
    o.A1 = 0; o.c1 = h; o.A2 = 2 * h; o.c2 = 2 * h + h * h; o.A3 = 3 * h + h * h; o.c3 = o.A3 + m * h;
    return o;
}

// The hypernetwork for one stage time, by all threads of a block: h1, h2 (shared memory, h floats each), `ws` = W [w][d], b [w],
// U [w][d], c [w] (shared memory).  `keep` (global, or null): h1, h2, ws in that order, for the backward pass.
template <typename T>
__device__ void hyper_eval_block(const float* __restrict__ theta, float tau16, int h, int w, int d, float* h1, float* h2, float* ws,
                                 float* __restrict__ keep) {
    const int m = w * (2 * d + 1);
    const ThetaOffsets o = theta_offsets(h, m);
    for (int i = threadIdx.x; i < h; i += blockDim.x)
        h1[i] = q16<T>(tanhf(fmaf(q16<T>(theta[o.A1 + i]), tau16, q16<T>(theta[o.c1 + i]))));
    __syncthreads();
    for (int i = threadIdx.x; i < h; i += blockDim.x) {
        float z = 0.f;
        for (int j = 0; j < h; ++j) z = fmaf(q16<T>(theta[o.A2 + i * h + j]), h1[j], z);
        h2[i] = q16<T>(tanhf(z + q16<T>(theta[o.c2 + i])));
    }
    __syncthreads();
    for (int i = threadIdx.x; i < m; i += blockDim.x) {
        float z = 0.f;
#pragma unroll 4
        for (int j = 0; j < h; ++j) z = fmaf(q16<T>(theta[o.A3 + i * h + j]), h2[j], z);
        ws[i] = q16<T>(z + q16<T>(theta[o.c3 + i]));
    }
    __syncthreads();
    const float* W = ws;
    const float* U = ws + w * d + w;
    for (int j = threadIdx.x; j < w; j += blockDim.x) {
        float c = 0.f;
        for (int k = 0; k < d; ++k) c = fmaf(U[j * d + k], W[j * d + k], c);
        ws[m + j] = q16<T>(c);
    }
    __syncthreads();
    if (keep != nullptr) {
        for (int i = threadIdx.x; i < h; i += blockDim.x) { keep[i] = h1[i]; keep[h + i] = h2[i]; }
        for (int i = threadIdx.x; i < m + w; i += blockDim.x) keep[2 * h + i] = ws[i];
    }
}

// k = [v; -tr]: one thread per sample; A [w][B] keeps the units for the vector-Jacobian product.  DC: the state width when it is a
// compile-time constant (loops unrolled, the sample's vectors in registers), 0 = any width up to HYPER_MAX_D.
template <typename T, int DC>
__global__ void __launch_bounds__(256) hyper_forward_kernel(const float* __restrict__ theta, float tau16, int h, int w, int d_rt,
                                                             float* __restrict__ hyp, const T* __restrict__ Y, T* __restrict__ A,
                                                             T* __restrict__ k, T* __restrict__ k_l, int B) {
    constexpr int DM = DC > 0 ? DC : HYPER_MAX_D;
    const int d = DC > 0 ? DC : d_rt;
    extern __shared__ float sm[];                     // h1 [h], h2 [h], W [w][d], b [w], U [w][d], c [w]
    hyper_eval_block<T>(theta, tau16, h, w, d, sm, sm + h, sm + 2 * h, blockIdx.x == 0 ? hyp : nullptr);
    const float* W = sm + 2 * h;
    const float* bb = W + w * d;
    const float* U = bb + w;
    const float* c = U + w * d;
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    float z[DM], v[DM];
#pragma unroll
    for (int i = 0; i < DM; ++i) { z[i] = i < d ? Low<T>::to_f(Y[(long long)b * d + i]) : 0.f; v[i] = 0.f; }
    float tr = 0.f;
#pragma unroll 4
    for (int j = 0; j < w; ++j) {
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < DM; ++i)
            if (i < d) s = fmaf(W[j * d + i], z[i], s);
        const T aq = Low<T>::from_f(tanhf(s + bb[j]));
        A[(long long)j * B + b] = aq;
        const float a = Low<T>::to_f(aq);
#pragma unroll
        for (int i = 0; i < DM; ++i)
            if (i < d) v[i] = fmaf(U[j * d + i], a, v[i]);
        tr = fmaf(c[j], 1.f - a * a, tr);
    }
    const float inv_w = 1.f / (float)w;
#pragma unroll
    for (int i = 0; i < DM; ++i)
        if (i < d) k[(long long)b * d + i] = Low<T>::from_f(v[i] * inv_w);
    k_l[b] = Low<T>::from_f(-tr * inv_w);
}

// Per sample: the unit cotangents sbar_j = Q16(abar_j (1 - a_j^2)) into Sb [w][B], and psi = Q16(sum_j sbar_j W_j)
template <typename T, int DC>
__global__ void __launch_bounds__(256) hyper_unit_cot_kernel(const float* __restrict__ hyp, int h, int w, int d_rt, const T* __restrict__ A,
                                                              const T* __restrict__ kappa, const T* __restrict__ kappa_l, T* __restrict__ Sb,
                                                              T* __restrict__ psi, int B, unsigned* __restrict__ flag) {
    constexpr int DM = DC > 0 ? DC : HYPER_MAX_D;
    const int d = DC > 0 ? DC : d_rt;
    extern __shared__ float sm[];                     // W, b, U, c
    const int n = w * (2 * d + 1) + w;
    for (int i = threadIdx.x; i < n; i += blockDim.x) sm[i] = hyp[2 * h + i];
    __syncthreads();
    const float* W = sm;
    const float* U = sm + w * d + w;
    const float* c = U + w * d;
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    const bool on = b < B;
    float kz[DM], ps[DM];
#pragma unroll
    for (int i = 0; i < DM; ++i) { kz[i] = (on && i < d) ? Low<T>::to_f(kappa[(long long)b * d + i]) : 0.f; ps[i] = 0.f; }
    const float kl = on ? Low<T>::to_f(kappa_l[b]) : 0.f;
    const float inv_w = 1.f / (float)w;
    bool bad = false;
    if (on) {
#pragma unroll 4
        for (int j = 0; j < w; ++j) {
            const float a = Low<T>::to_f(A[(long long)j * B + b]);
            float ku = 0.f;
#pragma unroll
            for (int i = 0; i < DM; ++i)
                if (i < d) ku = fmaf(kz[i], U[j * d + i], ku);
            // l' = -tr: the trace's unit derivative -2 a c_j / w meets the cotangent -kappa_l
            const float abar = fmaf(kl * (2.f * inv_w) * c[j], a, ku * inv_w);
            const T sq = Low<T>::from_f(abar * (1.f - a * a));
            bad |= Low<T>::nonfinite(sq);
            Sb[(long long)j * B + b] = sq;
            const float sbar = Low<T>::to_f(sq);
#pragma unroll
            for (int i = 0; i < DM; ++i)
                if (i < d) ps[i] = fmaf(sbar, W[j * d + i], ps[i]);
        }
#pragma unroll
        for (int i = 0; i < DM; ++i)
            if (i < d) {
                const T pq = Low<T>::from_f(ps[i]);
                bad |= Low<T>::nonfinite(pq);
                psi[(long long)b * d + i] = pq;
            }
    }
    warp_flag_or(flag, bad);
}

// The batch sums of weight set j's cotangents, Wbar_j = sum_b sbar z, bbar_j = sum_b sbar, Ubar_j = sum_b a kappa_z / w,
// cbar_j = -sum_b kappa_l (1 - a^2) / w (samples strided over the threads, lanes by shuffles, warps in ascending order), by all
// threads of a block into out[2 d + 2] (and into the shared array `tot`, if given).  sm: [warps][2 d + 2] floats.
template <typename T>
__device__ void hyper_cot_sums(int j, int w, int d, const T* __restrict__ Y, const T* __restrict__ A, const T* __restrict__ Sb,
                               const T* __restrict__ kappa, const T* __restrict__ kappa_l, int B, float* __restrict__ out, float* sm,
                               float* tot = nullptr) {
    const int nv = 2 * d + 2;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float inv_w = 1.f / (float)w;
    float acc[2 * HYPER_MAX_D + 2];
#pragma unroll
    for (int q = 0; q < 2 * HYPER_MAX_D + 2; ++q) acc[q] = 0.f;
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        const float a = Low<T>::to_f(A[(long long)j * B + b]), sbar = Low<T>::to_f(Sb[(long long)j * B + b]);
        const float kl = Low<T>::to_f(kappa_l[b]);
#pragma unroll
        for (int i = 0; i < HYPER_MAX_D; ++i)
            if (i < d) {
                acc[i] = fmaf(sbar, Low<T>::to_f(Y[(long long)b * d + i]), acc[i]);
                acc[HYPER_MAX_D + 1 + i] = fmaf(a * inv_w, Low<T>::to_f(kappa[(long long)b * d + i]), acc[HYPER_MAX_D + 1 + i]);
            }
        acc[HYPER_MAX_D] += sbar;
        acc[2 * HYPER_MAX_D + 1] = fmaf(-kl * inv_w, 1.f - a * a, acc[2 * HYPER_MAX_D + 1]);
    }
    // registers are laid out for HYPER_MAX_D; the sums are stored densely: Wbar [d], bbar, Ubar [d], cbar
#pragma unroll
    for (int q = 0; q < 2 * HYPER_MAX_D + 2; ++q) {
        const bool used = q < HYPER_MAX_D ? q < d : (q == HYPER_MAX_D ? true : (q <= 2 * HYPER_MAX_D ? q - HYPER_MAX_D - 1 < d : true));
        if (used) {
            float x = acc[q];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            const int dense = q < HYPER_MAX_D ? q : (q == HYPER_MAX_D ? d : (q <= 2 * HYPER_MAX_D ? d + 1 + (q - HYPER_MAX_D - 1) : 2 * d + 1));
            if (lane == 0) sm[warp * nv + dense] = x;
        }
    }
    __syncthreads();
    if (threadIdx.x < nv) {
        float x = 0.f;
        for (int ww = 0; ww < (int)(blockDim.x >> 5); ++ww) x += sm[ww * nv + threadIdx.x];
        out[threadIdx.x] = x;
        if (tot != nullptr) tot[threadIdx.x] = x;
        __threadfence();
    }
    __syncthreads();
}

// One stage's parameter gradient from the batch sums of its w weight sets, by all threads of a block: the chain rule through
// c_j = U_j . W_j, the rounded cotangent of the hypernetwork's output, then the hypernetwork backwards:
// dg = (beta != 0 ? beta * dg : 0) + gradient of this stage.  Every entry of dg is written by the same thread for every stage.
// sm: obar [m], h2bar [h], h1bar [h], partial sums [max(256, h)].  Returns whether a rounded value was non-finite.
template <typename T>
__device__ bool hyper_backprop(const float* __restrict__ hyp, const float* __restrict__ theta, float tau16, int h, int w, int d,
                               const float* __restrict__ sums, float* __restrict__ dg, float beta, float* sm) {
    const int m = w * (2 * d + 1), nv = 2 * d + 2;
    const ThetaOffsets o = theta_offsets(h, m);
    float* obar = sm;
    float* h2bar = sm + m;
    float* h1bar = h2bar + h;
    float* psum = h1bar + h;
    const float* h1 = hyp;
    const float* h2 = hyp + h;
    const float* W = hyp + 2 * h;
    const float* U = W + w * d + w;
    bool bad = false;
    for (int jj = threadIdx.x; jj < w; jj += blockDim.x) {
        const float* s = sums + (long long)jj * nv;
        const float cbar = __ldcg(s + 2 * d + 1);
        for (int i = 0; i < d; ++i) {
            const float wb = q16<T>(fmaf(cbar, U[jj * d + i], __ldcg(s + i)));
            const float ub = q16<T>(fmaf(cbar, W[jj * d + i], __ldcg(s + d + 1 + i)));
            bad |= q_bad<T>(wb) | q_bad<T>(ub);
            obar[jj * d + i] = wb;
            obar[w * d + w + jj * d + i] = ub;
        }
        const float bq = q16<T>(__ldcg(s + d));
        bad |= q_bad<T>(bq);
        obar[w * d + jj] = bq;
    }
    __syncthreads();
    auto put = [&](int idx, float v) { dg[idx] = (beta != 0.f ? beta * dg[idx] : 0.f) + v; };
    for (int i = threadIdx.x; i < m * h; i += blockDim.x) put(o.A3 + i, obar[i / h] * h2[i % h]);
    for (int i = threadIdx.x; i < m; i += blockDim.x) put(o.c3 + i, obar[i]);
    {   // t[k] = sum_i A3[i][k] obar[i]: the block's threads take interleaved pieces of the sum over i, added in ascending order
        const int parts = h <= (int)blockDim.x ? (int)blockDim.x / h : 1;
        const int k = threadIdx.x % h, pc = threadIdx.x / h;
        if (pc < parts) {
            for (int k0 = k; k0 < h; k0 += (int)blockDim.x) {      // one pass unless h exceeds the block
                float t = 0.f;
#pragma unroll 4
                for (int i = pc; i < m; i += parts) t = fmaf(q16<T>(theta[o.A3 + i * h + k0]), obar[i], t);
                psum[pc * h + k0] = t;
            }
        }
        __syncthreads();
        for (int k0 = threadIdx.x; k0 < h; k0 += blockDim.x) {
            float t = 0.f;
            for (int q = 0; q < parts; ++q) t += psum[q * h + k0];
            const float v = q16<T>((1.f - h2[k0] * h2[k0]) * t);
            bad |= q_bad<T>(v);
            h2bar[k0] = v;
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < h * h; i += blockDim.x) put(o.A2 + i, h2bar[i / h] * h1[i % h]);
    for (int i = threadIdx.x; i < h; i += blockDim.x) put(o.c2 + i, h2bar[i]);
    for (int l = threadIdx.x; l < h; l += blockDim.x) {
        float t = 0.f;
        for (int k = 0; k < h; ++k) t = fmaf(q16<T>(theta[o.A2 + k * h + l]), h2bar[k], t);
        const float v = q16<T>((1.f - h1[l] * h1[l]) * t);
        bad |= q_bad<T>(v);
        h1bar[l] = v;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < h; i += blockDim.x) { put(o.A1 + i, h1bar[i] * tau16); put(o.c1 + i, h1bar[i]); }
    __syncthreads();
    return bad;
}

// Block j: the batch sums of weight set j into sums[j][2 d + 2].  The block that finishes last (a counter that it sets back to
// zero) runs the hypernetwork backwards.
template <typename T>
__global__ void __launch_bounds__(256) hyper_param_cot_kernel(const float* __restrict__ hyp, const float* __restrict__ theta, float tau16, int h,
                                                               int w, int d, const T* __restrict__ Y, const T* __restrict__ A,
                                                               const T* __restrict__ Sb, const T* __restrict__ kappa, const T* __restrict__ kappa_l,
                                                               float* __restrict__ sums, float* __restrict__ dg, float beta, int B,
                                                               unsigned* __restrict__ flag, unsigned* __restrict__ counter) {
    extern __shared__ float sm[];
    __shared__ bool last;
    const int j = blockIdx.x, nv = 2 * d + 2;
    hyper_cot_sums<T>(j, w, d, Y, A, Sb, kappa, kappa_l, B, sums + (long long)j * nv, sm);
    if (threadIdx.x == 0) last = atomicAdd(counter, 1u) == (unsigned)(gridDim.x - 1);
    __syncthreads();
    if (!last) return;
    __threadfence();
    const bool bad = hyper_backprop<T>(hyp, theta, tau16, h, w, d, sums, dg, beta, sm);
    warp_flag_or(flag, bad);
    if (threadIdx.x == 0) *counter = 0u;
}

// The same for all stages of a step, with the work of the chain rule spread out: block (stage, j) sums weight set j's cotangents,
// rounds its 2 d + 1 entries of the hypernetwork's output cotangent, writes their rows of the last layer's gradient and its part
// of the cotangent of h2; the block that finishes a stage last adds those parts (ascending j) and runs the two hidden layers
// backwards; stage gradients go to dgs[stage][p] (a launch of hyper_sum_stages_kernel then adds them into dg, last stage first).
// counters[stage]: blocks done, zero between launches.
template <typename T>
__global__ void __launch_bounds__(256) hyper_step_param_cot_kernel(const float* __restrict__ theta, RkStepScalars sc, int stages, int h, int w,
                                                                    int d, HyperStagePtrs ptr, const T* __restrict__ ybar,
                                                                    float* __restrict__ sums, float* __restrict__ tpart, float* __restrict__ dgs,
                                                                    long long p, int B, unsigned* __restrict__ flag,
                                                                    unsigned* __restrict__ counters) {
    extern __shared__ float sm[];                     // [8 warps][2 d + 2]; a stage's last block: partial sums [max(256, h)], h2bar [h], h1bar [h]
    __shared__ bool last_of_stage;
    __shared__ float tot[2 * HYPER_MAX_D + 2], ob[2 * HYPER_MAX_D + 1];
    __shared__ int ob_row[2 * HYPER_MAX_D + 1];
    const int stage = blockIdx.x / w, j = blockIdx.x % w, nv = 2 * d + 2, m = w * (2 * d + 1);
    hyper_cot_sums<T>(j, w, d, stage == 0 ? ybar : (const T*)ptr.y[stage], (const T*)ptr.A[stage], (const T*)ptr.sb[stage],
                      (const T*)ptr.kap[stage], (const T*)ptr.kapl[stage], B, sums + ((long long)stage * w + j) * nv, sm, tot);
    const ThetaOffsets o = theta_offsets(h, m);
    const float* hyp = ptr.hyp[stage];
    const float* h1 = hyp;
    const float* h2 = hyp + h;
    const float* W = hyp + 2 * h;
    const float* U = W + w * d + w;
    float* dgst = dgs + (long long)stage * p;
    bool bad = false;
    if ((int)threadIdx.x < 2 * d + 1) {               // the chain rule through c_j = U_j . W_j, then one rounding
        const int q = threadIdx.x;
        const float cbar = tot[2 * d + 1];
        float val;
        int row;
        if (q < d) { val = q16<T>(fmaf(cbar, U[j * d + q], tot[q])); row = j * d + q; }
        else if (q == d) { val = q16<T>(tot[d]); row = w * d + j; }
        else { val = q16<T>(fmaf(cbar, W[j * d + (q - d - 1)], tot[q])); row = w * d + w + j * d + (q - d - 1); }
        bad |= q_bad<T>(val);
        ob[q] = val;
        ob_row[q] = row;
        dgst[o.c3 + row] = val;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < (2 * d + 1) * h; idx += blockDim.x) dgst[o.A3 + ob_row[idx / h] * h + idx % h] = ob[idx / h] * h2[idx % h];
    for (int k = threadIdx.x; k < h; k += blockDim.x) {
        float t = 0.f;
        for (int q = 0; q < 2 * d + 1; ++q) t = fmaf(q16<T>(theta[o.A3 + ob_row[q] * h + k]), ob[q], t);
        tpart[((long long)stage * w + j) * h + k] = t;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last_of_stage = atomicAdd(counters + stage, 1u) == (unsigned)(w - 1);
    __syncthreads();
    if (last_of_stage) {
        __threadfence();
        float* psum = sm;
        float* h2bar = sm + (h > 256 ? h : 256);
        float* h1bar = h2bar + h;
        const float tau16 = sc.tau16[stage];
        {   // t[k] = sum_j tpart[j][k]: the threads take interleaved pieces of the sum over j, added in ascending order
            const int parts = h <= (int)blockDim.x ? (int)blockDim.x / h : 1;
            const int k = threadIdx.x % h, pc = threadIdx.x / h;
            if (pc < parts) {
                for (int k0 = k; k0 < h; k0 += (int)blockDim.x) {
                    float t = 0.f;
#pragma unroll 4
                    for (int jj = pc; jj < w; jj += parts) t += __ldcg(tpart + ((long long)stage * w + jj) * h + k0);
                    psum[pc * h + k0] = t;
                }
            }
            __syncthreads();
            for (int k0 = threadIdx.x; k0 < h; k0 += blockDim.x) {
                float t = 0.f;
                for (int q = 0; q < parts; ++q) t += psum[q * h + k0];
                const float v = q16<T>((1.f - h2[k0] * h2[k0]) * t);
                bad |= q_bad<T>(v);
                h2bar[k0] = v;
            }
        }
        __syncthreads();
        for (int i = threadIdx.x; i < h * h; i += blockDim.x) dgst[o.A2 + i] = h2bar[i / h] * h1[i % h];
        for (int i = threadIdx.x; i < h; i += blockDim.x) dgst[o.c2 + i] = h2bar[i];
        for (int l = threadIdx.x; l < h; l += blockDim.x) {
            float t = 0.f;
            for (int k = 0; k < h; ++k) t = fmaf(q16<T>(theta[o.A2 + k * h + l]), h2bar[k], t);
            const float v = q16<T>((1.f - h1[l] * h1[l]) * t);
            bad |= q_bad<T>(v);
            h1bar[l] = v;
        }
        __syncthreads();
        for (int i = threadIdx.x; i < h; i += blockDim.x) { dgst[o.A1 + i] = h1bar[i] * tau16; dgst[o.c1 + i] = h1bar[i]; }
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) counters[stage] = 0u;
    }
    warp_flag_or(flag, bad);
}

__global__ void __launch_bounds__(256) hyper_sum_stages_kernel(const float* __restrict__ dgs, int stages, long long p, float* __restrict__ dg) {
    const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (idx >= p) return;
    float x = 0.f + dgs[(long long)(stages - 1) * p + idx];
    for (int q = stages - 2; q >= 0; --q) x += dgs[(long long)q * p + idx];
    dg[idx] = x;
}

// ---------------------------------------------------------------- a whole Runge-Kutta step per launch
// The weight sets depend on the stage time alone, so one launch before the time loop evaluates the hypernetwork for every stage
// time of the solve: block (step, stage) writes h1, h2 and the weight sets into table[step][stage].
template <typename T>
__global__ void __launch_bounds__(256) hyper_table_kernel(const float* __restrict__ theta, const float* __restrict__ taus, int h, int w, int d,
                                                           float* __restrict__ table, long long stage_floats) {
    extern __shared__ float sm[];
    hyper_eval_block<T>(theta, taus[blockIdx.x], h, w, d, sm, sm + h, sm + 2 * h, table + (long long)blockIdx.x * stage_floats);
}

// Samples are independent and a sample's stage inputs need only its own stage derivatives, so one launch evaluates all stages of
// a step, and one launch forms all stage cotangents kappa_j = Q16(b_j v + sum_{l>j} h a_lj psi_l), unit cotangents and psi_j of
// the vector-Jacobian products, last stage first.  kHyperLanes threads share a sample: lane q takes the units q, q + kHyperLanes,
// ... and the lanes' partial sums meet in a butterfly of shuffles, which leaves the same bits in every lane.
constexpr int kHyperLanes = 8;
__device__ __forceinline__ float lanes_sum(float x) {
#pragma unroll
    for (int o = 1; o < kHyperLanes; o <<= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

template <typename T, int DC>
__global__ void __launch_bounds__(256) hyper_step_forward_kernel(RkStepScalars sc, int stages, int h, int w, int d_rt, HyperStagePtrs ptr,
                                                                  const T* __restrict__ ybar, int B) {
    constexpr int DM = DC > 0 ? DC : HYPER_MAX_D;
    const int d = DC > 0 ? DC : d_rt;
    extern __shared__ float sm[];                     // per stage W [w][d], b [w], U [w][d], c [w]
    const int set = w * (2 * d + 1) + w;
    for (int j = 0; j < stages; ++j)
        for (int i = threadIdx.x; i < set; i += blockDim.x) sm[j * set + i] = ptr.hyp[j][2 * h + i];
    __syncthreads();
    const int gt = blockIdx.x * blockDim.x + threadIdx.x;
    const int part = gt % kHyperLanes;
    const bool on = gt / kHyperLanes < B;
    const int b = on ? gt / kHyperLanes : B - 1;      // lanes past the batch compute along (the shuffles want whole warps), store nothing
    const bool writer = on && part == 0;
    float y0[DM], K[RK_MAX_STAGES][DM];
#pragma unroll
    for (int i = 0; i < DM; ++i) y0[i] = i < d ? Low<T>::to_f(ybar[(long long)b * d + i]) : 0.f;
    const float inv_w = 1.f / (float)w;
#pragma unroll
    for (int j = 0; j < RK_MAX_STAGES; ++j) {
        if (j < stages) {
            float z[DM];
#pragma unroll
            for (int i = 0; i < DM; ++i) {
                float acc = y0[i];
#pragma unroll
                for (int l = 0; l < RK_MAX_STAGES; ++l)
                    if (l < j && sc.a[j][l] != 0.f) acc = fmaf(sc.ha[j][l], K[l][i], acc);
                z[i] = j == 0 ? y0[i] : q16<T>(acc);
                if (j > 0 && i < d && writer) ((T*)ptr.y[j])[(long long)b * d + i] = Low<T>::from_f(z[i]);
            }
            const float* W = sm + j * set;
            const float* bb = W + w * d;
            const float* U = bb + w;
            const float* c = U + w * d;
            T* A = (T*)ptr.A[j];
            float v[DM];
#pragma unroll
            for (int i = 0; i < DM; ++i) v[i] = 0.f;
            float tr = 0.f;
#pragma unroll 4
            for (int u = part; u < w; u += kHyperLanes) {
                float sdot = 0.f;
#pragma unroll
                for (int i = 0; i < DM; ++i)
                    if (i < d) sdot = fmaf(W[u * d + i], z[i], sdot);
                const T aq = Low<T>::from_f(tanhf(sdot + bb[u]));
                if (on) A[(long long)u * B + b] = aq;
                const float a = Low<T>::to_f(aq);
#pragma unroll
                for (int i = 0; i < DM; ++i)
                    if (i < d) v[i] = fmaf(U[u * d + i], a, v[i]);
                tr = fmaf(c[u], 1.f - a * a, tr);
            }
#pragma unroll
            for (int i = 0; i < DM; ++i) {
                const T kq = Low<T>::from_f(lanes_sum(v[i]) * inv_w);
                K[j][i] = Low<T>::to_f(kq);
                if (i < d && writer) ((T*)ptr.k[j])[(long long)b * d + i] = kq;
            }
            tr = lanes_sum(tr);
            if (writer) ((T*)ptr.kl[j])[b] = Low<T>::from_f(-tr * inv_w);
        }
    }
}

template <typename T, int DC>
__global__ void __launch_bounds__(256) hyper_step_cot_kernel(RkStepScalars sc, int stages, int h, int w, int d_rt, HyperStagePtrs ptr,
                                                              const T* __restrict__ v, const T* __restrict__ v_l, int B,
                                                              unsigned* __restrict__ flag) {
    constexpr int DM = DC > 0 ? DC : HYPER_MAX_D;
    const int d = DC > 0 ? DC : d_rt;
    extern __shared__ float sm[];                     // per stage W, b, U, c
    const int set = w * (2 * d + 1) + w;
    for (int j = 0; j < stages; ++j)
        for (int i = threadIdx.x; i < set; i += blockDim.x) sm[j * set + i] = ptr.hyp[j][2 * h + i];
    __syncthreads();
    const int gt = blockIdx.x * blockDim.x + threadIdx.x;
    const int part = gt % kHyperLanes;
    const bool on = gt / kHyperLanes < B;
    const int b = on ? gt / kHyperLanes : B - 1;
    const bool writer = on && part == 0;
    bool bad = false;
    float vz[DM], psi[RK_MAX_STAGES][DM];
#pragma unroll
    for (int i = 0; i < DM; ++i) vz[i] = i < d ? Low<T>::to_f(v[(long long)b * d + i]) : 0.f;
    const float vl = Low<T>::to_f(v_l[b]);
    const float inv_w = 1.f / (float)w;
#pragma unroll
    for (int jr = 0; jr < RK_MAX_STAGES; ++jr) {
        const int j = stages - 1 - jr;
        if (j >= 0) {
            float kz[DM], ps[DM];
#pragma unroll
            for (int i = 0; i < DM; ++i) {
                float acc = sc.b[j] * vz[i];
#pragma unroll
                for (int l = 0; l < RK_MAX_STAGES; ++l)
                    if (l > j && l < stages && sc.a[l][j] != 0.f) acc = fmaf(sc.ha[l][j], psi[l][i], acc);
                const T kq = Low<T>::from_f(acc);
                if (i < d && writer) {
                    bad |= Low<T>::nonfinite(kq);
                    ((T*)ptr.kap[j])[(long long)b * d + i] = kq;
                }
                kz[i] = Low<T>::to_f(kq);
                ps[i] = 0.f;
            }
            const T klq = Low<T>::from_f(sc.b[j] * vl);
            if (writer) {
                bad |= Low<T>::nonfinite(klq);
                ((T*)ptr.kapl[j])[b] = klq;
            }
            const float kl = Low<T>::to_f(klq);
            const float* W = sm + j * set;
            const float* U = W + w * d + w;
            const float* c = U + w * d;
            const T* A = (const T*)ptr.A[j];
            T* Sb = (T*)ptr.sb[j];
#pragma unroll 8
            for (int u = part; u < w; u += kHyperLanes) {
                const float a = Low<T>::to_f(A[(long long)u * B + b]);
                float ku = 0.f;
#pragma unroll
                for (int i = 0; i < DM; ++i)
                    if (i < d) ku = fmaf(kz[i], U[u * d + i], ku);
                const float abar = fmaf(kl * (2.f * inv_w) * c[u], a, ku * inv_w);
                const T sq = Low<T>::from_f(abar * (1.f - a * a));
                if (on) {
                    bad |= Low<T>::nonfinite(sq);
                    Sb[(long long)u * B + b] = sq;
                }
                const float sbar = Low<T>::to_f(sq);
#pragma unroll
                for (int i = 0; i < DM; ++i)
                    if (i < d) ps[i] = fmaf(sbar, W[u * d + i], ps[i]);
            }
#pragma unroll
            for (int i = 0; i < DM; ++i) {
                const T pq = Low<T>::from_f(lanes_sum(ps[i]));
                psi[j][i] = Low<T>::to_f(pq);
                if (i < d && writer) {
                    bad |= Low<T>::nonfinite(pq);
                    ((T*)ptr.psi[j])[(long long)b * d + i] = pq;
                }
            }
        }
    }
    warp_flag_or(flag, bad);
}

}  // namespace

size_t hyper_param_count(int h, int w, int d) {
    const int m = w * (2 * d + 1);
    return (size_t)3 * h + (size_t)h * h + (size_t)m * h + m;
}
size_t hyper_stage_floats(int h, int w, int d) { return (size_t)2 * h + (size_t)w * (2 * d + 1) + w; }
size_t hyper_scratch_floats(int w, int d) { return (size_t)w * (2 * d + 2); }
size_t hyper_step_scratch_floats(int h, int w, int d) {
    return (size_t)RK_MAX_STAGES * ((size_t)w * (2 * d + 2) + (size_t)w * h + hyper_param_count(h, w, d));
}
bool hyper_shape_ok(int h, int w, int d) {
    // the hypernetwork and the weight sets of one stage time live in shared memory
    const size_t fwd = ((size_t)2 * h + (size_t)w * (2 * d + 1) + w) * sizeof(float);
    const size_t fin = ((size_t)w * (2 * d + 1) + 2 * h + (h > 256 ? h : 256)) * sizeof(float);
    return d >= 1 && d <= HYPER_MAX_D && h >= 1 && w >= 1 && fwd <= 48 * 1024 && fin <= 48 * 1024;
}

void launch_hyper_forward(mpode_dtype dt, const float* theta, float tau16, int h, int w, int d, float* hyp, const void* Y, void* A, void* k,
                          void* k_l, int B, cudaStream_t st, long long* launches) {
    const size_t smem = ((size_t)2 * h + (size_t)w * (2 * d + 1) + w) * sizeof(float);
    const int blocks = (B + 255) / 256;
    if (d == 2) {
        MPODE_DISPATCH_T(dt, T, (hyper_forward_kernel<T, 2><<<blocks, 256, smem, st>>>(theta, tau16, h, w, d, hyp, (const T*)Y, (T*)A, (T*)k, (T*)k_l, B)));
    } else {
        MPODE_DISPATCH_T(dt, T, (hyper_forward_kernel<T, 0><<<blocks, 256, smem, st>>>(theta, tau16, h, w, d, hyp, (const T*)Y, (T*)A, (T*)k, (T*)k_l, B)));
    }
    if (launches) ++*launches;
}

void launch_hyper_vjp(mpode_dtype dt, const float* theta, float tau16, int h, int w, int d, const float* hyp, const void* Y, const void* A,
                      void* Sb, const void* kappa, const void* kappa_l, void* psi, float* sums, float* dg, float beta, int B, unsigned* flag,
                      unsigned* counter, cudaStream_t st, long long* launches) {
    const int blocks = (B + 255) / 256, nv = 2 * d + 2, m = w * (2 * d + 1);
    const size_t sm_unit = ((size_t)w * (2 * d + 1) + w) * sizeof(float);
    size_t sm_par = ((size_t)m + 2 * h + (h > 256 ? h : 256)) * sizeof(float);
    if (sm_par < (size_t)8 * nv * sizeof(float)) sm_par = (size_t)8 * nv * sizeof(float);
    if (d == 2) {
        MPODE_DISPATCH_T(dt, T, (hyper_unit_cot_kernel<T, 2><<<blocks, 256, sm_unit, st>>>(hyp, h, w, d, (const T*)A, (const T*)kappa, (const T*)kappa_l,
                                                                                           (T*)Sb, (T*)psi, B, flag)));
    } else {
        MPODE_DISPATCH_T(dt, T, (hyper_unit_cot_kernel<T, 0><<<blocks, 256, sm_unit, st>>>(hyp, h, w, d, (const T*)A, (const T*)kappa, (const T*)kappa_l,
                                                                                           (T*)Sb, (T*)psi, B, flag)));
    }
    if (launches) ++*launches;
    MPODE_DISPATCH_T(dt, T, (hyper_param_cot_kernel<T><<<w, 256, sm_par, st>>>(hyp, theta, tau16, h, w, d, (const T*)Y, (const T*)A, (const T*)Sb,
                                                                               (const T*)kappa, (const T*)kappa_l, sums, dg, beta, B, flag, counter)));
    if (launches) ++*launches;
}

bool hyper_step_shape_ok(int h, int w, int d, int stages) {
    const size_t set = (size_t)w * (2 * d + 1) + w;
    return hyper_shape_ok(h, w, d) && stages >= 1 && stages <= RK_MAX_STAGES && stages * set * sizeof(float) <= 48 * 1024;
}

void launch_hyper_table(mpode_dtype dt, const float* theta, const float* taus, int count, int h, int w, int d, float* table, cudaStream_t st,
                        long long* launches) {
    const size_t smem = ((size_t)2 * h + (size_t)w * (2 * d + 1) + w) * sizeof(float);
    MPODE_DISPATCH_T(dt, T, (hyper_table_kernel<T><<<count, 256, smem, st>>>(theta, taus, h, w, d, table, (long long)hyper_stage_floats(h, w, d))));
    if (launches) ++*launches;
}

void launch_hyper_step_forward(mpode_dtype dt, const RkStepScalars& sc, int stages, int h, int w, int d,
                               const HyperStagePtrs& ptr, const void* ybar, int B, cudaStream_t st, long long* launches) {
    const size_t smem = (size_t)stages * ((size_t)w * (2 * d + 1) + w) * sizeof(float);
    const int blocks = (int)(((long long)B * kHyperLanes + 255) / 256);
    if (d == 2) {
        MPODE_DISPATCH_T(dt, T, (hyper_step_forward_kernel<T, 2><<<blocks, 256, smem, st>>>(sc, stages, h, w, d, ptr, (const T*)ybar, B)));
    } else {
        MPODE_DISPATCH_T(dt, T, (hyper_step_forward_kernel<T, 0><<<blocks, 256, smem, st>>>(sc, stages, h, w, d, ptr, (const T*)ybar, B)));
    }
    if (launches) ++*launches;
}

void launch_hyper_step_vjp(mpode_dtype dt, const float* theta, const RkStepScalars& sc, int stages, int h, int w, int d,
                           const HyperStagePtrs& ptr, const void* ybar, const void* v, const void* v_l, float* scratch, float* dg, int B,
                           unsigned* flag, unsigned* counters, cudaStream_t st, long long* launches) {
    const int blocks = (int)(((long long)B * kHyperLanes + 255) / 256), nv = 2 * d + 2;
    const size_t sm_unit = (size_t)stages * ((size_t)w * (2 * d + 1) + w) * sizeof(float);
    size_t sm_par = ((size_t)2 * h + (h > 256 ? h : 256)) * sizeof(float);
    if (sm_par < (size_t)8 * nv * sizeof(float)) sm_par = (size_t)8 * nv * sizeof(float);
    const long long p = (long long)hyper_param_count(h, w, d);
    float* sums = scratch;                                         // [stages][w][2 d + 2]
    float* tpart = sums + (size_t)RK_MAX_STAGES * w * nv;          // [stages][w][h]
    float* dgs = tpart + (size_t)RK_MAX_STAGES * w * h;            // [stages][p]
    if (d == 2) {
        MPODE_DISPATCH_T(dt, T, (hyper_step_cot_kernel<T, 2><<<blocks, 256, sm_unit, st>>>(sc, stages, h, w, d, ptr, (const T*)v, (const T*)v_l, B, flag)));
    } else {
        MPODE_DISPATCH_T(dt, T, (hyper_step_cot_kernel<T, 0><<<blocks, 256, sm_unit, st>>>(sc, stages, h, w, d, ptr, (const T*)v, (const T*)v_l, B, flag)));
    }
    if (launches) ++*launches;
    MPODE_DISPATCH_T(dt, T, (hyper_step_param_cot_kernel<T><<<stages * w, 256, sm_par, st>>>(theta, sc, stages, h, w, d, ptr, (const T*)ybar, sums, tpart,
                                                                                             dgs, p, B, flag, counters)));
    if (launches) ++*launches;
    hyper_sum_stages_kernel<<<(unsigned)((p + 255) / 256), 256, 0, st>>>(dgs, stages, p, dg);
    if (launches) ++*launches;
}


}  // namespace mpode
