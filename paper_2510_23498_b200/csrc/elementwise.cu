// Memory-bound pieces of Alg. 1 and Alg. 2: parameter quantisation, stage combinations, state update and
// trajectory store, adjoint seed / commit, infinity norms and the non-finite flag.  128-bit vectorised,
// grid-stride, grid sized as a multiple of the SM count.
#include "common.cuh"

namespace mpode {

namespace {

constexpr int kThreads = 256;
constexpr int kSMs = 148;

template <typename T, int V> struct alignas(sizeof(T) * V) Pack { T v[V]; };

inline int grid_for(long long work_items) {
    long long b = (work_items + kThreads - 1) / kThreads;
    long long cap = (long long)kSMs * 8;
    if (b < 1) b = 1;
    return (int)(b < cap ? b : cap);
}
inline bool aligned_to(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

#define MPODE_DISPATCH_T(dt, T, ...)                                         \
    do {                                                                     \
        if ((dt) == MPODE_BF16) { using T = __nv_bfloat16; __VA_ARGS__; }    \
        else if ((dt) == MPODE_F16) { using T = __half; __VA_ARGS__; }       \
        else { using T = float; __VA_ARGS__; }                               \
    } while (0)

// ---------------------------------------------------------------- theta -> Q16(theta) (Alg. 1, Alg. 2: weights in low precision)
// src: fp32 [rows, src_ld] (only the first `cols` columns are taken); dst: low [rows, cols]; dst_t: low [cols, rows].
template <typename T>
__global__ void quantize_matrix_kernel(const float* __restrict__ src, long long src_ld, int rows, int cols,
                                       T* __restrict__ dst, T* __restrict__ dst_t) {
    __shared__ float tile[32][33];
    int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    for (int i = threadIdx.y; i < 32; i += blockDim.y) {
        int r = r0 + i, c = c0 + threadIdx.x;
        float v = (r < rows && c < cols) ? src[(long long)r * src_ld + c] : 0.f;
        tile[i][threadIdx.x] = v;
        if (dst != nullptr && r < rows && c < cols) dst[(long long)r * cols + c] = Low<T>::from_f(v);
    }
    __syncthreads();
    if (dst_t != nullptr) {
        for (int i = threadIdx.y; i < 32; i += blockDim.y) {
            int c = c0 + i, r = r0 + threadIdx.x;
            if (r < rows && c < cols) dst_t[(long long)c * rows + r] = Low<T>::from_f(tile[threadIdx.x][i]);
        }
    }
}

// Conv weights: src fp32 [cout][9][cin_total]; dst low [cout][9][cin_keep] (first cin_keep channels);
// dst_flip_t low [cin_keep][9][cout] with the taps reversed (the operand of the input-gradient convolution).
template <typename T>
__global__ void quantize_conv_weights_kernel(const float* __restrict__ src, int cout, int cin_total, int cin_keep,
                                             T* __restrict__ dst, T* __restrict__ dst_flip_t, float sign) {
    long long n = (long long)cout * 9 * cin_keep;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        int c = (int)(i % cin_keep);
        int tap = (int)((i / cin_keep) % 9);
        int o = (int)(i / ((long long)cin_keep * 9));
        T v = Low<T>::from_f(sign * src[((long long)o * 9 + tap) * cin_total + c]);      // Q16(-w) = -Q16(w)
        if (dst != nullptr) dst[i] = v;
        if (dst_flip_t != nullptr) dst_flip_t[((long long)c * 9 + (8 - tap)) * cout + o] = v;
    }
}

// Per position class of a 3x3 convolution with zero padding (3 * row class + column class; 0 first, 1 interior, 2
// last row / column): out[cls][cout] = b[cout] + tau * sum over the taps that fall inside the image of the weight of
// the appended time channel (the last of cin_total input channels); w = null gives the bias alone.
template <typename T>
__global__ void conv_class_bias_kernel(const T* __restrict__ b, const T* __restrict__ w, int cin_total, float tau, int C,
                                       float* __restrict__ out) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 9 * C) return;
    int cls = i / C, co = i - cls * C, ry = cls / 3, rx = cls - ry * 3;
    float s = 0.f;
    if (w != nullptr) {
        for (int tap = 0; tap < 9; ++tap) {
            int dy = tap / 3 - 1, dx = tap % 3 - 1;
            if ((ry == 0 && dy < 0) || (ry == 2 && dy > 0) || (rx == 0 && dx < 0) || (rx == 2 && dx > 0)) continue;
            s += Low<T>::to_f(w[((long long)co * 9 + tap) * cin_total + cin_total - 1]);
        }
    }
    out[i] = fmaf(tau, s, b != nullptr ? Low<T>::to_f(b[co]) : 0.f);
}

// Slices of the transposed convolution weight gradient summed in ascending order into the [cout][tap][ct] layout.  The slices
// are [tap * C + cin][cout] (cout contiguous), the destination has cin contiguous: a block moves a 32 x 32 (cin, cout) piece of one
// tap through shared memory so that both sides are read and written in whole 128-byte lines.  C is a multiple of 32.
__global__ void __launch_bounds__(256) conv_wgrad_reduce_kernel(const float* __restrict__ partial, int S, int C, int ct, float* __restrict__ out,
                                                                 float beta, float sign) {
    __shared__ float tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int cin0 = blockIdx.x * 32, co0 = blockIdx.y * 32, tap = blockIdx.z;
    const long long n_el = (long long)9 * C * C;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int cin = cin0 + ty + 8 * r;
        const long long i = ((long long)tap * C + cin) * C + co0 + tx;
        float s = 0.f;
        for (int z = 0; z < S; ++z) s += partial[(long long)z * n_el + i];
        tile[ty + 8 * r][tx] = s;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int co = co0 + ty + 8 * r;
        float* o = out + ((long long)co * 9 + tap) * ct + cin0 + tx;
        *o = (beta != 0.f ? *o : 0.f) + sign * tile[tx][ty + 8 * r];
    }
}

// Sums of dZ[p][cout] over the pixels of each position class (3 * row class + column class), per block of pixels.
// A thread owns 8 consecutive channels (one 16-byte load per pixel) and every `lanes`-th pixel of the block's range, and keeps
// nine sums in registers: all its pixels, those of the first / last row, of the first / last column, and of the four corners
// (the border ones are touched for border pixels only).  The nine class sums follow by inclusion and exclusion.
template <typename T>
__global__ void __launch_bounds__(128, 4) conv_class_sums_kernel(const T* __restrict__ dz, long long pixels, int H, int W, int C,
                                                                long long per_block, float* __restrict__ part) {
    extern __shared__ float sm[];                    // [9 * 8][128]: value (class, e) of every thread
    const int groups = C / 8;                        // threads per pixel
    const int cg = threadIdx.x % groups, pl = threadIdx.x / groups, lanes = blockDim.x / groups;
    const long long p0 = blockIdx.x * per_block, p1 = min(pixels, p0 + per_block);
    enum { ALL, TOP, BOT, LEFT, RIGHT, TL, TR, BL, BR };
    float acc[9][8];
#pragma unroll
    for (int k = 0; k < 9; ++k)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[k][e] = 0.f;
    if (pl < lanes && p0 + pl < p1) {
        int x = (int)((p0 + pl) % W), y = (int)(((p0 + pl) / W) % H);
        // four pixels per trip, their loads issued together: the kernel lives on bytes in flight
        for (long long p = p0 + pl; p < p1; p += 4 * lanes) {
            Pack<T, 8> v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const long long pp = p + (long long)u * lanes;
                if (pp < p1) v[u] = *reinterpret_cast<const Pack<T, 8>*>(dz + pp * C + cg * 8);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (p + (long long)u * lanes < p1) {
                    float f[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) { f[e] = Low<T>::to_f(v[u].v[e]); acc[ALL][e] += f[e]; }
                    const bool top = y == 0, bot = y == H - 1, left = x == 0, right = x == W - 1;
                    if (top | bot | left | right) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            if (top) acc[TOP][e] += f[e];
                            if (bot) acc[BOT][e] += f[e];
                            if (left) acc[LEFT][e] += f[e];
                            if (right) acc[RIGHT][e] += f[e];
                            if (top & left) acc[TL][e] += f[e];
                            if (top & right) acc[TR][e] += f[e];
                            if (bot & left) acc[BL][e] += f[e];
                            if (bot & right) acc[BR][e] += f[e];
                        }
                    }
                }
                x += lanes;                           // the next pixel of this thread
                while (x >= W) { x -= W; y = y + 1 == H ? 0 : y + 1; }
            }
        }
    }
    // class = 3 * (row: first, inner, last) + (column: first, inner, last); H = 1 or W = 1 make first = last, where the
    // overlap terms below count a pixel in both, as the convolution's zero padding does on both sides
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const float all = acc[ALL][e], t = acc[TOP][e], b = acc[BOT][e], l = acc[LEFT][e], r = acc[RIGHT][e];
        const float tl = acc[TL][e], tr = acc[TR][e], bl = acc[BL][e], br = acc[BR][e];
        float cls[9];
        cls[0] = tl;            cls[1] = t - tl - tr;                              cls[2] = tr;
        cls[3] = l - tl - bl;   cls[4] = all - t - b - l - r + tl + tr + bl + br;  cls[5] = r - tr - br;
        cls[6] = bl;            cls[7] = b - bl - br;                              cls[8] = br;
#pragma unroll
        for (int k = 0; k < 9; ++k) sm[(k * 8 + e) * 128 + threadIdx.x] = cls[k];
    }
    __syncthreads();
    for (int j = threadIdx.x; j < 72 * groups; j += blockDim.x) {
        const int ke = j / groups, g = j - ke * groups;
        float s = 0.f;
        for (int l = 0; l < lanes; ++l) s += sm[ke * 128 + l * groups + g];
        part[(long long)blockIdx.x * 9 * C + (ke >> 3) * C + g * 8 + (ke & 7)] = s;
    }
}
// From the class sums: the bias gradient (sum over all classes) and, for a layer with an appended time channel, the
// gradient of that channel's weights per tap (tau times the sum over the classes in which the tap is inside the image).
// One warp per (class, channel): the per-block sums added by the lanes in a fixed order, then a fixed shuffle tree
__global__ void conv_class_reduce_kernel(const float* __restrict__ part, int blocks, int n, float* __restrict__ cs) {
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (i >= n) return;
    float s = 0.f;
    for (int b = lane; b < blocks; b += 32) s += part[(long long)b * n + i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) cs[i] = s;
}
__global__ void conv_class_final_kernel(const float* __restrict__ cs_in, int C, int ct, float tau, float* __restrict__ wt_out,
                                        float* __restrict__ bias_out, float beta) {
    extern __shared__ float cs[];                    // [9][C] class sums
    for (int i = threadIdx.x; i < 9 * C; i += blockDim.x) cs[i] = cs_in[i];
    __syncthreads();
    conv_class_finish(cs, C, ct, tau, wt_out, bias_out, beta);
}

// ---------------------------------------------------------------- Alg. 1 initialisation: y <- Q32(x), traj[0] = Q16(y)
template <typename T, int V>
__global__ void init_state_kernel(const float* __restrict__ y0, float* __restrict__ y, T* __restrict__ traj0, int B,
                                  int d, int D) {
    long long nv = (long long)B * (d / V);
    int dv = d / V;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < nv; i += (long long)gridDim.x * blockDim.x) {
        long long row = i / dv;
        int col = (int)(i % dv) * V;
        Pack<float, V> in = *reinterpret_cast<const Pack<float, V>*>(y0 + row * d + col);
        Pack<T, V> q;
#pragma unroll
        for (int k = 0; k < V; ++k) q.v[k] = Low<T>::from_f(in.v[k]);
        *reinterpret_cast<Pack<float, V>*>(y + row * D + col) = in;
        *reinterpret_cast<Pack<T, V>*>(traj0 + row * d + col) = q;
    }
    if (D > d) {  // CNF: the log-density column starts at zero
        for (long long r = blockIdx.x * (long long)blockDim.x + threadIdx.x; r < B; r += (long long)gridDim.x * blockDim.x)
            for (int c = d; c < D; ++c) y[r * D + c] = 0.f;
    }
}

// ---------------------------------------------------------------- stage input Y_j = Q16(ybar + sum_l (h a_jl) k_l)
template <typename T, int V>
__global__ void stage_input_kernel(const T* __restrict__ base, Terms t, T* __restrict__ out, long long nv) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < nv; i += (long long)gridDim.x * blockDim.x) {
        Pack<T, V> b = reinterpret_cast<const Pack<T, V>*>(base)[i];
        float acc[V];
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] = Low<T>::to_f(b.v[k]);
        for (int l = 0; l < t.n; ++l) {
            Pack<T, V> kk = reinterpret_cast<const Pack<T, V>*>(t.p[l])[i];
#pragma unroll
            for (int k = 0; k < V; ++k) acc[k] = fmaf(t.c[l], Low<T>::to_f(kk.v[k]), acc[k]);
        }
        Pack<T, V> o;
#pragma unroll
        for (int k = 0; k < V; ++k) o.v[k] = Low<T>::from_f(acc[k]);
        reinterpret_cast<Pack<T, V>*>(out)[i] = o;
    }
}

// ---------------------------------------------------------------- Alg. 1 accumulate and store: y += h Phi (fp32), traj[i+1] = Q16(y)
template <typename T, int V>
__global__ void final_combine_kernel(float* __restrict__ y, Terms t, T* __restrict__ traj_next, int B, int d, int D,
                                     int round_increment, float h) {
    int dv = d / V;
    long long nv = (long long)B * dv;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < nv; i += (long long)gridDim.x * blockDim.x) {
        long long row = i / dv;
        int col = (int)(i % dv) * V;
        float acc[V];
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] = 0.f;
        for (int l = 0; l < t.n; ++l) {
            Pack<T, V> kk = *reinterpret_cast<const Pack<T, V>*>((const T*)t.p[l] + row * d + col);
#pragma unroll
            for (int k = 0; k < V; ++k) acc[k] = fmaf(t.c[l], Low<T>::to_f(kk.v[k]), acc[k]);
        }
        Pack<float, V> yy = *reinterpret_cast<Pack<float, V>*>(y + row * D + col);
        Pack<T, V> q;
#pragma unroll
        for (int k = 0; k < V; ++k) {
            float inc = round_increment ? h * Low<T>::to_f(Low<T>::from_f(acc[k])) : acc[k];
            yy.v[k] = yy.v[k] + inc;
            q.v[k] = Low<T>::from_f(yy.v[k]);
        }
        *reinterpret_cast<Pack<float, V>*>(y + row * D + col) = yy;
        *reinterpret_cast<Pack<T, V>*>(traj_next + row * d + col) = q;
    }
}

// One extra column of the wide state (the CNF log-density): y[:, col] += sum_j c_j k_j[b]
template <typename T>
__global__ void column_combine_kernel(float* __restrict__ y, int D, int col, Terms t, int B, int round_increment,
                                      float h) {
    for (long long r = blockIdx.x * (long long)blockDim.x + threadIdx.x; r < B; r += (long long)gridDim.x * blockDim.x) {
        float acc = 0.f;
        for (int l = 0; l < t.n; ++l) acc = fmaf(t.c[l], Low<T>::to_f(((const T*)t.p[l])[r]), acc);
        float inc = round_increment ? h * Low<T>::to_f(Low<T>::from_f(acc)) : acc;
        y[r * D + col] += inc;
    }
}

// ---------------------------------------------------------------- infinity norm (order independent) + non-finite flag
__device__ __forceinline__ void block_amax_commit(float m, bool bad, float* amax, unsigned* flag) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    __shared__ float sm[kThreads / 32];
    int w = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) sm[w] = m;
    warp_flag_or(flag, bad);
    __syncthreads();
    if (threadIdx.x == 0) {
        float mm = sm[0];
        for (int i = 1; i < (int)(blockDim.x >> 5); ++i) mm = fmaxf(mm, sm[i]);
        // non-negative floats order like their bit patterns
        if (amax != nullptr) atomicMax(reinterpret_cast<unsigned*>(amax), __float_as_uint(mm));
    }
}

__global__ void copy_amax_kernel(const float* __restrict__ src, float* __restrict__ dst, long long n,
                                 float* __restrict__ amax, unsigned* __restrict__ flag) {
    float m = 0.f;
    bool bad = false;
    const long long stride = (long long)gridDim.x * blockDim.x, tid = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if ((((uintptr_t)src | (uintptr_t)dst) & 15) == 0) {      // 16-byte pieces, then the tail
        const long long n4 = n / 4;
        for (long long i = tid; i < n4; i += stride) {
            const float4 v = reinterpret_cast<const float4*>(src)[i];
            if (dst != nullptr) reinterpret_cast<float4*>(dst)[i] = v;
            bad |= Low<float>::nonfinite(v.x) | Low<float>::nonfinite(v.y) | Low<float>::nonfinite(v.z) | Low<float>::nonfinite(v.w);
            m = fmaxf(fmaxf(m, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
        }
        for (long long i = n4 * 4 + tid; i < n; i += stride) {
            const float v = src[i];
            if (dst != nullptr) dst[i] = v;
            bad |= Low<float>::nonfinite(v);
            m = fmaxf(m, fabsf(v));
        }
    } else {
        for (long long i = tid; i < n; i += stride) {
            const float v = src[i];
            if (dst != nullptr) dst[i] = v;
            bad |= Low<float>::nonfinite(v);
            m = fmaxf(m, fabsf(v));
        }
    }
    block_amax_commit(m, bad, amax, flag);
}

// ---------------------------------------------------------------- Eq. (vjp) seed: v = Q16(S a), S = 2^e
template <typename T, int V>
__global__ void seed_kernel(const float* __restrict__ a, int e, T* __restrict__ v, T* __restrict__ v_l, int B, int d,
                            int D, unsigned* __restrict__ flag, T* __restrict__ kap, float bk, const int* __restrict__ e_dev) {
    if (e_dev != nullptr) e = *e_dev;               // the exponent lives on the device (dynamic scaling)
    int dv = d / V;
    long long nv = (long long)B * dv;
    bool bad = false;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < nv; i += (long long)gridDim.x * blockDim.x) {
        long long row = i / dv;
        int col = (int)(i % dv) * V;
        Pack<float, V> aa = *reinterpret_cast<const Pack<float, V>*>(a + row * D + col);
        Pack<T, V> q;
#pragma unroll
        for (int k = 0; k < V; ++k) {
            q.v[k] = Low<T>::from_f(ldexpf(aa.v[k], e));
            bad |= Low<T>::nonfinite(q.v[k]);
        }
        *reinterpret_cast<Pack<T, V>*>(v + row * d + col) = q;
        if (kap != nullptr) {   // cotangent of the last stage, kappa_s = Q16(b_s v), for the fused backward kernel
            Pack<T, V> kq;
#pragma unroll
            for (int k = 0; k < V; ++k) {
                kq.v[k] = Low<T>::from_f(bk * Low<T>::to_f(q.v[k]));
                bad |= Low<T>::nonfinite(kq.v[k]);
            }
            *reinterpret_cast<Pack<T, V>*>(kap + row * d + col) = kq;
        }
    }
    if (D > d) {
        for (long long r = blockIdx.x * (long long)blockDim.x + threadIdx.x; r < B; r += (long long)gridDim.x * blockDim.x) {
            T q = Low<T>::from_f(ldexpf(a[r * D + d], e));
            bad |= Low<T>::nonfinite(q);
            v_l[r] = q;
        }
    }
    warp_flag_or(flag, bad);
}

// ---------------------------------------------------------------- kappa_j = Q16(b_j v + sum_{l>j} (h a_lj) psi_l)
template <typename T, int V>
__global__ void kappa_kernel(const T* __restrict__ v, float bj, Terms t, T* __restrict__ out, long long nv,
                             unsigned* __restrict__ flag) {
    bool bad = false;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < nv; i += (long long)gridDim.x * blockDim.x) {
        Pack<T, V> vv = reinterpret_cast<const Pack<T, V>*>(v)[i];
        float acc[V];
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] = bj * Low<T>::to_f(vv.v[k]);
        for (int l = 0; l < t.n; ++l) {
            Pack<T, V> pp = reinterpret_cast<const Pack<T, V>*>(t.p[l])[i];
#pragma unroll
            for (int k = 0; k < V; ++k) acc[k] = fmaf(t.c[l], Low<T>::to_f(pp.v[k]), acc[k]);
        }
        Pack<T, V> o;
#pragma unroll
        for (int k = 0; k < V; ++k) {
            o.v[k] = Low<T>::from_f(acc[k]);
            bad |= Low<T>::nonfinite(o.v[k]);
        }
        reinterpret_cast<Pack<T, V>*>(out)[i] = o;
    }
    warp_flag_or(flag, bad);
}

// ---------------------------------------------------------------- Alg. 2 adjoint update: a <- a + (h / S) sum_j psi_j, and ||a||_inf
template <typename T, int V>
__global__ void commit_a_kernel(float* __restrict__ a, Terms psis, float coef, int B, int d, int D,
                                float* __restrict__ amax, const unsigned* __restrict__ skip_if_set, const float* __restrict__ add,
                                const int* __restrict__ e_dev) {
    if (skip_if_set != nullptr && *skip_if_set != 0u) return;   // a non-finite attempt is not committed (it is repeated)
    if (e_dev != nullptr) coef = ldexpf(coef, -*e_dev);         // h / S with the device's exponent: exact
    int dv = d / V;
    long long nv = (long long)B * dv;
    float m = 0.f;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < nv; i += (long long)gridDim.x * blockDim.x) {
        long long row = i / dv;
        int col = (int)(i % dv) * V;
        float da[V];
#pragma unroll
        for (int k = 0; k < V; ++k) da[k] = 0.f;
        for (int l = 0; l < psis.n; ++l) {
            Pack<T, V> pp = *reinterpret_cast<const Pack<T, V>*>((const T*)psis.p[l] + row * d + col);
#pragma unroll
            for (int k = 0; k < V; ++k) da[k] += Low<T>::to_f(pp.v[k]);
        }
        Pack<float, V> aa = *reinterpret_cast<Pack<float, V>*>(a + row * D + col);
#pragma unroll
        for (int k = 0; k < V; ++k) aa.v[k] = fmaf(coef, da[k], aa.v[k]);
        if (add != nullptr) {
            const Pack<float, V> ad = *reinterpret_cast<const Pack<float, V>*>(add + row * D + col);
#pragma unroll
            for (int k = 0; k < V; ++k) aa.v[k] += ad.v[k];
        }
#pragma unroll
        for (int k = 0; k < V; ++k) m = fmaxf(m, fabsf(aa.v[k]));
        *reinterpret_cast<Pack<float, V>*>(a + row * D + col) = aa;
    }
    if (D > d) {
        for (long long r = blockIdx.x * (long long)blockDim.x + threadIdx.x; r < B; r += (long long)gridDim.x * blockDim.x)
            for (int c = d; c < D; ++c) {
                if (add != nullptr) a[r * D + c] += add[r * D + c];
                m = fmaxf(m, fabsf(a[r * D + c]));
            }
    }
    block_amax_commit(m, false, amax, nullptr);
}

// Alg. 2 gradient update: g <- g + (h / S) dg
__global__ void commit_g_kernel(float* __restrict__ g, const float* __restrict__ dg, float coef, long long p,
                                const unsigned* __restrict__ skip_if_set, const int* __restrict__ e_dev) {
    if (skip_if_set != nullptr && *skip_if_set != 0u) return;
    if (e_dev != nullptr) coef = ldexpf(coef, -*e_dev);
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < p; i += (long long)gridDim.x * blockDim.x)
        g[i] = fmaf(coef, dg[i], g[i]);
}

// Alg. 2 finiteness test for the parameter gradient: is Q16(dg) finite?
template <typename T>
__global__ void check_as_low_kernel(const float* __restrict__ x, long long n, unsigned* __restrict__ flag) {
    bool bad = false;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        bad |= Low<T>::nonfinite(Low<T>::from_f(x[i]));
    warp_flag_or(flag, bad);
}

// ---------------------------------------------------------------- Alg. 2 scale state machine on the device
// state = {log2 S, first step whose attempt was not finite (-1: none), 1 when dL/dy_N is not finite}; `mirror` is the same
// three words in mapped host memory, which the host reads without a copy once it knows the kernel has finished.
__global__ void scale_init_kernel(unsigned* __restrict__ flag, const float* __restrict__ amax, int pbits, int e_fixed, int from_norm,
                                  int e_min, int e_max, int* __restrict__ state, volatile int* __restrict__ mirror) {
    int e = e_fixed, bad = 0;
    const float m = *amax;
    if (*flag != 0u || !(m <= 3.4028234e38f)) {
        bad = 1;
        *flag = 1u;                                  // stays raised: no update of this pass is committed
    } else if (from_norm) {                          // S_0 = 2^(p - ceil(log2 ||a||_inf)); 1 for a zero adjoint
        e = 0;
        if (m != 0.f) {
            int E;
            const float f = frexpf(m, &E);
            e = pbits - (f > 0.5f ? E : E - 1);
        }
        e = e < e_min ? e_min : (e > e_max ? e_max : e);
    }
    state[0] = e; state[1] = -1; state[2] = bad;
    mirror[0] = e; mirror[1] = -1; mirror[2] = bad;
    __threadfence_system();
}

// After the queued updates of step `step` (which skipped themselves if the flag was raised): record the accepted attempt and
// apply the growth test, or note the failure and halve.  Once a step has failed, nothing more is decided (and, the flag
// staying raised, nothing more is committed) until the host clears the failure and queues that step again.
__global__ void scale_decide_kernel(const unsigned* __restrict__ flag, const float* __restrict__ amax, int* __restrict__ state,
                                    volatile int* __restrict__ mirror, int step, int k_try, int growth_rule, int pbits, int e_min,
                                    int e_max, int* __restrict__ log_exp, int* __restrict__ log_att, unsigned char* __restrict__ log_dbl) {
    if (state[1] >= 0 || state[2] != 0) return;
    int e = state[0];
    if (*flag != 0u) {
        if (e > e_min) --e;
        state[0] = e; state[1] = step;
        mirror[0] = e; mirror[1] = step;
        __threadfence_system();
        return;
    }
    log_exp[step] = e; log_att[step] = k_try;
    unsigned char dbl = 0;
    if (k_try == 1) {                                // growth test on ||a_i||_inf (scaled by S or not, by the rule)
        const double scaled = growth_rule == 0 ? ldexp((double)*amax, e) : (double)*amax;
        if (scaled <= ldexp(1.0, pbits - 1) && e < e_max) { ++e; dbl = 1; }
    }
    log_dbl[step] = dbl;
    state[0] = e;
    mirror[0] = e;
}

template <typename T>
__global__ void fill_low_kernel(T* __restrict__ x, float v, long long n) {
    const T q = Low<T>::from_f(v);
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) x[i] = q;
}

__global__ void scale_kernel(float* __restrict__ x, float v, long long n) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) x[i] *= v;
}

__global__ void fill_kernel(float* __restrict__ x, float v, long long n) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        x[i] = v;
}

// ---------------------------------------------------------------- deterministic column sums (bias / time-column gradients)
constexpr int kColsPerBlock = 64;   // 32 lanes x 2 columns
constexpr int kRowLanes = 8;

// With `counters` (one zero word per column block, left zero again) the block that finishes a column block last also adds the
// partial rows in ascending order and writes the result as colsum_final_kernel would.
template <typename T>
__global__ void colsum_partial_kernel(const T* __restrict__ x, int M, int N, int rows_per_block,
                                      float* __restrict__ partial, unsigned* __restrict__ counters, float* __restrict__ dst1,
                                      long long s1, float* __restrict__ dst2, long long s2, float scale2, float beta) {
    __shared__ float sm[kRowLanes][kColsPerBlock];
    __shared__ bool last;
    int lane = threadIdx.x & 31, rl = threadIdx.x >> 5;
    int c = blockIdx.x * kColsPerBlock + lane * 2;
    int r0 = blockIdx.y * rows_per_block;
    int r1 = min(M, r0 + rows_per_block);
    float a0 = 0.f, a1 = 0.f;
    for (int r = r0 + rl; r < r1; r += kRowLanes) {
        if (c < N) a0 += Low<T>::to_f(x[(long long)r * N + c]);
        if (c + 1 < N) a1 += Low<T>::to_f(x[(long long)r * N + c + 1]);
    }
    sm[rl][lane * 2] = a0;
    sm[rl][lane * 2 + 1] = a1;
    __syncthreads();
    if (threadIdx.x < kColsPerBlock) {
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < kRowLanes; ++i) s += sm[i][threadIdx.x];
        int cc = blockIdx.x * kColsPerBlock + threadIdx.x;
        if (cc < N) partial[(long long)blockIdx.y * N + cc] = s;
        __threadfence();
    }
    if (counters == nullptr) return;
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(counters + blockIdx.x, 1u) == gridDim.y - 1;
    __syncthreads();
    if (!last) return;
    __threadfence();
    const int cc = blockIdx.x * kColsPerBlock + threadIdx.x;
    if (threadIdx.x < kColsPerBlock && cc < N) {
        float s = 0.f;
        for (int r = 0; r < (int)gridDim.y; ++r) s += __ldcg(partial + (long long)r * N + cc);
        if (dst1 != nullptr) dst1[cc * s1] = (beta != 0.f ? dst1[cc * s1] : 0.f) + s;
        if (dst2 != nullptr) dst2[cc * s2] = (beta != 0.f ? dst2[cc * s2] : 0.f) + scale2 * s;
    }
    if (threadIdx.x == 0) counters[blockIdx.x] = 0u;
}

__global__ void colsum_final_kernel(const float* __restrict__ partial, int R, int N, float* __restrict__ dst1,
                                    long long s1, float* __restrict__ dst2, long long s2, float scale2, float beta) {
    int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= N) return;
    float s = 0.f;
    for (int r = 0; r < R; ++r) s += partial[(long long)r * N + c];
    if (dst1 != nullptr) dst1[c * s1] = (beta != 0.f ? dst1[c * s1] : 0.f) + s;
    if (dst2 != nullptr) dst2[c * s2] = (beta != 0.f ? dst2[c * s2] : 0.f) + scale2 * s;
}

// Column sums of a low-format [M, N] matrix per group of 128 rows: out[g][n] = sum_{r in group g} x[r][n]
template <typename T>
__global__ void colsum_groups_kernel(const T* __restrict__ x, int M, int N, float* __restrict__ out) {
    int n = blockIdx.x * blockDim.x + threadIdx.x;
    int g = blockIdx.y;
    if (n >= N) return;
    int r0 = g * 128, r1 = min(M, r0 + 128);
    float s = 0.f;
    for (int r = r0; r < r1; ++r) s += Low<T>::to_f(x[(long long)r * N + n]);
    out[(long long)g * N + n] = s;
}

// Step parameter gradient from the fused kernel's scratch (see GradFinishArgs): blockIdx.y = layer; the first
// blocks of a layer walk its weight elements, the last ones its bias / time-column entries (one warp per entry,
// lanes split the (stage, row block) terms and are combined by a fixed shuffle tree).
constexpr int kFinishBiasBlocks = 16;
__global__ void grad_finish_kernel(GradFinishArgs a) {
    const GradFinishLayer& L = a.layer[blockIdx.y];
    const int wblocks = (int)gridDim.x - kFinishBiasBlocks;
    if ((int)blockIdx.x < wblocks) {
        const long long n_el = (long long)L.M * L.N;
        for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n_el; i += (long long)wblocks * blockDim.x) {
            float s = 0.f;
            for (int z = 0; z < L.splits; ++z) s += L.partial[(long long)z * n_el + i];
            float* o = a.out + L.w_off + (i / L.N) * L.ldo + (i % L.N);
            *o = (a.beta != 0.f ? a.beta * *o : 0.f) + a.coef * s;
        }
    } else if (L.bias_off >= 0 || L.time_off >= 0) {
        const int lane = threadIdx.x & 31;
        const int warps = kFinishBiasBlocks * (blockDim.x >> 5);
        const int terms = L.terms * L.rows;
        for (int m = ((int)blockIdx.x - wblocks) * (blockDim.x >> 5) + (threadIdx.x >> 5); m < L.M; m += warps) {
            float sb = 0.f, stime = 0.f;
            for (int t = lane; t < terms; t += 32) {
                const int j = t / L.rows, r = t - j * L.rows;      // stage j, batch slice r: column 0 of the stored ones-product
                const float v = L.colpart[L.col_off[j] + ((long long)r * L.M + m) * 8];
                sb += v;
                stime = fmaf(L.tau[j], v, stime);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                sb += __shfl_xor_sync(0xffffffffu, sb, o);
                stime += __shfl_xor_sync(0xffffffffu, stime, o);
            }
            if (lane == 0) {
                if (L.bias_off >= 0) {
                    float* o = a.out + L.bias_off + m;
                    *o = (a.beta != 0.f ? a.beta * *o : 0.f) + a.coef * sb;
                }
                if (L.time_off >= 0) {
                    float* o = a.out + L.time_off + (long long)m * L.ldo;
                    *o = (a.beta != 0.f ? a.beta * *o : 0.f) + a.coef * stime;
                }
            }
        }
    }
}

// ---------------------------------------------------------------- instance normalisation (parabolic layer, Sec. 6.3)
// One block per (image, group of 32 channels): 8 pixel lanes x 32 channels.  Per channel, sums over the plane's pixels are taken
// lane by lane and combined in a fixed order.
constexpr int kNormCh = 32, kNormLanes = kThreads / kNormCh;

__device__ __forceinline__ float plane_sum(float v, float (*sm)[kNormCh], int pl, int c) {
    __syncthreads();
    sm[pl][c] = v;
    __syncthreads();
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < kNormLanes; ++i) s += sm[i][c];
    return s;
}

// Z = Q16((S - mean) * rstd), rstd = 1 / sqrt(var + eps) per (image, channel), biased variance; rstd is kept for the backward pass
template <typename T>
__global__ void instnorm_fwd_kernel(const T* __restrict__ S, T* __restrict__ Z, float* __restrict__ rstd, int HW, int C, float eps) {
    __shared__ float sm[kNormLanes][kNormCh];
    const int c = threadIdx.x % kNormCh, pl = threadIdx.x / kNormCh;
    const int ch = blockIdx.x * kNormCh + c, img = blockIdx.y;
    const bool on = ch < C;
    const T* s = S + (long long)img * HW * C + ch;
    float a = 0.f;
    for (int p = pl; p < HW && on; p += kNormLanes) a += Low<T>::to_f(s[(long long)p * C]);
    const float mean = plane_sum(a, sm, pl, c) / (float)HW;
    float v = 0.f;
    for (int p = pl; p < HW && on; p += kNormLanes) { const float d = Low<T>::to_f(s[(long long)p * C]) - mean; v = fmaf(d, d, v); }
    const float r = rsqrtf(plane_sum(v, sm, pl, c) / (float)HW + eps);
    if (on && pl == 0) rstd[(long long)img * C + ch] = r;
    T* z = Z + (long long)img * HW * C + ch;
    for (int p = pl; p < HW && on; p += kNormLanes) z[(long long)p * C] = Low<T>::from_f((Low<T>::to_f(s[(long long)p * C]) - mean) * r);
}

// dS = Q16(rstd (dZ - mean(dZ) - Z mean(dZ Z))), dU = Q16(act'(S) dS); non-finite dS raises the flag.  norm = 0: dS = dZ.
template <typename T>
__global__ void instnorm_bwd_kernel(const T* __restrict__ dZ, const T* __restrict__ Z, const T* __restrict__ S, const float* __restrict__ rstd,
                                    T* __restrict__ dU, int HW, int C, int act, int norm, unsigned* __restrict__ flag) {
    __shared__ float sm[kNormLanes][kNormCh];
    const int c = threadIdx.x % kNormCh, pl = threadIdx.x / kNormCh;
    const int ch = blockIdx.x * kNormCh + c, img = blockIdx.y;
    const bool on = ch < C;
    const long long base = (long long)img * HW * C + ch;
    float m1 = 0.f, m2 = 0.f, r = 1.f;
    if (norm) {
        float a1 = 0.f, a2 = 0.f;
        for (int p = pl; p < HW && on; p += kNormLanes) {
            const float g = Low<T>::to_f(dZ[base + (long long)p * C]);
            a1 += g;
            a2 = fmaf(g, Low<T>::to_f(Z[base + (long long)p * C]), a2);
        }
        m1 = plane_sum(a1, sm, pl, c) / (float)HW;
        m2 = plane_sum(a2, sm, pl, c) / (float)HW;
        if (on) r = rstd[(long long)img * C + ch];
    }
    bool bad = false;
    for (int p = pl; p < HW && on; p += kNormLanes) {
        const long long i = base + (long long)p * C;
        const float g = Low<T>::to_f(dZ[i]);
        const T ds = norm ? Low<T>::from_f(r * (g - m1 - Low<T>::to_f(Z[i]) * m2)) : dZ[i];
        bad |= Low<T>::nonfinite(ds);
        dU[i] = Low<T>::from_f(act_deriv_from_output(act, Low<T>::to_f(S[i])) * Low<T>::to_f(ds));
    }
    warp_flag_or(flag, bad);
}

// The same two kernels for channel counts that are multiples of 64 in a 16-bit format: a thread owns 8 consecutive channels (one
// 16-byte load per pixel) and every 64th pixel, a block one image and 64 channels, so that a warp reads whole 128-byte lines.
// Plane sums: the 64 pixel lanes' partial sums added in ascending order.
constexpr int kNorm8Lanes = 64, kNorm8Threads = kNorm8Lanes * 8;

__device__ __forceinline__ void plane_sum8(float (&v)[8], float (*sm)[64 + 1], int pl, int cg) {
    __syncthreads();
#pragma unroll
    for (int e = 0; e < 8; ++e) sm[pl][cg * 8 + e] = v[e];
    __syncthreads();
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        float s = 0.f;
        for (int i = 0; i < kNorm8Lanes; ++i) s += sm[i][cg * 8 + e];
        v[e] = s;
    }
}

template <typename T>
__global__ void __launch_bounds__(kNorm8Threads) instnorm_fwd8_kernel(const T* __restrict__ S, T* __restrict__ Z, float* __restrict__ rstd,
                                                                        int HW, int C, float eps) {
    __shared__ float sm[kNorm8Lanes][64 + 1];
    const int cg = threadIdx.x & 7, pl = threadIdx.x >> 3;
    const int ch0 = blockIdx.x * 64 + cg * 8, img = blockIdx.y;
    const T* s = S + (long long)img * HW * C + ch0;
    T* z = Z + (long long)img * HW * C + ch0;
    float mean[8], var[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) mean[e] = var[e] = 0.f;
#pragma unroll 4
    for (int p = pl; p < HW; p += kNorm8Lanes) {
        const Pack<T, 8> v = *reinterpret_cast<const Pack<T, 8>*>(s + (long long)p * C);
#pragma unroll
        for (int e = 0; e < 8; ++e) mean[e] += Low<T>::to_f(v.v[e]);
    }
    plane_sum8(mean, sm, pl, cg);
#pragma unroll
    for (int e = 0; e < 8; ++e) mean[e] /= (float)HW;
#pragma unroll 4
    for (int p = pl; p < HW; p += kNorm8Lanes) {
        const Pack<T, 8> v = *reinterpret_cast<const Pack<T, 8>*>(s + (long long)p * C);
#pragma unroll
        for (int e = 0; e < 8; ++e) { const float d = Low<T>::to_f(v.v[e]) - mean[e]; var[e] = fmaf(d, d, var[e]); }
    }
    plane_sum8(var, sm, pl, cg);
    float r[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) r[e] = rsqrtf(var[e] / (float)HW + eps);
    if (pl == 0) {
#pragma unroll
        for (int e = 0; e < 8; ++e) rstd[(long long)img * C + ch0 + e] = r[e];
    }
#pragma unroll 4
    for (int p = pl; p < HW; p += kNorm8Lanes) {
        const Pack<T, 8> v = *reinterpret_cast<const Pack<T, 8>*>(s + (long long)p * C);
        Pack<T, 8> o;
#pragma unroll
        for (int e = 0; e < 8; ++e) o.v[e] = Low<T>::from_f((Low<T>::to_f(v.v[e]) - mean[e]) * r[e]);
        *reinterpret_cast<Pack<T, 8>*>(z + (long long)p * C) = o;
    }
}

template <typename T>
__global__ void __launch_bounds__(kNorm8Threads) instnorm_bwd8_kernel(const T* __restrict__ dZ, const T* __restrict__ Z, const T* __restrict__ S,
                                                                        const float* __restrict__ rstd, T* __restrict__ dU, int HW, int C, int act,
                                                                        int norm, unsigned* __restrict__ flag) {
    __shared__ float sm[kNorm8Lanes][64 + 1];
    const int cg = threadIdx.x & 7, pl = threadIdx.x >> 3;
    const int ch0 = blockIdx.x * 64 + cg * 8, img = blockIdx.y;
    const long long base = (long long)img * HW * C + ch0;
    float m1[8], m2[8], r[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { m1[e] = m2[e] = 0.f; r[e] = 1.f; }
    if (norm) {
#pragma unroll 4
        for (int p = pl; p < HW; p += kNorm8Lanes) {
            const Pack<T, 8> g = *reinterpret_cast<const Pack<T, 8>*>(dZ + base + (long long)p * C);
            const Pack<T, 8> zz = *reinterpret_cast<const Pack<T, 8>*>(Z + base + (long long)p * C);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float gf = Low<T>::to_f(g.v[e]);
                m1[e] += gf;
                m2[e] = fmaf(gf, Low<T>::to_f(zz.v[e]), m2[e]);
            }
        }
        plane_sum8(m1, sm, pl, cg);
        plane_sum8(m2, sm, pl, cg);
#pragma unroll
        for (int e = 0; e < 8; ++e) { m1[e] /= (float)HW; m2[e] /= (float)HW; r[e] = rstd[(long long)img * C + ch0 + e]; }
    }
    bool bad = false;
#pragma unroll 2
    for (int p = pl; p < HW; p += kNorm8Lanes) {
        const long long i = base + (long long)p * C;
        const Pack<T, 8> g = *reinterpret_cast<const Pack<T, 8>*>(dZ + i);
        const Pack<T, 8> sv = *reinterpret_cast<const Pack<T, 8>*>(S + i);
        Pack<T, 8> zz;
        if (norm) zz = *reinterpret_cast<const Pack<T, 8>*>(Z + i);
        Pack<T, 8> o;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float gf = Low<T>::to_f(g.v[e]);
            const T ds = norm ? Low<T>::from_f(r[e] * (gf - m1[e] - Low<T>::to_f(zz.v[e]) * m2[e])) : g.v[e];
            bad |= Low<T>::nonfinite(ds);
            o.v[e] = Low<T>::from_f(act_deriv_from_output(act, Low<T>::to_f(sv.v[e])) * Low<T>::to_f(ds));
        }
        *reinterpret_cast<Pack<T, 8>*>(dU + i) = o;
    }
    warp_flag_or(flag, bad);
}

// ---------------------------------------------------------------- time-grid gradient (Alg. 2, the two t' updates)
// Fixed-order block reduction: lanes by shuffles, warps in ascending order; the result is valid in thread 0.
__device__ __forceinline__ float block_sum_fixed(float v, float* sm) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = v;
    __syncthreads();
    float s = 0.f;
    if (threadIdx.x == 0)
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) s += sm[i];
    return s;
}

template <typename T>
__global__ void dot_partial_kernel(DotPairs pr, int B, int d, float* __restrict__ part) {
    __shared__ float sm[kThreads / 32];
    const int rows_per = (B + (int)gridDim.x - 1) / (int)gridDim.x;
    const int r0 = blockIdx.x * rows_per, r1 = min(B, r0 + rows_per);
    const long long n = (long long)max(0, r1 - r0) * d;
    float acc = 0.f;
    for (int q = 0; q < pr.n; ++q) {
        const T* x = (const T*)pr.x[q];
        float s = 0.f;
        for (long long i = threadIdx.x; i < n; i += blockDim.x) {
            const long long r = r0 + i / d;
            const int c = (int)(i % d);
            const float xv = Low<T>::to_f(x[r * pr.ldx[q] + c]);
            const float yv = pr.y_f32[q] ? ((const float*)pr.y[q])[r * pr.ldy[q] + c] : Low<T>::to_f(((const T*)pr.y[q])[r * pr.ldy[q] + c]);
            s = fmaf(xv, yv, s);
        }
        acc = fmaf(pr.coef[q], s, acc);
    }
    const float tot = block_sum_fixed(acc, sm);
    if (threadIdx.x == 0) part[blockIdx.x] = tot;
}

template <typename T>
__global__ void stage_time_cot_kernel(StageTimeArgs a) {
    __shared__ float sm[kThreads / 32];
    const T* wt = (const T*)a.wt;
    for (int j = 0; j < a.terms; ++j) {
        float acc = 0.f;
        for (int m = threadIdx.x; m < a.M; m += blockDim.x) {
            float cs = 0.f;
            for (int r = 0; r < a.rows; ++r) cs += a.colsum[a.off[j] + ((long long)r * a.M + m) * a.stride];
            acc = fmaf(Low<T>::to_f(wt[m]), cs, acc);
        }
        const float tot = block_sum_fixed(acc, sm);
        if (threadIdx.x == 0) a.dtau[j] = tot;
        __syncthreads();
    }
}

template <typename T>
__global__ void tgrad_reduce_kernel(const float* __restrict__ part_phi, const float* __restrict__ part_dh, const float* __restrict__ dtau,
                                    const float* __restrict__ c, int stages, float* __restrict__ out, unsigned* __restrict__ flag) {
    __shared__ float sm[kThreads / 32];
    float p1 = 0.f, p2 = 0.f;
    for (int i = threadIdx.x; i < kDotBlocks; i += blockDim.x) { p1 += part_phi[i]; p2 += part_dh[i]; }
    const float phi = block_sum_fixed(p1, sm);
    const float dhd = block_sum_fixed(p2, sm);
    if (threadIdx.x == 0) {
        float dt = 0.f, dh = dhd;
        for (int j = 0; j < stages; ++j) { dt += dtau[j]; dh = fmaf(c[j], dtau[j], dh); }
        out[0] = phi; out[1] = dt; out[2] = dh;
        if (flag != nullptr && (Low<T>::nonfinite(Low<T>::from_f(dt)) || Low<T>::nonfinite(Low<T>::from_f(dh)))) atomicOr(flag, 1u);
    }
}

__global__ void tgrad_update_kernel(float* __restrict__ tprime, int i, const float* __restrict__ vals, float coef,
                                    const unsigned* __restrict__ skip_if_set, const int* __restrict__ e_dev) {
    if (threadIdx.x != 0 || (skip_if_set != nullptr && *skip_if_set != 0u)) return;
    if (e_dev != nullptr) coef = ldexpf(coef, -*e_dev);
    const float phi = vals[0], dt = vals[1], dh = vals[2];
    tprime[i] = tprime[i] + coef * (dt - dh) - phi;
    tprime[i + 1] = tprime[i + 1] + coef * dh + phi;
}

// ---------------------------------------------------------------- CNF tangent path (Sec. 6.1)
// G = Q16(sigma'(z) * U), sigma' taken from the rounded layer output H
template <typename T>
__global__ void cnf_tangent_act_kernel(int act, const T* __restrict__ H, const T* __restrict__ U, T* __restrict__ G,
                                       long long n) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        G[i] = Low<T>::from_f(act_deriv_from_output(act, Low<T>::to_f(H[i])) * Low<T>::to_f(U[i]));
}

// k_l[b] = Q16(-sum_n eps[b, n] U[b, n]); one warp per sample
template <typename T>
__global__ void cnf_trace_kernel(const signed char* __restrict__ eps, const T* __restrict__ U, T* __restrict__ k_l,
                                 int B, int d) {
    int warps_per_block = blockDim.x >> 5;
    int lane = threadIdx.x & 31;
    for (long long b = blockIdx.x * (long long)warps_per_block + (threadIdx.x >> 5); b < B;
         b += (long long)gridDim.x * warps_per_block) {
        float s = 0.f;
        for (int n = lane; n < d; n += 32) s += (float)eps[b * d + n] * Low<T>::to_f(U[b * d + n]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) k_l[b] = Low<T>::from_f(-s);
    }
}

template <typename T>
__global__ void cnf_probe_to_low_kernel(const signed char* __restrict__ eps, T* __restrict__ out, long long n) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        out[i] = Low<T>::from_f((float)eps[i]);
}

// cotangent of the last tangent output: ubar[b, n] = Q16(-kappa_l[b] * eps[b, n])
template <typename T>
__global__ void cnf_ubar_last_kernel(const T* __restrict__ kappa_l, const signed char* __restrict__ eps,
                                     T* __restrict__ ubar, int B, int d, unsigned* __restrict__ flag) {
    long long n = (long long)B * d;
    bool bad = false;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        T q = Low<T>::from_f(-Low<T>::to_f(kappa_l[i / d]) * (float)eps[i]);
        bad |= Low<T>::nonfinite(q);
        ubar[i] = q;
    }
    warp_flag_or(flag, bad);
}

// ubar' = Q16(s * gbar), zeta' = Q16(s * hbar + s (1 - s) * U * gbar), s = sigma'(z) from the rounded output H
template <typename T>
__global__ void cnf_backprop_act_kernel(int act, const T* __restrict__ H, const T* __restrict__ U,
                                        const float* __restrict__ hbar, const float* __restrict__ gbar,
                                        T* __restrict__ zeta, T* __restrict__ ubar, long long n,
                                        unsigned* __restrict__ flag) {
    bool bad = false;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        float s = act_deriv_from_output(act, Low<T>::to_f(H[i]));
        float gb = gbar[i];
        T ub = Low<T>::from_f(s * gb);
        T ze = Low<T>::from_f(s * hbar[i] + s * (1.f - s) * Low<T>::to_f(U[i]) * gb);
        bad |= Low<T>::nonfinite(ub) | Low<T>::nonfinite(ze);
        ubar[i] = ub;
        zeta[i] = ze;
    }
    warp_flag_or(flag, bad);
}

}  // namespace

// ================================================================= launchers

#define COUNT(l) do { if (l) ++*(l); } while (0)

void launch_quantize_matrix(mpode_dtype dt, const float* src, long long src_ld, int rows, int cols, void* dst,
                            void* dst_t, cudaStream_t st, long long* launches) {
    dim3 grid((cols + 31) / 32, (rows + 31) / 32), block(32, 8);
    MPODE_DISPATCH_T(dt, T, (quantize_matrix_kernel<T><<<grid, block, 0, st>>>(src, src_ld, rows, cols, (T*)dst, (T*)dst_t)));
    COUNT(launches);
}

void launch_quantize_conv_weights(mpode_dtype dt, const float* src, int cout, int cin_total, int cin_keep, void* dst,
                                  void* dst_flip_t, cudaStream_t st, long long* launches, float sign) {
    long long n = (long long)cout * 9 * cin_keep;
    MPODE_DISPATCH_T(dt, T, (quantize_conv_weights_kernel<T><<<grid_for(n), kThreads, 0, st>>>(
                                src, cout, cin_total, cin_keep, (T*)dst, (T*)dst_flip_t, sign)));
    COUNT(launches);
}

static inline bool vec8_ok(int d, int D, std::initializer_list<const void*> ptrs) {
    if (d % 8 != 0 || D % 8 != 0) return false;
    for (const void* p : ptrs)
        if (p != nullptr && !aligned_to(p, 32)) return false;
    return true;
}

void launch_conv_wgrad_reduce(const float* partial, int S, int C, int ct, float* out, float beta, cudaStream_t st, long long* launches,
                              float sign) {
    conv_wgrad_reduce_kernel<<<dim3(C / 32, C / 32, 9), 256, 0, st>>>(partial, S, C, ct, out, beta, sign);
    COUNT(launches);
}

void launch_conv_class_grads(mpode_dtype dt, const void* dz, int B, int H, int W, int C, int ct, float tau, float* scratch,
                             float* wt_out, float* bias_out, float beta, cudaStream_t st, long long* launches) {
    const long long pixels = (long long)B * H * W;
    int blocks = (int)((pixels + 255) / 256);        // 128-thread blocks of about 128 registers a thread: four per SM, one wave
    if (blocks > 4 * kSMs) blocks = 4 * kSMs;
    const long long per_block = (pixels + blocks - 1) / blocks;
    MPODE_DISPATCH_T(dt, T, (conv_class_sums_kernel<T><<<blocks, 128, (size_t)72 * 128 * sizeof(float), st>>>(
                                (const T*)dz, pixels, H, W, C, per_block, scratch)));
    COUNT(launches);
    float* cs = scratch + (size_t)8 * kSMs * 9 * C;   // reduced class sums behind the per-block ones
    conv_class_reduce_kernel<<<(9 * C + 7) / 8, 256, 0, st>>>(scratch, blocks, 9 * C, cs);
    COUNT(launches);
    conv_class_final_kernel<<<1, 576, (size_t)9 * C * sizeof(float), st>>>(cs, C, ct, tau, wt_out, bias_out, beta);
    COUNT(launches);
}

// [H * W][64] low-format table of one image: column c < 9 is 1 where the pixel's position class (3 * row class + column class)
// is c, everything else 0.  As a 64-channel operand block beside the image it turns the class sums into rows of a contraction.
template <typename T>
__global__ void conv_class_indicator_kernel(int H, int W, T* __restrict__ out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= H * W * 64) return;
    const int c = i & 63, pix = i >> 6, y = pix / W, x = pix - y * W;
    const int cls = 3 * (y == 0 ? 0 : (y == H - 1 ? 2 : 1)) + (x == 0 ? 0 : (x == W - 1 ? 2 : 1));
    out[i] = Low<T>::from_f(c == cls ? 1.f : 0.f);
}

void launch_conv_class_indicator(mpode_dtype dt, int H, int W, void* out, cudaStream_t st, long long* launches) {
    MPODE_DISPATCH_T(dt, T, (conv_class_indicator_kernel<T><<<(H * W * 64 + 255) / 256, 256, 0, st>>>(H, W, (T*)out)));
    COUNT(launches);
}

void launch_conv_class_bias(mpode_dtype dt, const void* b, const void* w, int cin_total, float tau, int C, float* out,
                            cudaStream_t st, long long* launches) {
    MPODE_DISPATCH_T(dt, T, (conv_class_bias_kernel<T><<<(9 * C + 127) / 128, 128, 0, st>>>((const T*)b, (const T*)w, cin_total, tau, C, out)));
    COUNT(launches);
}

// 16 elements per thread and iteration (64 bytes of an fp32 tensor, 32 of a 16-bit one): enough bytes in flight to fill
// the memory pipe; needs widths that are multiples of 16 and 64-byte aligned pointers
static inline bool vec16_ok(mpode_dtype dt, int d, int D, std::initializer_list<const void*> ptrs) {
    if (dt == MPODE_F32 || d % 16 != 0 || D % 16 != 0) return false;
    for (const void* p : ptrs)
        if (p != nullptr && !aligned_to(p, 64)) return false;
    return true;
}

void launch_init_state(mpode_dtype dt, const float* y0, float* y, void* traj0, int B, int d, int D, cudaStream_t st,
                       long long* launches) {
    if (vec8_ok(d, D, {y0, y, traj0})) {
        MPODE_DISPATCH_T(dt, T, (init_state_kernel<T, 8><<<grid_for((long long)B * d / 8), kThreads, 0, st>>>(y0, y, (T*)traj0, B, d, D)));
    } else {
        MPODE_DISPATCH_T(dt, T, (init_state_kernel<T, 1><<<grid_for((long long)B * d), kThreads, 0, st>>>(y0, y, (T*)traj0, B, d, D)));
    }
    COUNT(launches);
}

void launch_stage_input(mpode_dtype dt, const void* base, const Terms& t, void* out, long long n, cudaStream_t st,
                        long long* launches) {
    bool v8 = (n % 8 == 0) && aligned_to(base, 32) && aligned_to(out, 32);
    for (int l = 0; l < t.n; ++l) v8 = v8 && aligned_to(t.p[l], 32);
    if (v8 && n % 16 == 0 && dt != MPODE_F32) {   // 32 bytes per operand and thread in flight: needed to fill the memory pipe
        MPODE_DISPATCH_T(dt, T, (stage_input_kernel<T, 16><<<grid_for(n / 16), kThreads, 0, st>>>((const T*)base, t, (T*)out, n / 16)));
    } else if (v8) {
        MPODE_DISPATCH_T(dt, T, (stage_input_kernel<T, 8><<<grid_for(n / 8), kThreads, 0, st>>>((const T*)base, t, (T*)out, n / 8)));
    } else {
        MPODE_DISPATCH_T(dt, T, (stage_input_kernel<T, 1><<<grid_for(n), kThreads, 0, st>>>((const T*)base, t, (T*)out, n)));
    }
    COUNT(launches);
}

void launch_final_combine(mpode_dtype dt, float* y, const Terms& t, void* traj_next, int B, int d, int D,
                          int round_increment, float h, cudaStream_t st, long long* launches) {
    bool v8 = vec8_ok(d, D, {y, traj_next});
    for (int l = 0; l < t.n; ++l) v8 = v8 && aligned_to(t.p[l], 32);
    bool v16 = v8 && vec16_ok(dt, d, D, {y, traj_next});
    for (int l = 0; l < t.n; ++l) v16 = v16 && aligned_to(t.p[l], 64);
    if (v16) {
        MPODE_DISPATCH_T(dt, T, (final_combine_kernel<T, 16><<<grid_for((long long)B * d / 16), kThreads, 0, st>>>(
                                    y, t, (T*)traj_next, B, d, D, round_increment, h)));
    } else if (v8) {
        MPODE_DISPATCH_T(dt, T, (final_combine_kernel<T, 8><<<grid_for((long long)B * d / 8), kThreads, 0, st>>>(
                                    y, t, (T*)traj_next, B, d, D, round_increment, h)));
    } else {
        MPODE_DISPATCH_T(dt, T, (final_combine_kernel<T, 1><<<grid_for((long long)B * d), kThreads, 0, st>>>(
                                    y, t, (T*)traj_next, B, d, D, round_increment, h)));
    }
    COUNT(launches);
}

void launch_column_combine(mpode_dtype dt, float* y, int D, int col, const Terms& t, int B, int round_increment,
                           float h, cudaStream_t st, long long* launches) {
    MPODE_DISPATCH_T(dt, T, (column_combine_kernel<T><<<grid_for(B), kThreads, 0, st>>>(y, D, col, t, B, round_increment, h)));
    COUNT(launches);
}

void launch_copy_amax(const float* src, float* dst, long long n, float* amax, unsigned* flag, cudaStream_t st,
                      long long* launches) {
    copy_amax_kernel<<<grid_for(n), kThreads, 0, st>>>(src, dst, n, amax, flag);
    COUNT(launches);
}

void launch_seed(mpode_dtype dt, const float* a, int e, void* v, void* v_l, int B, int d, int D, unsigned* flag,
                 cudaStream_t st, long long* launches, void* kappa_last, float b_last, const int* e_dev) {
    if (vec16_ok(dt, d, D, {a, v, kappa_last})) {
        MPODE_DISPATCH_T(dt, T, (seed_kernel<T, 16><<<grid_for((long long)B * d / 16), kThreads, 0, st>>>(a, e, (T*)v, (T*)v_l, B, d, D, flag,
                                                                                                        (T*)kappa_last, b_last, e_dev)));
    } else if (vec8_ok(d, D, {a, v, kappa_last})) {
        MPODE_DISPATCH_T(dt, T, (seed_kernel<T, 8><<<grid_for((long long)B * d / 8), kThreads, 0, st>>>(a, e, (T*)v, (T*)v_l, B, d, D, flag,
                                                                                                      (T*)kappa_last, b_last, e_dev)));
    } else {
        MPODE_DISPATCH_T(dt, T, (seed_kernel<T, 1><<<grid_for((long long)B * d), kThreads, 0, st>>>(a, e, (T*)v, (T*)v_l, B, d, D, flag,
                                                                                                  (T*)kappa_last, b_last, e_dev)));
    }
    COUNT(launches);
}

void launch_kappa(mpode_dtype dt, const void* v, float bj, const Terms& t, void* out, long long n, unsigned* flag,
                  cudaStream_t st, long long* launches) {
    bool v8 = (n % 8 == 0) && aligned_to(v, 32) && aligned_to(out, 32);
    for (int l = 0; l < t.n; ++l) v8 = v8 && aligned_to(t.p[l], 32);
    if (v8 && n % 16 == 0 && dt != MPODE_F32) {
        MPODE_DISPATCH_T(dt, T, (kappa_kernel<T, 16><<<grid_for(n / 16), kThreads, 0, st>>>((const T*)v, bj, t, (T*)out, n / 16, flag)));
    } else if (v8) {
        MPODE_DISPATCH_T(dt, T, (kappa_kernel<T, 8><<<grid_for(n / 8), kThreads, 0, st>>>((const T*)v, bj, t, (T*)out, n / 8, flag)));
    } else {
        MPODE_DISPATCH_T(dt, T, (kappa_kernel<T, 1><<<grid_for(n), kThreads, 0, st>>>((const T*)v, bj, t, (T*)out, n, flag)));
    }
    COUNT(launches);
}

void launch_commit_a(mpode_dtype dt, float* a, const Terms& psis, float coef, int B, int d, int D, float* amax,
                     cudaStream_t st, long long* launches, const unsigned* skip_if_set, const float* add, const int* e_dev) {
    bool v8 = vec8_ok(d, D, {a, add});
    for (int l = 0; l < psis.n; ++l) v8 = v8 && aligned_to(psis.p[l], 32);
    bool v16 = v8 && vec16_ok(dt, d, D, {a, add});
    for (int l = 0; l < psis.n; ++l) v16 = v16 && aligned_to(psis.p[l], 64);
    if (v16) {
        MPODE_DISPATCH_T(dt, T, (commit_a_kernel<T, 16><<<grid_for((long long)B * d / 16), kThreads, 0, st>>>(a, psis, coef, B, d, D, amax, skip_if_set, add, e_dev)));
    } else if (v8) {
        MPODE_DISPATCH_T(dt, T, (commit_a_kernel<T, 8><<<grid_for((long long)B * d / 8), kThreads, 0, st>>>(a, psis, coef, B, d, D, amax, skip_if_set, add, e_dev)));
    } else {
        MPODE_DISPATCH_T(dt, T, (commit_a_kernel<T, 1><<<grid_for((long long)B * d), kThreads, 0, st>>>(a, psis, coef, B, d, D, amax, skip_if_set, add, e_dev)));
    }
    COUNT(launches);
}

void launch_commit_g(float* g, const float* dg, float coef, long long p, cudaStream_t st, long long* launches,
                     const unsigned* skip_if_set, const int* e_dev) {
    commit_g_kernel<<<grid_for(p), kThreads, 0, st>>>(g, dg, coef, p, skip_if_set, e_dev);
    COUNT(launches);
}

void launch_scale_init(unsigned* flag, const float* amax, int pbits, int e_fixed, int from_norm, int e_min, int e_max, int* state,
                       int* mirror, cudaStream_t st, long long* launches) {
    scale_init_kernel<<<1, 1, 0, st>>>(flag, amax, pbits, e_fixed, from_norm, e_min, e_max, state, mirror);
    COUNT(launches);
}

void launch_scale_decide(const unsigned* flag, const float* amax, int* state, int* mirror, int step, int k_try, int growth_rule,
                         int pbits, int e_min, int e_max, int* log_exp, int* log_att, unsigned char* log_dbl, cudaStream_t st,
                         long long* launches) {
    scale_decide_kernel<<<1, 1, 0, st>>>(flag, amax, state, mirror, step, k_try, growth_rule, pbits, e_min, e_max, log_exp, log_att,
                                          log_dbl);
    COUNT(launches);
}

void launch_check_as_low(mpode_dtype dt, const float* x, long long n, unsigned* flag, cudaStream_t st,
                         long long* launches) {
    MPODE_DISPATCH_T(dt, T, (check_as_low_kernel<T><<<grid_for(n), kThreads, 0, st>>>(x, n, flag)));
    COUNT(launches);
}

void launch_fill_low(mpode_dtype dt, void* x, float v, long long n, cudaStream_t st, long long* launches) {
    MPODE_DISPATCH_T(dt, T, (fill_low_kernel<T><<<grid_for(n), kThreads, 0, st>>>((T*)x, v, n)));
    COUNT(launches);
}

void launch_scale(float* x, float v, long long n, cudaStream_t st, long long* launches) {
    scale_kernel<<<grid_for(n), kThreads, 0, st>>>(x, v, n);
    COUNT(launches);
}

void launch_fill(float* x, float v, long long n, cudaStream_t st, long long* launches) {
    fill_kernel<<<grid_for(n), kThreads, 0, st>>>(x, v, n);
    COUNT(launches);
}

void launch_instnorm_fwd(mpode_dtype dt, const void* S, void* Z, float* rstd, int B, int HW, int C, float eps, cudaStream_t st,
                         long long* launches) {
    if (dt != MPODE_F32 && C % 64 == 0 && aligned_to(S, 16) && aligned_to(Z, 16)) {
        dim3 grid8(C / 64, B);
        MPODE_DISPATCH_T(dt, T, (instnorm_fwd8_kernel<T><<<grid8, kNorm8Threads, 0, st>>>((const T*)S, (T*)Z, rstd, HW, C, eps)));
        COUNT(launches);
        return;
    }
    dim3 grid((C + kNormCh - 1) / kNormCh, B);
    MPODE_DISPATCH_T(dt, T, (instnorm_fwd_kernel<T><<<grid, kThreads, 0, st>>>((const T*)S, (T*)Z, rstd, HW, C, eps)));
    COUNT(launches);
}

void launch_instnorm_bwd(mpode_dtype dt, const void* dZ, const void* Z, const void* S, const float* rstd, void* dU, int B, int HW, int C,
                         int act, int norm, unsigned* flag, cudaStream_t st, long long* launches) {
    if (dt != MPODE_F32 && C % 64 == 0 && aligned_to(dZ, 16) && aligned_to(Z, 16) && aligned_to(S, 16) && aligned_to(dU, 16)) {
        dim3 grid8(C / 64, B);
        MPODE_DISPATCH_T(dt, T, (instnorm_bwd8_kernel<T><<<grid8, kNorm8Threads, 0, st>>>((const T*)dZ, (const T*)Z, (const T*)S, rstd, (T*)dU,
                                                                                            HW, C, act, norm, flag)));
        COUNT(launches);
        return;
    }
    dim3 grid((C + kNormCh - 1) / kNormCh, B);
    MPODE_DISPATCH_T(dt, T, (instnorm_bwd_kernel<T><<<grid, kThreads, 0, st>>>((const T*)dZ, (const T*)Z, (const T*)S, rstd, (T*)dU, HW, C, act,
                                                                            norm, flag)));
    COUNT(launches);
}

void launch_dot_partial(mpode_dtype dt, const DotPairs& pr, int B, int d, float* part, cudaStream_t st, long long* launches) {
    MPODE_DISPATCH_T(dt, T, (dot_partial_kernel<T><<<kDotBlocks, kThreads, 0, st>>>(pr, B, d, part)));
    COUNT(launches);
}

void launch_stage_time_cot(mpode_dtype dt, const StageTimeArgs& a, cudaStream_t st, long long* launches) {
    MPODE_DISPATCH_T(dt, T, (stage_time_cot_kernel<T><<<1, kThreads, 0, st>>>(a)));
    COUNT(launches);
}

void launch_tgrad_reduce(mpode_dtype dt, const float* part_phi, const float* part_dh, const float* dtau, const float* c, int stages,
                         float* out, unsigned* flag, cudaStream_t st, long long* launches) {
    MPODE_DISPATCH_T(dt, T, (tgrad_reduce_kernel<T><<<1, kThreads, 0, st>>>(part_phi, part_dh, dtau, c, stages, out, flag)));
    COUNT(launches);
}

void launch_tgrad_update(float* tprime, int i, const float* vals, float coef, const unsigned* skip_if_set, cudaStream_t st,
                         long long* launches, const int* e_dev) {
    tgrad_update_kernel<<<1, 32, 0, st>>>(tprime, i, vals, coef, skip_if_set, e_dev);
    COUNT(launches);
}

int launch_colsum(mpode_dtype dt, const void* x, int M, int N, float* partial, float* dst1, long long s1, float* dst2,
                  long long s2, float scale2, float beta, cudaStream_t st, long long* launches, unsigned* counters) {
    // row chunks: enough blocks to fill the GPU, at most 64 partial rows (the scratch holds 64 * N floats)
    int col_blocks = (N + kColsPerBlock - 1) / kColsPerBlock;
    int R = (2 * kSMs + col_blocks - 1) / col_blocks;
    if (R > 64) R = 64;
    int max_r = (M + kRowLanes - 1) / kRowLanes;
    if (R > max_r) R = max_r;
    if (R < 1) R = 1;
    int rows_per_block = (M + R - 1) / R;
    R = (M + rows_per_block - 1) / rows_per_block;
    dim3 grid(col_blocks, R);
    if (counters != nullptr && col_blocks > kColsumCounters) counters = nullptr;
    MPODE_DISPATCH_T(dt, T, (colsum_partial_kernel<T><<<grid, kThreads, 0, st>>>((const T*)x, M, N, rows_per_block, partial, counters, dst1, s1, dst2,
                                                                                   s2, scale2, beta)));
    COUNT(launches);
    if (counters == nullptr) {
        colsum_final_kernel<<<(N + 127) / 128, 128, 0, st>>>(partial, R, N, dst1, s1, dst2, s2, scale2, beta);
        COUNT(launches);
    }
    return R;
}

void launch_colsum_groups(mpode_dtype dt, const void* x, int M, int N, float* out, cudaStream_t st, long long* launches) {
    dim3 grid((N + 127) / 128, (M + 127) / 128);
    MPODE_DISPATCH_T(dt, T, (colsum_groups_kernel<T><<<grid, 128, 0, st>>>((const T*)x, M, N, out)));
    COUNT(launches);
}

void launch_grad_finish(const GradFinishArgs& a, cudaStream_t st, long long* launches) {
    dim3 grid(kSMs * 2 + kFinishBiasBlocks, a.n_layers);
    grad_finish_kernel<<<grid, kThreads, 0, st>>>(a);
    COUNT(launches);
}

void launch_cnf_tangent_act(mpode_dtype dt, int act, const void* H, const void* U, void* G, long long n,
                            cudaStream_t st, long long* launches) {
    MPODE_DISPATCH_T(dt, T, (cnf_tangent_act_kernel<T><<<grid_for(n), kThreads, 0, st>>>(act, (const T*)H, (const T*)U, (T*)G, n)));
    COUNT(launches);
}

void launch_cnf_trace(mpode_dtype dt, const signed char* eps, const void* U, void* k_l, int B, int d, cudaStream_t st,
                      long long* launches) {
    int blocks = (B + 7) / 8;
    if (blocks > kSMs * 8) blocks = kSMs * 8;
    MPODE_DISPATCH_T(dt, T, (cnf_trace_kernel<T><<<blocks, kThreads, 0, st>>>(eps, (const T*)U, (T*)k_l, B, d)));
    COUNT(launches);
}

void launch_cnf_probe_to_low(mpode_dtype dt, const signed char* eps, void* out, long long n, cudaStream_t st,
                             long long* launches) {
    MPODE_DISPATCH_T(dt, T, (cnf_probe_to_low_kernel<T><<<grid_for(n), kThreads, 0, st>>>(eps, (T*)out, n)));
    COUNT(launches);
}

void launch_cnf_ubar_last(mpode_dtype dt, const void* kappa_l, const signed char* eps, void* ubar, int B, int d,
                          unsigned* flag, cudaStream_t st, long long* launches) {
    MPODE_DISPATCH_T(dt, T, (cnf_ubar_last_kernel<T><<<grid_for((long long)B * d), kThreads, 0, st>>>(
                                (const T*)kappa_l, eps, (T*)ubar, B, d, flag)));
    COUNT(launches);
}

void launch_cnf_backprop_act(mpode_dtype dt, int act, const void* H, const void* U, const float* hbar,
                             const float* gbar, void* zeta, void* ubar, long long n, unsigned* flag, cudaStream_t st,
                             long long* launches) {
    MPODE_DISPATCH_T(dt, T, (cnf_backprop_act_kernel<T><<<grid_for(n), kThreads, 0, st>>>(
                                act, (const T*)H, (const T*)U, hbar, gbar, (T*)zeta, (T*)ubar, n, flag)));
    COUNT(launches);
}

}  // namespace mpode
