// General contraction on the CUDA cores: C(m, n) = sum_k A(m, k) B(n, k) with arbitrary operand strides, an
// optional implicit 3x3-convolution view of one operand, fp32 accumulation in a fixed order (deterministic),
// and the fused epilogues of the velocity layers.  It serves every shape and all three low formats; it is
// the float32 path (TF32 cannot meet the 1e-5 accuracy target) and the fallback for shapes the tensor-core
// kernels do not take.
#include "common.cuh"

namespace mpode {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4;
constexpr int kGemmThreads = (BM / TM) * (BN / TN);  // 256

// Element (i, k) of an operand.  In the convolution view the pixel index is the row index of operand A
// (pix_is_k = false) or the reduction index of operand B (pix_is_k = true); the other index is (tap, channel).
template <typename T>
__device__ __forceinline__ float load_operand(const T* __restrict__ p, long long rs, long long ks, int i, int k,
                                              int rows, int K, bool conv, bool pix_is_k, int H, int W, int Cd, int Ct,
                                              float tau) {
    if (i >= rows || k >= K) return 0.f;
    if (!conv) return Low<T>::to_f(p[i * rs + k * ks]);
    int pixel = pix_is_k ? k : i;
    int tc = pix_is_k ? i : k;
    int tap = tc / Ct, c = tc - tap * Ct;
    int x = pixel % W;
    int y = (pixel / W) % H;
    int dy = tap / 3 - 1, dx = tap % 3 - 1;
    if (y + dy < 0 || y + dy >= H || x + dx < 0 || x + dx >= W) return 0.f;
    if (c >= Cd) return tau;
    return Low<T>::to_f(p[((long long)pixel + (long long)dy * W + dx) * Cd + c]);
}

template <typename T>
__global__ void __launch_bounds__(kGemmThreads) gemm_simt_kernel(GemmArgs g) {
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const T* A = (const T*)g.A;
    const T* B = (const T*)g.B;
    int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    int tx = threadIdx.x % (BN / TN), ty = threadIdx.x / (BN / TN);
    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

    int k_begin = 0, k_end = g.K;
    if (g.split_k > 1) {
        int chunk = ((g.K + g.split_k - 1) / g.split_k + BK - 1) / BK * BK;
        k_begin = blockIdx.z * chunk;
        k_end = min(g.K, k_begin + chunk);
    }
    // When the reduction index is the contiguous one, consecutive threads walk k; otherwise they walk rows.
    bool a_kfast = (g.conv_on == 1) || (g.a_ks == 1);
    bool b_kfast = (g.conv_on != 2) && (g.b_ks == 1);
    for (int k0 = k_begin; k0 < k_end; k0 += BK) {
#pragma unroll
        for (int it = 0; it < (BM * BK) / kGemmThreads; ++it) {
            int idx = threadIdx.x + it * kGemmThreads;
            int mm = a_kfast ? idx / BK : idx % BM;
            int kk = a_kfast ? idx % BK : idx / BM;
            int kg = k0 + kk;
            As[kk][mm] = load_operand<T>(A, g.a_rs, g.a_ks, m0 + mm, kg < k_end ? kg : g.K, g.M, g.K, g.conv_on == 1, false,
                                         g.conv_h, g.conv_w, g.conv_cd, g.conv_ct, g.conv_tau);
        }
#pragma unroll
        for (int it = 0; it < (BN * BK) / kGemmThreads; ++it) {
            int idx = threadIdx.x + it * kGemmThreads;
            int nn = b_kfast ? idx / BK : idx % BN;
            int kk = b_kfast ? idx % BK : idx / BN;
            int kg = k0 + kk;
            Bs[kk][nn] = load_operand<T>(B, g.b_rs, g.b_ks, n0 + nn, kg < k_end ? kg : g.K, g.N, g.K, g.conv_on == 2, true,
                                         g.conv_h, g.conv_w, g.conv_cd, g.conv_ct, g.conv_tau);
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[TM], b[TN];
#pragma unroll
            for (int i = 0; i < TM; ++i) a[i] = As[kk][ty * TM + i];
#pragma unroll
            for (int j = 0; j < TN; ++j) b[j] = Bs[kk][tx * TN + j];
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }

    bool bad = false;
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        int m = m0 + ty * TM + i;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            int n = n0 + tx * TN + j;
            if (m >= g.M || n >= g.N) continue;
            float v = acc[i][j];
            if (g.epi == EPI_FWD) {
                if (g.out2 != nullptr && m >= g.m_split) {
                    ((T*)g.out2)[(long long)(m - g.m_split) * g.ldo + n] = Low<T>::from_f(v);
                } else {
                    if (g.bias != nullptr) v += Low<T>::to_f(((const T*)g.bias)[n]);
                    if (g.wt != nullptr) v = fmaf(g.tau, Low<T>::to_f(((const T*)g.wt)[n]), v);
                    ((T*)g.out)[(long long)m * g.ldo + n] = Low<T>::from_f(act_fwd(g.act, v));
                }
            } else if (g.epi == EPI_DGRAD) {
                if (g.hprev != nullptr)
                    v *= act_deriv_from_output(g.act, Low<T>::to_f(((const T*)g.hprev)[(long long)m * g.ldh + n]));
                T q = Low<T>::from_f(v);
                bad |= Low<T>::nonfinite(q);
                ((T*)g.out)[(long long)m * g.ldo + n] = q;
            } else if (g.epi == EPI_WGRAD) {
                if (g.split_k > 1) {
                    g.partial[((long long)blockIdx.z * g.M + m) * g.N + n] = v;
                } else {
                    float* o = (float*)g.out + (long long)m * g.ldo + n;
                    *o = (g.beta != 0.f ? *o : 0.f) + v;
                }
            } else {
                ((float*)g.out)[(long long)m * g.ldo + n] = v;
            }
        }
    }
    if (g.epi == EPI_DGRAD) warp_flag_or(g.flag, bad);
}

__global__ void splitk_reduce_kernel(const float* __restrict__ partial, int S, int M, int N, float* __restrict__ out,
                                     long long ldo, float beta) {
    long long n_el = (long long)M * N;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n_el; i += (long long)gridDim.x * blockDim.x) {
        float s = 0.f;
        for (int z = 0; z < S; ++z) s += partial[(long long)z * n_el + i];
        float* o = out + (i / N) * ldo + (i % N);
        *o = (beta != 0.f ? *o : 0.f) + s;
    }
}

// The same four columns at a time (N, ldo multiples of 4, 16-byte aligned pointers, fewer than 2^31 elements): the slices are
// still added in ascending order per element
__global__ void splitk_reduce4_kernel(const float4* __restrict__ partial, int S, unsigned n4, unsigned N4, float* __restrict__ out,
                                      long long ldo, float beta) {
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += gridDim.x * blockDim.x) {
        float4 s = partial[i];
        for (int z = 1; z < S; ++z) {
            const float4 v = partial[(size_t)z * n4 + i];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        const unsigned row = i / N4, col = i - row * N4;
        float4* o = reinterpret_cast<float4*>(out + (long long)row * ldo) + col;
        if (beta != 0.f) {
            const float4 old = *o;
            s.x += old.x; s.y += old.y; s.z += old.z; s.w += old.w;
        }
        *o = s;
    }
}

void reduce_slices(const float* partial, int S, int M, int N, float* out, long long ldo, float beta, cudaStream_t st) {
    const long long n_el = (long long)M * N;
    if (N % 4 == 0 && ldo % 4 == 0 && n_el < 0x7fffffffLL && ((((uintptr_t)partial) | ((uintptr_t)out)) & 15) == 0 && S >= 1) {
        const unsigned n4 = (unsigned)(n_el / 4);
        int blocks = (int)((n4 + 255) / 256);
        if (blocks > 148 * 8) blocks = 148 * 8;
        splitk_reduce4_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(partial), S, n4, (unsigned)(N / 4), out, ldo, beta);
        return;
    }
    int blocks = (int)((n_el + 255) / 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    splitk_reduce_kernel<<<blocks, 256, 0, st>>>(partial, S, M, N, out, ldo, beta);
}

}  // namespace

void launch_splitk_reduce(const float* partial, int S, int M, int N, float* out, long long ldo, float beta, cudaStream_t st,
                          long long* launches) {
    reduce_slices(partial, S, M, N, out, ldo, beta, st);
    if (launches) ++*launches;
}

void launch_gemm_simt(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* launches) {
    if (g.M <= 0 || g.N <= 0) return;
    dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.split_k > 1 ? g.split_k : 1);
    if (dt == MPODE_BF16) gemm_simt_kernel<__nv_bfloat16><<<grid, kGemmThreads, 0, st>>>(g);
    else if (dt == MPODE_F16) gemm_simt_kernel<__half><<<grid, kGemmThreads, 0, st>>>(g);
    else gemm_simt_kernel<float><<<grid, kGemmThreads, 0, st>>>(g);
    if (launches) ++*launches;
    if (g.split_k > 1) {
        reduce_slices(g.partial, g.split_k, g.M, g.N, (float*)g.out, g.ldo, g.beta, st);
        if (launches) ++*launches;
    }
}

}  // namespace mpode
