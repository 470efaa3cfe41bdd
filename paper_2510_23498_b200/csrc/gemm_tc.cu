// Velocity-layer contractions on the 5th-generation tensor cores (sm_100a): C[M, N] = A[M, K] * B[N, K]^T with both
// operands K-major in global memory, fp32 accumulation in tensor memory, and the layer epilogue fused:
//   forward  : out = Q16(act(acc + b + tau * w_t))                      (Alg. 1 increment, one rounding per layer)
//   backward : out = Q16(act'(H_prev) * acc), non-finite outputs flagged (Eq. (vjp), Alg. 2 finiteness test)
//
// Persistent, warp-specialised CTA (one per SM): warp 0 issues TMA tile loads into a ring of 128B-swizzled
// shared-memory stages, warp 1 issues tcgen05.mma (128 x BN x 16 per instruction) into one of two TMEM
// accumulators, warps 2..9 drain the other accumulator with tcgen05.ld and run the epilogue, so the epilogue of
// tile i overlaps the main loop of tile i+1.  Every mbarrier wait is bounded in time; a wait that gives up sets an
// error word and the kernel winds down without trapping.
#include <cuda.h>

#include <mutex>
#include <unordered_map>

#include "common.cuh"
#include "gemm_tc.h"

namespace mpode {
namespace {

constexpr int BM = 128;
constexpr int BK = 64;                 // 64 16-bit elements = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int kEpiWarps = 8;           // two warps per TMEM lane quadrant, each takes half of the columns
constexpr int kThreadsTc = 64 + 32 * kEpiWarps;   // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue
constexpr int kSmemBudget = 196608;    // bytes of operand stages
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct TcParams {
    int M, N, K;
    int epi;
    void* out; long long ldo;
    void* out2; int m_split;
    const void* bias; const void* wt; float tau; int act;
    const void* hprev; long long ldh;
    unsigned* flag;
    unsigned* err;
    int tiles_m, tiles_n;
    int splits, kb_per_split;   // weight-gradient kernels: the reduction (batch) range is cut into `splits` slices
    float* partial;             // [splits][M][N] fp32 partial sums of the slices
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kWaitLimitNs, records `code` in *err and returns false.
__device__ __noinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned* err, unsigned code) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = globaltimer_ns();
    unsigned it = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++it & 255u) == 0u) {
            if (globaltimer_ns() - t0 > kWaitLimitNs || *(volatile unsigned*)err != 0u) {
                atomicOr(err, code);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap* tmap, uint64_t* bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst_smem), "l"((unsigned long long)tmap), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t* holder_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(holder_smem)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives on the mbarrier once all tcgen05.mma issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives row (lane base + i)
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile stored as rows of 128 bytes with the 128-byte swizzle:
// 8-row groups are 1024 bytes apart (stride byte offset), the leading byte offset is unused for swizzled K-major
// tiles (encoded 1), descriptor version 1, layout type 2 (SWIZZLE_128B).  Addresses are in units of 16 bytes.
__device__ __forceinline__ uint64_t smem_desc_k_major_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
    d |= (uint64_t)1u << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1u << 46;
    d |= (uint64_t)2u << 61;
    return d;
}

// The same for an MN-major operand tile (the reduction index is the row index in memory): every 64-element chunk
// of the M/N extent is one [64 reduction rows][128 bytes] swizzled block of 8192 bytes; chunks are 8192 bytes apart
// (leading byte offset), 8-row groups of the reduction index 1024 bytes apart (stride byte offset).
__device__ __forceinline__ uint64_t smem_desc_mn_major_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
    d |= (uint64_t)(8192u >> 4) << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1u << 46;
    d |= (uint64_t)2u << 61;
    return d;
}

// Instruction descriptor of kind::f16: fp32 accumulator, A and B of the same 16-bit format; bit 15 / 16 select the
// MN-major (transposed) form of A / B.
__host__ __device__ constexpr uint32_t make_idesc(int fmt /*0 f16, 1 bf16*/, int m, int n, bool mn_major) {
    return (1u << 4) | ((uint32_t)fmt << 7) | ((uint32_t)fmt << 10) | ((mn_major ? 3u : 0u) << 15) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

template <typename T> struct Fmt;
template <> struct Fmt<__half> { static constexpr int id = 0; };
template <> struct Fmt<__nv_bfloat16> { static constexpr int id = 1; };

template <typename T> __device__ __forceinline__ uint32_t pack2(T a, T b);
template <> __device__ __forceinline__ uint32_t pack2<__half>(__half a, __half b) {
    return (uint32_t)__half_as_ushort(a) | ((uint32_t)__half_as_ushort(b) << 16);
}
template <> __device__ __forceinline__ uint32_t pack2<__nv_bfloat16>(__nv_bfloat16 a, __nv_bfloat16 b) {
    return (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
}
template <typename T> __device__ __forceinline__ T from_bits(unsigned short u);
template <> __device__ __forceinline__ __half from_bits<__half>(unsigned short u) { return __ushort_as_half(u); }
template <> __device__ __forceinline__ __nv_bfloat16 from_bits<__nv_bfloat16>(unsigned short u) { return __ushort_as_bfloat16(u); }

// Packed round-to-nearest-even conversion of two floats (one cvt instruction).
template <typename T> __device__ __forceinline__ uint32_t cvt_pack(float a, float b);
template <> __device__ __forceinline__ uint32_t cvt_pack<__half>(float a, float b) {
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
template <> __device__ __forceinline__ uint32_t cvt_pack<__nv_bfloat16>(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
// |v| at or above this rounds to Inf in the low format (largest finite value plus half a unit in the last place);
// the comparison is false for NaN, so !(|v| < limit) is exactly "Q16(v) is not finite".
template <typename T> struct OverflowLimit;
template <> struct OverflowLimit<__half> { static __device__ __forceinline__ float value() { return 65520.f; } };
template <> struct OverflowLimit<__nv_bfloat16> { static __device__ __forceinline__ float value() { return __uint_as_float(0x7F7F8000u); } };

// Activations for the tensor-core epilogue: one MUFU (ex2) per element plus FMA-pipe polynomials, fp32-accurate.
//   softplus(z) = max(z, 0) + log1p(t), t = exp(-|z|) in (0, 1]; log1p(t) = t * P8(t), |rel. err| < 2e-7
//   softplus'   = 1 - exp(-H) from the stored output H (Taylor series below 1/8, where the difference cancels)
template <int ACT> __device__ __forceinline__ float fast_act(float z) {
    if (ACT == MPODE_ACT_SOFTPLUS) {
        float t = __expf(-fabsf(z));
        float p = 5.253457796e-03f;
        p = fmaf(p, t, -2.958850739e-02f);
        p = fmaf(p, t, 7.836166801e-02f);
        p = fmaf(p, t, -1.367476971e-01f);
        p = fmaf(p, t, 1.911143108e-01f);
        p = fmaf(p, t, -2.484436989e-01f);
        p = fmaf(p, t, 3.331927134e-01f);
        p = fmaf(p, t, -4.999950152e-01f);
        p = fmaf(p, t, 9.999999705e-01f);
        return fmaf(t, p, fmaxf(z, 0.f));
    }
    if (ACT == MPODE_ACT_RELU) return fmaxf(z, 0.f);
    if (ACT == MPODE_ACT_TANH) return tanhf(z);
    return z;
}
template <int ACT> __device__ __forceinline__ float fast_act_deriv(float h) {
    if (ACT == MPODE_ACT_SOFTPLUS) {
        float big = 1.f - __expf(-h);
        float small = h * fmaf(h, fmaf(h, fmaf(h, fmaf(h, -1.f / 120.f, 1.f / 24.f), -1.f / 6.f), 0.5f) * -1.f, 1.f);
        return h < 0.125f ? small : big;
    }
    if (ACT == MPODE_ACT_RELU) return h > 0.f ? 1.f : 0.f;
    if (ACT == MPODE_ACT_TANH) return fmaf(-h, h, 1.f);
    return 1.f;
}

// One 32-column chunk of one accumulator row: epilogue math, rounding, 16-byte stores.
template <typename T, int ACT, bool FWD>
__device__ __forceinline__ bool epilogue_chunk(const uint32_t (&r)[32], const float* sb, bool plain, const T* hrow, T* orow,
                                               int nb, int N) {
    uint32_t packed[16];
    bool bad = false;
    if (FWD) {
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
            float v0 = __uint_as_float(r[i]), v1 = __uint_as_float(r[i + 1]);
            if (!plain) {
                v0 = fast_act<ACT>(v0 + sb[i]);
                v1 = fast_act<ACT>(v1 + sb[i + 1]);
            }
            packed[i >> 1] = cvt_pack<T>(v0, v1);
        }
    } else {
        uint4 hv[4];
        if (hrow != nullptr) {
#pragma unroll
            for (int v = 0; v < 4; ++v)
                hv[v] = (nb + v * 8 < N) ? *reinterpret_cast<const uint4*>(hrow + nb + v * 8) : make_uint4(0, 0, 0, 0);
        }
        const uint32_t* hw = reinterpret_cast<const uint32_t*>(hv);
        const float lim = OverflowLimit<T>::value();
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
            float v0 = __uint_as_float(r[i]), v1 = __uint_as_float(r[i + 1]);
            if (hrow != nullptr) {
                uint32_t w = hw[i >> 1];
                v0 *= fast_act_deriv<ACT>(Low<T>::to_f(from_bits<T>((unsigned short)(w & 0xFFFFu))));
                v1 *= fast_act_deriv<ACT>(Low<T>::to_f(from_bits<T>((unsigned short)(w >> 16))));
            }
            bad |= (nb + i < N) && !(fabsf(v0) < lim);
            bad |= (nb + i + 1 < N) && !(fabsf(v1) < lim);
            packed[i >> 1] = cvt_pack<T>(v0, v1);
        }
    }
#pragma unroll
    for (int v = 0; v < 4; ++v) {
        if (nb + v * 8 < N)   // N is a multiple of 8: whole 16-byte groups are in or out
            *reinterpret_cast<uint4*>(orow + nb + v * 8) = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
    }
    return bad;
}

template <int BN> struct TileCfg {
    static constexpr int kStageBytes = BM * BK * 2 + BN * BK * 2;
    static constexpr int kStages = kSmemBudget / kStageBytes;
    static constexpr int kTmemCols = 2 * BN;            // two accumulators; 128, 256 or 512 columns (powers of two)
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 4 * BN * 4 /*bias, one copy per epilogue warp*/ + 256 /*barriers*/;
};

// WG = false: C[M, N] = A[M, K] B[N, K]^T, operands K-major in memory, low-format output with fused epilogue.
// WG = true : C[M, N] = sum_r A[r, M] B[r, N] (weight gradient: the reduction index r runs over the batch rows of two
//             row-major activations), fp32 partial sums per reduction slice, reduced afterwards in a fixed order.
template <typename T, int BN, bool WG>
__global__ void __launch_bounds__(kThreadsTc, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, TcParams p) {
    using Cfg = TileCfg<BN>;
    constexpr int S = Cfg::kStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;                                   // S stages of [128][64] 16-bit
    uint8_t* sB = smem + (size_t)S * BM * BK * 2;         // S stages of [BN][64] 16-bit
    float* sbias = (float*)(smem + (size_t)S * Cfg::kStageBytes);   // [4 epilogue warps][BN]
    uint64_t* bars = (uint64_t*)(sbias + 4 * BN);
    uint64_t* full_bar = bars;                // [S]
    uint64_t* empty_bar = bars + S;           // [S]
    uint64_t* tfull_bar = bars + 2 * S;       // [2]
    uint64_t* tempty_bar = bars + 2 * S + 2;  // [2]
    uint32_t* tmem_holder = (uint32_t*)(bars + 2 * S + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int n_work = n_tiles * p.splits;
    const int kb_total = (p.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&tfull_bar[a], 1); mbar_init(&tempty_bar[a], kEpiWarps); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_holder, Cfg::kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *(volatile uint32_t*)tmem_holder;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < n_work && ok; w += gridDim.x) {
                const int tile = w % n_tiles, z = w / n_tiles;
                const int m0 = (tile / p.tiles_n) * BM, n0 = (tile % p.tiles_n) * BN;
                const int kb0 = z * p.kb_per_split, kb1 = min(kb_total, kb0 + p.kb_per_split);
                for (int kb = kb0; kb < kb1; ++kb) {
                    ok = mbar_wait(&empty_bar[s], phase ^ 1u, p.err, 1u);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&full_bar[s], (uint32_t)Cfg::kStageBytes);
                    const uint32_t a_dst = smem_u32(sA + (size_t)s * BM * BK * 2), b_dst = smem_u32(sB + (size_t)s * BN * BK * 2);
                    if (!WG) {
                        tma_load_2d(a_dst, &tmA, &full_bar[s], kb * BK, m0);
                        tma_load_2d(b_dst, &tmB, &full_bar[s], kb * BK, n0);
                    } else {
                        // [64 reduction rows][64 columns] boxes, one per 64-wide chunk of the tile's M / N extent
#pragma unroll
                        for (int c = 0; c < BM / 64; ++c) tma_load_2d(a_dst + c * 8192, &tmA, &full_bar[s], m0 + c * 64, kb * BK);
#pragma unroll
                        for (int c = 0; c < BN / 64; ++c) tma_load_2d(b_dst + c * 8192, &tmB, &full_bar[s], n0 + c * 64, kb * BK);
                    }
                    if (++s == S) { s = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(Fmt<T>::id, BM, BN, WG);
            int s = 0;
            uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < n_work && ok; w += gridDim.x, ++it) {
                const int acc = it & 1;
                const uint32_t use = (uint32_t)(it >> 1);
                const int z = w / n_tiles;
                const int kb0 = z * p.kb_per_split, kb1 = min(kb_total, kb0 + p.kb_per_split);
                ok = mbar_wait(&tempty_bar[acc], (use & 1u) ^ 1u, p.err, 2u);      // epilogue has drained this accumulator
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BN);
                for (int kb = kb0; kb < kb1; ++kb) {
                    ok = mbar_wait(&full_bar[s], phase, p.err, 4u);                // TMA bytes have landed
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(sA + (size_t)s * BM * BK * 2), b_addr = smem_u32(sB + (size_t)s * BN * BK * 2);
                    const uint64_t adesc = WG ? smem_desc_mn_major_sw128(a_addr) : smem_desc_k_major_sw128(a_addr);
                    const uint64_t bdesc = WG ? smem_desc_mn_major_sw128(b_addr) : smem_desc_k_major_sw128(b_addr);
                    // one instruction consumes 16 reduction elements: 32 bytes along a K-major swizzled row (+2 in
                    // 16-byte units), or 16 rows of 128 bytes of an MN-major block (+128)
                    constexpr uint64_t kstep = WG ? 128u : 2u;
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        umma_f16(tmem_d, adesc + kstep * (uint64_t)k, bdesc + kstep * (uint64_t)k, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
                    umma_commit(&empty_bar[s]);                                    // stage reusable once these MMAs retire
                    if (++s == S) { s = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit(&tfull_bar[acc]);                                      // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        // hardware rule: a warp reads the TMEM lanes [32 * (warp % 4), +32); the two warps of a quadrant split the columns
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        constexpr int kColsPerWarp = BN / 2;
        float* sb_warp = sbias + (warp - 2) * kColsPerWarp;   // this warp's slice of the effective bias b + tau * w_t
        bool bad = false;
        bool ok = true;
        int it = 0;
        for (int w = blockIdx.x; w < n_work && ok; w += gridDim.x, ++it) {
            const int acc = it & 1;
            const uint32_t use = (uint32_t)(it >> 1);
            const int tile = w % n_tiles, z = w / n_tiles;
            const int m0 = (tile / p.tiles_n) * BM, n0 = (tile % p.tiles_n) * BN + half * kColsPerWarp;
            if (!WG && p.epi == EPI_FWD) {
                for (int c = lane; c < kColsPerWarp; c += 32) {
                    int n = n0 + c;
                    float b = 0.f;
                    if (n < p.N) {
                        if (p.bias != nullptr) b = Low<T>::to_f(((const T*)p.bias)[n]);
                        if (p.wt != nullptr) b = fmaf(p.tau, Low<T>::to_f(((const T*)p.wt)[n]), b);
                    }
                    sb_warp[c] = b;
                }
                __syncwarp();
            }
            ok = mbar_wait(&tfull_bar[acc], use & 1u, p.err, 8u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const int m = m0 + q * 32 + lane;
            const bool row_ok = m < p.M;
            const bool second = (p.out2 != nullptr) && (m >= p.m_split);
            T* orow = second ? (T*)p.out2 + (long long)(m - p.m_split) * p.ldo : (T*)p.out + (long long)m * p.ldo;
            const T* hrow = (p.hprev != nullptr) ? (const T*)p.hprev + (long long)m * p.ldh : nullptr;
            const uint32_t tcol = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + half * kColsPerWarp);
#pragma unroll 1
            for (int c = 0; c < kColsPerWarp / 32; ++c) {
                uint32_t r[32];
                __syncwarp();   // tcgen05.ld is warp-collective: reconverge after the guarded body of the last chunk
                tmem_ld_32x32(tcol + (uint32_t)(c * 32), r);
                const int nb = n0 + c * 32;
                if (WG) {
                    if (row_ok && nb < p.N) {
                        float* prow = p.partial + ((long long)z * p.M + m) * p.N + nb;
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            if (nb + v * 4 < p.N)   // N is a multiple of 8
                                *reinterpret_cast<uint4*>(prow + v * 4) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                    }
                } else if (row_ok && nb < p.N) {
                    const float* sb = sb_warp + c * 32;
                    if (p.epi == EPI_FWD) {
                        switch (p.act) {
                            case MPODE_ACT_SOFTPLUS: epilogue_chunk<T, MPODE_ACT_SOFTPLUS, true>(r, sb, second, nullptr, orow, nb, p.N); break;
                            case MPODE_ACT_RELU: epilogue_chunk<T, MPODE_ACT_RELU, true>(r, sb, second, nullptr, orow, nb, p.N); break;
                            case MPODE_ACT_TANH: epilogue_chunk<T, MPODE_ACT_TANH, true>(r, sb, second, nullptr, orow, nb, p.N); break;
                            default: epilogue_chunk<T, MPODE_ACT_NONE, true>(r, sb, second, nullptr, orow, nb, p.N); break;
                        }
                    } else {
                        switch (p.act) {
                            case MPODE_ACT_SOFTPLUS: bad |= epilogue_chunk<T, MPODE_ACT_SOFTPLUS, false>(r, sb, false, hrow, orow, nb, p.N); break;
                            case MPODE_ACT_RELU: bad |= epilogue_chunk<T, MPODE_ACT_RELU, false>(r, sb, false, hrow, orow, nb, p.N); break;
                            case MPODE_ACT_TANH: bad |= epilogue_chunk<T, MPODE_ACT_TANH, false>(r, sb, false, hrow, orow, nb, p.N); break;
                            default: bad |= epilogue_chunk<T, MPODE_ACT_NONE, false>(r, sb, false, hrow, orow, nb, p.N); break;
                        }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tempty_bar[acc]);
        }
        if (!WG && p.epi == EPI_DGRAD) warp_flag_or(p.flag, bad);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

// ---------------------------------------------------------------- host side: tensor maps and launch
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

struct MapKey {
    const void* ptr; long long rows, cols, ld; int box_rows, dt;
    bool operator==(const MapKey& o) const {
        return ptr == o.ptr && rows == o.rows && cols == o.cols && ld == o.ld && box_rows == o.box_rows && dt == o.dt;
    }
};
struct MapKeyHash {
    size_t operator()(const MapKey& k) const {
        size_t h = (size_t)k.ptr;
        h = h * 1000003u ^ (size_t)k.rows;
        h = h * 1000003u ^ (size_t)k.cols;
        h = h * 1000003u ^ (size_t)k.ld;
        h = h * 1000003u ^ (size_t)(k.box_rows * 4 + k.dt);
        return h;
    }
};

// Tensor map of a row-major [rows, cols] 16-bit matrix with row stride ld (elements), box = [box_rows, 64 columns],
// 128-byte swizzle, out-of-range elements read as zero.  (Weight-gradient operands use box_rows = 64: the box is
// [64 reduction rows][64 columns].)
bool get_tensor_map(const void* ptr, long long rows, long long cols, long long ld, int box_rows, mpode_dtype dt,
                    CUtensorMap* out) {
    static std::mutex mu;
    static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
    MapKey key{ptr, rows, cols, ld, box_rows, (int)dt};
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find(key);
    if (it != cache.end()) { *out = it->second; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstr[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUtensorMap m;
    CUresult r = fn(&m, dt == MPODE_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2,
                    const_cast<void*>(ptr), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (cache.size() > 4096) cache.clear();
    cache.emplace(key, m);
    *out = m;
    return true;
}

int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

template <typename T, int BN, bool WG>
bool launch_tc(const CUtensorMap& ta, const CUtensorMap& tb, TcParams& p, cudaStream_t st) {
    using Cfg = TileCfg<BN>;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(gemm_tc_kernel<T, BN, WG>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess)
            return false;
        attr_set = true;
    }
    p.tiles_m = (p.M + BM - 1) / BM;
    p.tiles_n = (p.N + BN - 1) / BN;
    int work = p.tiles_m * p.tiles_n * p.splits;
    int grid = work < sm_count() ? work : sm_count();
    gemm_tc_kernel<T, BN, WG><<<grid, kThreadsTc, Cfg::kSmemBytes, st>>>(ta, tb, p);
    return true;
}

}  // namespace

bool tc_eligible(mpode_dtype dt, const GemmArgs& g) {
    if (dt != MPODE_BF16 && dt != MPODE_F16) return false;
    if (g.epi != EPI_FWD && g.epi != EPI_DGRAD) return false;
    if (g.conv_on != 0 || g.split_k > 1) return false;
    if (g.a_ks != 1 || g.b_ks != 1) return false;
    if (g.K % 8 != 0 || g.N % 8 != 0 || g.a_rs % 8 != 0 || g.b_rs % 8 != 0 || g.ldo % 8 != 0) return false;
    if (g.hprev != nullptr && g.ldh % 8 != 0) return false;
    if (((uintptr_t)g.A | (uintptr_t)g.B | (uintptr_t)g.out | (uintptr_t)g.out2 | (uintptr_t)g.hprev) & 15) return false;
    if (g.M < 128 || g.N < 64 || g.K < 64) return false;  // tiny problems stay on the CUDA cores
    if (g.err == nullptr) return false;
    return true;
}

bool launch_gemm_tc(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* launches) {
    int bn = 256;
    // narrow outputs: smaller tiles keep more SMs busy
    long long tiles256 = (long long)((g.M + BM - 1) / BM) * ((g.N + 255) / 256);
    if (g.N <= 64) bn = 64;
    else if (g.N <= 128 || tiles256 < sm_count()) bn = 128;
    if (bn == 128 && g.N > 64 && (long long)((g.M + BM - 1) / BM) * ((g.N + 127) / 128) < sm_count() / 2) bn = 64;
    CUtensorMap ta, tb;
    if (!get_tensor_map(g.A, g.M, g.K, g.a_rs, BM, dt, &ta)) return false;
    if (!get_tensor_map(g.B, g.N, g.K, g.b_rs, bn, dt, &tb)) return false;
    TcParams p{};
    p.M = g.M; p.N = g.N; p.K = g.K; p.epi = g.epi;
    p.out = g.out; p.ldo = g.ldo; p.out2 = g.out2; p.m_split = g.m_split;
    p.bias = g.bias; p.wt = g.wt; p.tau = g.tau; p.act = g.act;
    p.hprev = g.hprev; p.ldh = g.ldh; p.flag = g.flag; p.err = g.err;
    p.splits = 1; p.kb_per_split = (g.K + BK - 1) / BK; p.partial = nullptr;
    bool ok;
    if (dt == MPODE_BF16) {
        ok = bn == 256 ? launch_tc<__nv_bfloat16, 256, false>(ta, tb, p, st)
           : bn == 128 ? launch_tc<__nv_bfloat16, 128, false>(ta, tb, p, st) : launch_tc<__nv_bfloat16, 64, false>(ta, tb, p, st);
    } else {
        ok = bn == 256 ? launch_tc<__half, 256, false>(ta, tb, p, st)
           : bn == 128 ? launch_tc<__half, 128, false>(ta, tb, p, st) : launch_tc<__half, 64, false>(ta, tb, p, st);
    }
    if (ok && launches) ++*launches;
    return ok;
}

// ---------------------------------------------------------------- weight gradient
// How the reduction range is sliced so that tiles x slices fills the SMs (few waves, little partial-sum traffic).
static void wgrad_plan(int M, int N, int K, int* bn_out, int* splits_out, int* kb_per_split_out) {
    int bn = N >= 256 ? 256 : (N >= 128 ? 128 : 64);
    int tiles = ((M + BM - 1) / BM) * ((N + bn - 1) / bn);
    int kb_total = (K + BK - 1) / BK;
    int sms = 148;
    int best = 1;
    double best_score = -1.0;
    for (int s = 1; s <= 16 && s <= kb_total; ++s) {
        int work = tiles * s;
        double eff = (double)work / (double)(((work + sms - 1) / sms) * sms);
        double score = eff - 0.012 * s;
        if (score > best_score) { best_score = score; best = s; }
    }
    int per = (kb_total + best - 1) / best;
    *bn_out = bn;
    *kb_per_split_out = per;
    *splits_out = (kb_total + per - 1) / per;
}

size_t wgrad_tc_scratch_bytes(int M, int N, int K) {
    int bn, splits, per;
    wgrad_plan(M, N, K, &bn, &splits, &per);
    return (size_t)splits * M * N * sizeof(float);
}

bool wgrad_tc_eligible(mpode_dtype dt, const GemmArgs& g) {
    if (dt != MPODE_BF16 && dt != MPODE_F16) return false;
    if (g.epi != EPI_WGRAD || g.conv_on != 0 || g.split_k > 1) return false;
    if (g.a_rs != 1 || g.b_rs != 1) return false;                       // operands are [reduction rows, M] and [rows, N]
    if (g.M % 8 != 0 || g.N % 8 != 0 || g.a_ks % 8 != 0 || g.b_ks % 8 != 0) return false;
    if (((uintptr_t)g.A | (uintptr_t)g.B | (uintptr_t)g.partial) & 15) return false;
    if (g.M < 64 || g.N < 64 || g.K < 128) return false;
    if (g.err == nullptr || g.partial == nullptr) return false;
    return true;
}

void launch_splitk_reduce(const float* partial, int S, int M, int N, float* out, long long ldo, float beta, cudaStream_t st,
                          long long* launches);   // gemm_simt.cu

bool launch_wgrad_tc(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* launches) {
    int bn, splits, per;
    wgrad_plan(g.M, g.N, g.K, &bn, &splits, &per);
    CUtensorMap ta, tb;
    if (!get_tensor_map(g.A, g.K, g.M, g.a_ks, 64, dt, &ta)) return false;
    if (!get_tensor_map(g.B, g.K, g.N, g.b_ks, 64, dt, &tb)) return false;
    TcParams p{};
    p.M = g.M; p.N = g.N; p.K = g.K; p.epi = EPI_WGRAD; p.err = g.err;
    p.splits = splits; p.kb_per_split = per; p.partial = g.partial;
    bool ok;
    if (dt == MPODE_BF16) {
        ok = bn == 256 ? launch_tc<__nv_bfloat16, 256, true>(ta, tb, p, st)
           : bn == 128 ? launch_tc<__nv_bfloat16, 128, true>(ta, tb, p, st) : launch_tc<__nv_bfloat16, 64, true>(ta, tb, p, st);
    } else {
        ok = bn == 256 ? launch_tc<__half, 256, true>(ta, tb, p, st)
           : bn == 128 ? launch_tc<__half, 128, true>(ta, tb, p, st) : launch_tc<__half, 64, true>(ta, tb, p, st);
    }
    if (!ok) return false;
    if (launches) ++*launches;
    launch_splitk_reduce(g.partial, splits, g.M, g.N, (float*)g.out, g.ldo, g.beta, st, launches);
    return true;
}

}  // namespace mpode
