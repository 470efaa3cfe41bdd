// Inline-PTX wrappers and small device helpers shared by the tensor-core kernels (sm_100a): mbarriers with bounded
// waits, TMA tile loads, tcgen05 (TMEM allocation, MMA issue, commit, accumulator loads), shared-memory matrix
// descriptors, packed 16-bit conversions and the epilogue activations.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace mpode {
namespace tc {

constexpr int BM = 128;                // rows of one output tile = TMEM lanes
constexpr int BK = 64;                 // 64 16-bit elements = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

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
// Bounded wait: gives up after `limit_ns`, records `code` in *err and returns false.
static __device__ __noinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned* err, unsigned code,
                                              unsigned long long limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = globaltimer_ns();
    unsigned it = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++it & 255u) == 0u) {
            if (globaltimer_ns() - t0 > limit_ns || *(volatile unsigned*)err != 0u) {
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

// 32 lanes x 16 consecutive fp32 columns
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 2^x, flushing subnormal inputs and results to zero (one MUFU instruction, no range fix-up)
__device__ __forceinline__ float ex2_ftz(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
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

// Activations for the tensor-core epilogue: one MUFU (ex2) per element plus a short FMA-pipe polynomial.  The results
// are rounded to a 16-bit format next (unit roundoff 2^-8 or 2^-11), so a relative error near 1e-5 is invisible.
//   softplus(z) = max(z, 0) + log1p(t), t = exp(-|z|) in (0, 1]; log1p(t) = t * P5(t), |rel. err| < 9e-6
//   softplus'   = 1 - exp(-H) from the stored output H >= 0 (three Taylor terms below 1/32, where the difference cancels)
template <int ACT> __device__ __forceinline__ float fast_act(float z) {
    if (ACT == MPODE_ACT_SOFTPLUS) {
        float t = ex2_ftz(-1.4426950408889634f * fabsf(z));
        float p = -2.3869069e-02f;
        p = fmaf(p, t, 1.0122208e-01f);
        p = fmaf(p, t, -2.1004850e-01f);
        p = fmaf(p, t, 3.2520661e-01f);
        p = fmaf(p, t, -4.9936137e-01f);
        p = fmaf(p, t, 9.9999160e-01f);
        return fmaf(t, p, fmaxf(z, 0.f));
    }
    if (ACT == MPODE_ACT_RELU) return fmaxf(z, 0.f);
    if (ACT == MPODE_ACT_TANH) return tanhf(z);
    return z;
}
template <int ACT> __device__ __forceinline__ float fast_act_deriv(float h) {
    if (ACT == MPODE_ACT_SOFTPLUS) {
        float big = 1.f - ex2_ftz(-1.4426950408889634f * h);
        float small = h * fmaf(h, fmaf(h, 1.f / 6.f, -0.5f), 1.f);
        return h < 0.03125f ? small : big;
    }
    if (ACT == MPODE_ACT_RELU) return h > 0.f ? 1.f : 0.f;
    if (ACT == MPODE_ACT_TANH) return fmaf(-h, h, 1.f);
    return 1.f;
}

// ---------------------------------------------------------------- cross-CTA hand-off through global memory
// Data one CTA stores and another CTA's TMA unit reads: the writer runs writer_publish_fence() after its stores and
// before it releases the counter; the reader acquires the counter and runs reader_consume_fence() before it issues
// the bulk loads (ordering between the generic and the asynchronous proxy on both sides).
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_gpu_add(unsigned* p, unsigned v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded wait until *counter >= target; gives up after `limit_ns` (or when another wait already failed), records
// `code` in *err and returns false.
static __device__ __noinline__ bool wait_counter_ge(const unsigned* counter, unsigned target, unsigned* err, unsigned code,
                                                    unsigned long long limit_ns = kWaitLimitNs) {
    if (ld_acquire_gpu(counter) >= target) return true;
    unsigned long long t0 = globaltimer_ns();
    unsigned it = 0;
    while (true) {
        if (ld_acquire_gpu(counter) >= target) return true;
        __nanosleep(64);
        if ((++it & 63u) == 0u) {
            if (globaltimer_ns() - t0 > limit_ns || *(volatile unsigned*)err != 0u) {
                atomicOr(err, code);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst_smem, const CUtensorMap* tmap, uint64_t* bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst_smem), "l"((unsigned long long)tmap), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst_smem, const CUtensorMap* tmap, uint64_t* bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst_smem), "l"((unsigned long long)tmap), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)tmap) : "memory");
}

}  // namespace tc
}  // namespace mpode
