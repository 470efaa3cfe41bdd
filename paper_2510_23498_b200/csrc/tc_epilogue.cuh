// Epilogue arithmetic shared by the tensor-core kernels that write a low-format layer output: one 32-column chunk of one
// accumulator row (the 32 registers a tcgen05.ld 32x32b.x32 gives a lane).
#pragma once
#include "common.cuh"
#include "tc_ptx.cuh"

namespace mpode {
namespace tc {

// The stored layer output that multiplies a 32-column chunk of an input gradient (zero beyond column N): issued before the
// accumulator is waited for, so that its latency hides behind the MMAs.
template <typename T>
__device__ __forceinline__ void load_h_chunk(const T* hrow, int nb, int N, uint4 (&hv)[4]) {
#pragma unroll
    for (int v = 0; v < 4; ++v)
        hv[v] = (hrow != nullptr && nb + v * 8 < N) ? *reinterpret_cast<const uint4*>(hrow + nb + v * 8) : make_uint4(0, 0, 0, 0);
}

// One 32-column chunk of one accumulator row: epilogue math, rounding, 16-byte stores.  `hv`: load_h_chunk's result when
// `with_h` (input gradient through an activation).
template <typename T, int ACT, bool FWD>
__device__ __forceinline__ bool epilogue_chunk(const uint32_t (&r)[32], const float* sb, bool plain, bool with_h, const uint4 (&hv)[4],
                                               T* orow, int nb, int N) {
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
        const uint32_t* hw = reinterpret_cast<const uint32_t*>(hv);
        const float lim = OverflowLimit<T>::value();
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
            float v0 = __uint_as_float(r[i]), v1 = __uint_as_float(r[i + 1]);
            if (with_h) {
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

}  // namespace tc
}  // namespace mpode
