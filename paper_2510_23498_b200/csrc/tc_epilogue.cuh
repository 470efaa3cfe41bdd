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

// 32 rounded columns (16 packed words) of one row to global memory: whole 32-byte sectors when the row length is a multiple of
// 16 elements and the row starts on a 32-byte boundary, else guarded 16-byte pieces (N is a multiple of 8).
template <typename T>
__device__ __forceinline__ void store_chunk(T* orow, int nb, int N, const uint32_t (&w)[16]) {
    if ((N & 15) == 0 && ((uintptr_t)orow & 31) == 0) {
#pragma unroll
        for (int v = 0; v < 2; ++v)
            if (nb + v * 16 < N)
                asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(orow + nb + v * 16), "r"(w[8 * v]), "r"(w[8 * v + 1]),
                             "r"(w[8 * v + 2]), "r"(w[8 * v + 3]), "r"(w[8 * v + 4]), "r"(w[8 * v + 5]), "r"(w[8 * v + 6]), "r"(w[8 * v + 7])
                             : "memory");
        return;
    }
#pragma unroll
    for (int v = 0; v < 4; ++v)
        if (nb + v * 8 < N) *reinterpret_cast<uint4*>(orow + nb + v * 8) = make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
}

// One 32-column chunk of one accumulator row: epilogue math, rounding, stores.  `hv`: load_h_chunk's result when
// `with_h` (input gradient through an activation).
template <typename T, int ACT, bool FWD>
__device__ __forceinline__ bool epilogue_chunk(const uint32_t (&r)[32], const float* sb, bool plain, bool with_h, const uint4 (&hv)[4],
                                               T* orow, int nb, int N, uint32_t* keep = nullptr) {
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
    store_chunk<T>(orow, nb, N, packed);
    if (keep != nullptr) {      // the rounded chunk once more, 16-byte aligned (shared memory)
#pragma unroll
        for (int v = 0; v < 4; ++v)
            *reinterpret_cast<uint4*>(keep + 4 * v) = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
    }
    return bad;
}

// Two warps that hold the two halves of a sample pair meet at a named barrier of 64 threads.
__device__ __forceinline__ void pair_sync(int id) { asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory"); }
// ... and agree on a flag: true only when it is true in all 64 threads
__device__ __forceinline__ bool pair_all(int id, bool ok) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\tbar.red.and.pred q, %2, 64, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out)
        : "r"((uint32_t)ok), "r"(id)
        : "memory");
    return out != 0;
}

// 16 rounded columns (8 packed words) of one row: one 32-byte sector when the row allows it (see store_chunk), else two pieces
template <typename T>
__device__ __forceinline__ void store_half(T* orow, int nb, int N, const uint32_t (&w)[8]) {
    if (nb >= N) return;
    if ((N & 15) == 0 && ((uintptr_t)orow & 31) == 0) {
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(orow + nb), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]),
                     "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                     : "memory");
        return;
    }
    *reinterpret_cast<uint4*>(orow + nb) = make_uint4(w[0], w[1], w[2], w[3]);
    if (nb + 8 < N) *reinterpret_cast<uint4*>(orow + nb + 8) = make_uint4(w[4], w[5], w[6], w[7]);
}

// Tangent rows of the forward pass of the flow with a trace estimate: U = Q16(acc) and, given the rounded layer output H of the
// same samples (16 packed words in shared memory), G = Q16(act'(H) * U); 16 columns at a time to keep few values live.
template <typename T, int ACT>
__device__ __forceinline__ void tangent_chunk(const uint32_t (&r)[32], const uint32_t* hw, T* urow, T* grow, int nb, int N) {
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        uint32_t pu[8], pg[8];
        uint4 hq[2];
        if (grow != nullptr) {
            hq[0] = *reinterpret_cast<const uint4*>(hw + 8 * hf);
            hq[1] = *reinterpret_cast<const uint4*>(hw + 8 * hf + 4);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t u = cvt_pack<T>(__uint_as_float(r[16 * hf + 2 * i]), __uint_as_float(r[16 * hf + 2 * i + 1]));
            pu[i] = u;
            if (grow != nullptr) {
                const uint4 q4 = hq[i >> 2];
                const uint32_t w = (i & 3) == 0 ? q4.x : ((i & 3) == 1 ? q4.y : ((i & 3) == 2 ? q4.z : q4.w));
                const float g0 = fast_act_deriv<ACT>(Low<T>::to_f(from_bits<T>((unsigned short)(w & 0xFFFFu)))) *
                                 Low<T>::to_f(from_bits<T>((unsigned short)(u & 0xFFFFu)));
                const float g1 = fast_act_deriv<ACT>(Low<T>::to_f(from_bits<T>((unsigned short)(w >> 16)))) *
                                 Low<T>::to_f(from_bits<T>((unsigned short)(u >> 16)));
                pg[i] = cvt_pack<T>(g0, g1);
            }
        }
        store_half<T>(urow, nb + 16 * hf, N, pu);
        if (grow != nullptr) store_half<T>(grow, nb + 16 * hf, N, pg);
    }
}

// Backward pass of the same flow through one activation, 16 columns: s = act'(H); the tangent rows give ubar = Q16(s gbar), the
// primal rows zeta = Q16(s hbar + s (1 - s) U gbar) (softplus: act'' = s (1 - s)).  `acc`: 16 of this row's accumulators (gbar or
// hbar), `gb`: gbar of the sample (primal rows only), `hw` / `uw`: 8 packed words of H and U, `out`: 8 packed results.
// Returns whether a rounded value is not finite.
template <typename T, int ACT, int HF>
__device__ __forceinline__ bool cnf_backward_half(const uint32_t (&r)[32], bool tangent, const float (&gb)[16], const uint4 (&hv)[4],
                                                  const uint4 (&uv)[4], uint32_t (&packed)[16], int nb, int N) {
    const float lim = OverflowLimit<T>::value();
    bool bad = false;
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        const int word = 8 * HF + (i >> 1);       // packed word of the chunk: uint4 number word / 4, component word % 4
        const uint4 hq = hv[word >> 2], uq = uv[word >> 2];
        const uint32_t w = (word & 3) == 0 ? hq.x : ((word & 3) == 1 ? hq.y : ((word & 3) == 2 ? hq.z : hq.w));
        const float s0 = fast_act_deriv<ACT>(Low<T>::to_f(from_bits<T>((unsigned short)(w & 0xFFFFu))));
        const float s1 = fast_act_deriv<ACT>(Low<T>::to_f(from_bits<T>((unsigned short)(w >> 16))));
        float v0 = __uint_as_float(r[16 * HF + i]), v1 = __uint_as_float(r[16 * HF + i + 1]);
        if (tangent) {
            v0 *= s0;
            v1 *= s1;
        } else {
            const uint32_t u = (word & 3) == 0 ? uq.x : ((word & 3) == 1 ? uq.y : ((word & 3) == 2 ? uq.z : uq.w));
            v0 = s0 * v0 + s0 * (1.f - s0) * Low<T>::to_f(from_bits<T>((unsigned short)(u & 0xFFFFu))) * gb[i];
            v1 = s1 * v1 + s1 * (1.f - s1) * Low<T>::to_f(from_bits<T>((unsigned short)(u >> 16))) * gb[i + 1];
        }
        bad |= (nb + 16 * HF + i < N) && !(fabsf(v0) < lim);
        bad |= (nb + 16 * HF + i + 1 < N) && !(fabsf(v1) < lim);
        packed[word] = cvt_pack<T>(v0, v1);
    }
    return bad;
}

}  // namespace tc
}  // namespace mpode
