// 3x3 convolution (stride 1, zero padding 1) of an NHWC image with 64 input and 64 output channels on the 5th-generation
// tensor cores, as an implicit contraction that fetches every operand ONCE per output tile:
//   * the nine 64 x 64 weight tiles stay in shared memory for the life of the CTA (72 KB), laid out so that the three horizontal
//     taps of one stencil row form one 192-row B operand;
//   * an output tile is 128 pixels = R whole image rows of width W <= 32.  One 4-D bulk tensor load brings the R + 2 rows around
//     the tile as (R + 2) * W consecutive 128-byte rows (rows outside the image read as zero = the padding).  The three vertical
//     taps are three groups of MMAs whose A descriptors start W rows apart inside that block (W * 128 bytes is a multiple of the
//     1024-byte swizzle period, so the shifted views see the swizzle phase the load wrote);
//   * the horizontal taps are not loaded at all: every MMA has N = 192 = (dx, cout), i.e. the accumulator holds, per pixel, the
//     three partial sums P_dx over (dy, cin), and the epilogue adds P_-1 of the left neighbour, P_0 and P_+1 of the right
//     neighbour.  A warp's 32 TMEM lanes are whole image rows, so the neighbours are lanes of the same warp (two shuffles per
//     value), and the image border is a lane mask.
// Per tile that is one load of (R + 2) / R * 16 KB and 12 MMAs of 128 x 192 x 16, where the tap-by-tap form needs nine loads of
// 16 KB plus nine weight tiles and 36 MMAs of 128 x 64 x 16 (which shared-memory bandwidth, not the tensor pipe, paces).
//
// Persistent warp-specialised CTA, one per SM: warp 0 issues the loads, warp 1 the tcgen05.mma instructions into one of two
// TMEM accumulators (128 lanes x 192 columns), warps 2..17 drain finished accumulators (tcgen05.ld) and run the layer epilogue of
// the forward pass (position-class bias, activation, rounding) or of the input gradient (activation derivative from the stored
// layer output, rounding, overflow flag).  Every mbarrier wait is bounded; a wait that gives up sets the error word and the
// kernel winds down.
#include <cuda.h>

#include "common.cuh"
#include "conv_tc.h"
#include "tc_ptx.cuh"
#include "tensormap.h"

namespace mpode {
using namespace tc;
namespace {

constexpr int kC = 64;                          // channels in and out
constexpr int kWeightBytes = 9 * kC * kC * 2;   // nine [64 cout][64 cin] tiles
constexpr int kRingBytes = 147456;              // operand stages
constexpr int kMaxStages = 8;
constexpr int kAccs = 2;                        // TMEM accumulators
constexpr int kAccCols = 3 * kC;                // (dx, cout) columns of one accumulator
constexpr int kTmemCols = 512;                  // power of two >= kAccs * kAccCols
constexpr int kEpiWarps = 16;                    // two groups of eight (two per TMEM lane quadrant, 32 output channels each)
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kSmemBytes = kWeightBytes + kRingBytes + 1024 /*alignment slack*/ + 512 /*barriers*/;

struct ConvParams {
    int pixels, H, W;           // pixels = images * H * W
    int rows;                   // image rows per tile = 128 / W
    int stage_bytes, stages;    // (rows + 2) * W * 128
    int tiles;
    int epi, act;
    void* out;
    const float* tbias;         // EPI_FWD: [9 position classes][64] fp32 bias
    const void* hprev;          // EPI_DGRAD: stored output of the layer whose activation derivative multiplies the result, or null
    void* kap_out; const void* kap_v; float kap_bv, kap_c;   // EPI_DGRAD without hprev: also kap_out = Q16(kap_bv * v + kap_c * out), or null
    unsigned* flag;
    unsigned* err;
};

// three 16-column accumulator pieces (one per horizontal tap) of this lane's pixel, loaded together
__device__ __forceinline__ void tmem_ld_3x16(uint32_t t0, uint32_t t1, uint32_t t2, uint32_t (&a)[16], uint32_t (&b)[16], uint32_t (&c)[16]) {
#define MPODE_LD16(R, ADDR)                                                                                                          \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];" \
                 : "=r"(R[0]), "=r"(R[1]), "=r"(R[2]), "=r"(R[3]), "=r"(R[4]), "=r"(R[5]), "=r"(R[6]), "=r"(R[7]), "=r"(R[8]), "=r"(R[9]), \
                   "=r"(R[10]), "=r"(R[11]), "=r"(R[12]), "=r"(R[13]), "=r"(R[14]), "=r"(R[15])                                          \
                 : "r"(ADDR)                                                                                                             \
                 : "memory")
    MPODE_LD16(a, t0);
    MPODE_LD16(b, t1);
    MPODE_LD16(c, t2);
#undef MPODE_LD16
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// acc[i] = P_0 of this pixel + P_-1 of the left neighbour + P_+1 of the right neighbour (lanes of the same warp; `has_left` /
// `has_right` are false on the image border, where the neighbour is padding)
__device__ __forceinline__ void add_neighbours(const uint32_t (&rm)[16], const uint32_t (&rc)[16], const uint32_t (&rp)[16], bool has_left,
                                               bool has_right, float (&acc)[16]) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float left = __uint_as_float(__shfl_up_sync(0xffffffffu, rm[i], 1));
        const float right = __uint_as_float(__shfl_down_sync(0xffffffffu, rp[i], 1));
        acc[i] = __uint_as_float(rc[i]) + (has_left ? left : 0.f) + (has_right ? right : 0.f);
    }
}

// 16 columns of one output row: out = Q16(act(acc + bias))
template <typename T, int ACT>
__device__ __forceinline__ void store_forward(const float (&acc)[16], const float4* bv, T* orow) {
    const float* b = reinterpret_cast<const float*>(bv);
    uint32_t packed[8];
#pragma unroll
    for (int i = 0; i < 16; i += 2) packed[i >> 1] = cvt_pack<T>(fast_act<ACT>(acc[i] + b[i]), fast_act<ACT>(acc[i + 1] + b[i + 1]));
    *reinterpret_cast<uint4*>(orow) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    *reinterpret_cast<uint4*>(orow + 8) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
}

// out = Q16(act'(h) * acc) (h: the stored output of the layer, WITH_H) or Q16(acc); true if a value left the format's range
template <typename T, int ACT, bool WITH_H>
__device__ __forceinline__ bool store_backward(const float (&acc)[16], const uint4* hv, T* orow) {
    const uint32_t* hw = reinterpret_cast<const uint32_t*>(hv);
    const float lim = OverflowLimit<T>::value();
    uint32_t packed[8];
    bool bad = false;
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        float v0 = acc[i], v1 = acc[i + 1];
        if (WITH_H) {
            const uint32_t w = hw[i >> 1];
            v0 *= fast_act_deriv<ACT>(Low<T>::to_f(from_bits<T>((unsigned short)(w & 0xFFFFu))));
            v1 *= fast_act_deriv<ACT>(Low<T>::to_f(from_bits<T>((unsigned short)(w >> 16))));
        }
        bad |= !(fabsf(v0) < lim) | !(fabsf(v1) < lim);
        packed[i >> 1] = cvt_pack<T>(v0, v1);
    }
    *reinterpret_cast<uint4*>(orow) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    *reinterpret_cast<uint4*>(orow + 8) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
    return bad;
}

// Input gradient without an activation (the stage's psi): out = Q16(acc), and optionally the previous stage's cotangent from
// the rounded value, kappa = Q16(bv * v + c * psi), 16 columns; true if a value left the format's range
template <typename T>
__device__ __forceinline__ bool store_psi_kappa(const float (&acc)[16], T* orow, T* krow, const uint4 (&vv)[2], float bv, float c) {
    const float lim = OverflowLimit<T>::value();
    uint32_t packed[8];
    bool bad = false;
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        bad |= !(fabsf(acc[i]) < lim) | !(fabsf(acc[i + 1]) < lim);
        packed[i >> 1] = cvt_pack<T>(acc[i], acc[i + 1]);
    }
    *reinterpret_cast<uint4*>(orow) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    *reinterpret_cast<uint4*>(orow + 8) = make_uint4(packed[4], packed[5], packed[6], packed[7]);
    if (krow != nullptr) {
        const uint32_t* vw = reinterpret_cast<const uint32_t*>(vv);
        uint32_t kp[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float v0 = Low<T>::to_f(from_bits<T>((unsigned short)(vw[i] & 0xFFFFu))), v1 = Low<T>::to_f(from_bits<T>((unsigned short)(vw[i] >> 16)));
            const float q0 = Low<T>::to_f(from_bits<T>((unsigned short)(packed[i] & 0xFFFFu)));
            const float q1 = Low<T>::to_f(from_bits<T>((unsigned short)(packed[i] >> 16)));
            const T k0 = Low<T>::from_f(fmaf(c, q0, bv * v0)), k1 = Low<T>::from_f(fmaf(c, q1, bv * v1));
            bad |= Low<T>::nonfinite(k0) | Low<T>::nonfinite(k1);
            kp[i] = pack2<T>(k0, k1);
        }
        *reinterpret_cast<uint4*>(krow) = make_uint4(kp[0], kp[1], kp[2], kp[3]);
        *reinterpret_cast<uint4*>(krow + 8) = make_uint4(kp[4], kp[5], kp[6], kp[7]);
    }
    return bad;
}

template <typename T>
__global__ void __launch_bounds__(kThreads, 1)
conv3x3_halo_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, ConvParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sW = smem;                                   // [9 taps][64 cout][64 cin], 128-byte swizzled rows
    uint8_t* sA = smem + kWeightBytes;                    // `stages` halo blocks
    uint64_t* bars = (uint64_t*)(smem + kWeightBytes + kRingBytes);
    uint64_t* full_bar = bars;                            // [kMaxStages]
    uint64_t* empty_bar = bars + kMaxStages;              // [kMaxStages]
    uint64_t* tfull_bar = bars + 2 * kMaxStages;          // [kAccs]
    uint64_t* tempty_bar = bars + 2 * kMaxStages + kAccs; // [kAccs]
    uint64_t* w_bar = bars + 2 * kMaxStages + 2 * kAccs;
    uint32_t* tmem_holder = (uint32_t*)(w_bar + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.stages;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < kAccs; ++a) { mbar_init(&tfull_bar[a], 1); mbar_init(&tempty_bar[a], kEpiWarps / 2); }
        mbar_init(w_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_holder, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *(volatile uint32_t*)tmem_holder;

    if (warp == 0) {
        // ------------------------------------------------------------ loads: the weights once, then one halo block per tile
        if (lane == 0) {
            mbar_arrive_expect_tx(w_bar, (uint32_t)kWeightBytes);
            for (int t = 0; t < 9; ++t) tma_load_2d(smem_u32(sW + t * kC * kC * 2), &tmW, w_bar, t * kC, 0);
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x) {
                const int m0 = tile * BM;
                const int img = m0 / (p.H * p.W), y0 = (m0 / p.W) % p.H;
                ok = mbar_wait(&empty_bar[s], phase ^ 1u, p.err, 1u);
                if (!ok) break;
                mbar_arrive_expect_tx(&full_bar[s], (uint32_t)p.stage_bytes);
                tma_load_4d(smem_u32(sA + (size_t)s * p.stage_bytes), &tmX, &full_bar[s], 0, 0, y0 - 1, img);
                if (++s == S) { s = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(Fmt<T>::id, BM, kAccCols, false);
            int s = 0;
            uint32_t phase = 0;
            int it = 0;
            bool ok = mbar_wait(w_bar, 0u, p.err, 16u);
            const uint32_t w_addr = smem_u32(sW);
            const uint32_t dy_step = (uint32_t)(p.W * 128) >> 4;          // one image row of the halo block, in 16-byte units
            for (int tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x, ++it) {
                const int acc = it % kAccs;
                const uint32_t use = (uint32_t)(it / kAccs);
                ok = mbar_wait(&tempty_bar[acc], (use & 1u) ^ 1u, p.err, 2u);       // epilogue has drained this accumulator
                if (!ok) break;
                ok = mbar_wait(&full_bar[s], phase, p.err, 4u);                     // the halo block has landed
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t tmem_d = tmem_base + (uint32_t)(acc * kAccCols);
                const uint64_t adesc0 = smem_desc_k_major_sw128(smem_u32(sA + (size_t)s * p.stage_bytes));
#pragma unroll
                for (int dyi = 0; dyi < 3; ++dyi) {
                    // A: the tile's pixels one image row further down per dy; B: the three taps (dy, -1..1) as 192 rows
                    const uint64_t adesc = adesc0 + (uint64_t)(dy_step * (uint32_t)dyi);
                    const uint64_t bdesc = smem_desc_k_major_sw128(w_addr + (uint32_t)(dyi * 3 * kC * kC * 2));
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        umma_f16(tmem_d, adesc + 2u * (uint64_t)k, bdesc + 2u * (uint64_t)k, idesc, (dyi | k) != 0 ? 1u : 0u);
                }
                umma_commit(&empty_bar[s]);                                         // block reusable once these MMAs retire
                umma_commit(&tfull_bar[acc]);
                if (++s == S) { s = 0; phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        // hardware rule: a warp reads the TMEM lanes [32 * (warp % 4), +32).  The warps form two groups, one per accumulator: a
        // group's tile is every other one, so that the latency of one tile's epilogue (wake-up, accumulator load, shuffles,
        // stores) overlaps the other group's; within a group the two warps of a quadrant take 32 output channels each.
        const int q = warp & 3;
        const int group = (warp - 2) >> 3;
        const int nb = (((warp - 2) >> 2) & 1) * 32;
        const int w_shift = 31 - __clz(p.W);                    // W is a power of two
        bool bad = false;
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x, ++it) {
            const int acc = it % kAccs;
            if (acc != group) continue;
            const uint32_t use = (uint32_t)(it / kAccs);
            const int m = tile * BM + q * 32 + lane;
            T* orow = (T*)p.out + (long long)m * kC + nb;
            const int x = m & (p.W - 1);
            const bool has_left = x != 0, has_right = x != p.W - 1;
            // what the epilogue needs besides the accumulator is fetched before the wait for it
            const float4* sb = nullptr;
            uint4 hv[4];
            if (p.epi == EPI_FWD) {
                // the appended time channel is zero in the padding: its contribution (a bias per position class, a table of 2.3 KB
                // that stays in L1) depends on which taps are inside
                const int y = (m >> w_shift) % p.H;
                const int cls = 3 * (y == 0 ? 0 : (y == p.H - 1 ? 2 : 1)) + (x == 0 ? 0 : (x == p.W - 1 ? 2 : 1));
                sb = reinterpret_cast<const float4*>(p.tbias + cls * kC + nb);
            } else if (p.hprev != nullptr) {
                const uint4* hrow = reinterpret_cast<const uint4*>((const T*)p.hprev + (long long)m * kC + nb);
#pragma unroll
                for (int v = 0; v < 4; ++v) hv[v] = hrow[v];
            } else if (p.kap_out != nullptr) {      // the seed rows that enter the previous stage's cotangent
                const uint4* vrow = reinterpret_cast<const uint4*>((const T*)p.kap_v + (long long)m * kC + nb);
#pragma unroll
                for (int v = 0; v < 4; ++v) hv[v] = vrow[v];
            }
            ok = mbar_wait(&tfull_bar[acc], use & 1u, p.err, 8u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t tcol = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kAccCols + nb);
#pragma unroll
            for (int c = 0; c < 2; ++c) {                                           // 16 output channels at a time
                uint32_t rm[16], rc[16], rp[16];
                __syncwarp();
                tmem_ld_3x16(tcol + (uint32_t)(c * 16), tcol + (uint32_t)(kC + c * 16), tcol + (uint32_t)(2 * kC + c * 16), rm, rc, rp);
                if (c == 1) {
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tempty_bar[acc]);                   // the values are in registers
                }
                float v[16];
                add_neighbours(rm, rc, rp, has_left, has_right, v);
                T* o = orow + c * 16;
                if (p.epi == EPI_FWD) {
                    float4 bv[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) bv[u] = __ldg(sb + 4 * c + u);
                    switch (p.act) {
                        case MPODE_ACT_SOFTPLUS: store_forward<T, MPODE_ACT_SOFTPLUS>(v, bv, o); break;
                        case MPODE_ACT_RELU: store_forward<T, MPODE_ACT_RELU>(v, bv, o); break;
                        case MPODE_ACT_TANH: store_forward<T, MPODE_ACT_TANH>(v, bv, o); break;
                        default: store_forward<T, MPODE_ACT_NONE>(v, bv, o); break;
                    }
                } else if (p.hprev == nullptr) {
                    const uint4 vv[2] = {hv[2 * c], hv[2 * c + 1]};
                    T* krow = p.kap_out != nullptr ? (T*)p.kap_out + (long long)m * kC + nb + c * 16 : nullptr;
                    bad |= store_psi_kappa<T>(v, o, krow, vv, p.kap_bv, p.kap_c);
                } else {
                    switch (p.act) {
                        case MPODE_ACT_SOFTPLUS: bad |= store_backward<T, MPODE_ACT_SOFTPLUS, true>(v, hv + 2 * c, o); break;
                        case MPODE_ACT_RELU: bad |= store_backward<T, MPODE_ACT_RELU, true>(v, hv + 2 * c, o); break;
                        case MPODE_ACT_TANH: bad |= store_backward<T, MPODE_ACT_TANH, true>(v, hv + 2 * c, o); break;
                        default: bad |= store_backward<T, MPODE_ACT_NONE, true>(v, hv + 2 * c, o); break;
                    }
                }
            }
        }
        if (p.epi == EPI_DGRAD) warp_flag_or(p.flag, bad);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---------------------------------------------------------------- weight gradient
// dW[dy, dx][cin, cout] = sum over pixels (y, x) of X[y + dy, x + dx][cin] * dZ[y, x][cout], computed over slices of the pixels
// as a contraction whose reduction index is the pixel p = (y, x') with x' = x + dx:
//   A (MN-major): rows of the image block around the k-block's R' image rows, fetched once ((R' + 3) rows, the padding reads as
//     zero).  The view that starts v image rows into the block is X[y + (v - 1), x']: one MMA takes two views as its two
//     64-channel chunks of M by giving the descriptor's chunk stride the length of one image row.
//   B (MN-major): dZ[y, x' - dx] for dx = -1, 0, 1 as three 64-column chunks of N = 192, i.e. three loads of the k-block's dZ
//     rows whose x coordinate starts at -dx (the columns that fall outside read as zero, which is what the padding of X gives).
// Accumulator a holds the views dy = -1, 0 as its 128 lanes, accumulator b the view dy = +1 as lanes 0..63.  The other chunk of
// the second MMA is the k-block's piece of the position-class indicator table (column c is 1 where the pixel's class is c): its
// rows 64..72 are the sums of dZ over the pixels of each class, which the gradients of the bias and of an appended time
// channel are made of.  A CTA runs over its slice of the pixels, then writes [192 (dy, cin)][192 (dx, cout)] fp32 partial sums
// and [9 classes][64 cout] class sums; the slices are added in a fixed order afterwards.
struct WgradParams {
    int H, W;
    int kb_rows;                // image rows per k-block of 64 pixels
    int kblocks, per_cta;       // k-blocks in all, per CTA
    int a_bytes, stage_bytes, stages;
    float* partial;             // [gridDim.x][192][192]
    float* class_part;          // [gridDim.x][9][64] sums of dZ per position class
    unsigned* err;
};

constexpr int kWgRows = 3 * kC, kWgCols = 3 * kC;
constexpr int kWgRingBytes = 208 * 1024;

__device__ __forceinline__ uint64_t smem_desc_mn_major_sw128_stride(uint32_t smem_addr, uint32_t chunk_stride_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((chunk_stride_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1u << 46;
    d |= (uint64_t)2u << 61;
    return d;
}

template <typename T>
__global__ void __launch_bounds__(320, 1)
conv3x3_wgrad_halo_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmZ,
                          const __grid_constant__ CUtensorMap tmI, WgradParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = (uint64_t*)(smem + kWgRingBytes);
    uint64_t* full_bar = bars;                  // [kMaxStages]
    uint64_t* empty_bar = bars + kMaxStages;    // [kMaxStages]
    uint64_t* done_bar = bars + 2 * kMaxStages;
    uint32_t* tmem_holder = (uint32_t*)(done_bar + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.stages;
    const int kb0 = blockIdx.x * p.per_cta, kb1 = min(p.kblocks, kb0 + p.per_cta);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(done_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_holder, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *(volatile uint32_t*)tmem_holder;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int kb = kb0; kb < kb1 && ok; ++kb) {
                const int row0 = kb * p.kb_rows;                    // first image row of the k-block, counted over all images
                const int img = row0 / p.H, y0 = row0 % p.H;
                ok = mbar_wait(&empty_bar[s], phase ^ 1u, p.err, 1u);
                if (!ok) break;
                mbar_arrive_expect_tx(&full_bar[s], (uint32_t)p.stage_bytes);
                const uint32_t a_dst = smem_u32(smem + (size_t)s * p.stage_bytes), b_dst = a_dst + (uint32_t)p.a_bytes;
                tma_load_4d(a_dst, &tmX, &full_bar[s], 0, 0, y0 - 1, img);
#pragma unroll
                for (int j = 0; j < 3; ++j) tma_load_4d(b_dst + j * 8192, &tmZ, &full_bar[s], 0, 1 - j, y0, img);   // dx = j - 1: x starts at -dx
                tma_load_2d(b_dst + 3 * 8192, &tmI, &full_bar[s], 0, y0 * p.W);                                     // class indicators of these pixels
                if (++s == S) { s = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(Fmt<T>::id, BM, kWgCols, true);
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            const uint32_t row_bytes = (uint32_t)(p.W * 128);       // one image row of the block
            for (int kb = kb0; kb < kb1 && ok; ++kb) {
                ok = mbar_wait(&full_bar[s], phase, p.err, 4u);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t a_addr = smem_u32(smem + (size_t)s * p.stage_bytes), b_addr = a_addr + (uint32_t)p.a_bytes;
                const uint64_t adesc_a = smem_desc_mn_major_sw128_stride(a_addr, row_bytes);                    // views 0, 1
                // view 2, and as its second chunk the indicator block behind the three dZ blocks
                const uint64_t adesc_b = smem_desc_mn_major_sw128_stride(a_addr + 2u * row_bytes, (uint32_t)p.a_bytes + 3u * 8192u - 2u * row_bytes);
                const uint64_t bdesc = smem_desc_mn_major_sw128_stride(b_addr, 8192u);
                // one instruction consumes 16 pixels: 16 rows of 128 bytes (+128 in 16-byte units)
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k) {
                    const uint32_t accum = (kb > kb0 || k > 0) ? 1u : 0u;
                    umma_f16(tmem_base, adesc_a + 128u * (uint64_t)k, bdesc + 128u * (uint64_t)k, idesc, accum);
                    umma_f16(tmem_base + (uint32_t)kWgCols, adesc_b + 128u * (uint64_t)k, bdesc + 128u * (uint64_t)k, idesc, accum);
                }
                umma_commit(&empty_bar[s]);
                if (++s == S) { s = 0; phase ^= 1u; }
            }
            if (ok) umma_commit(done_bar);
        }
    } else {
        // ------------------------------------------------------------ the partial sums of this slice, once
        const int q = warp & 3, half = (warp - 2) >> 2;
        bool ok = kb1 > kb0 ? mbar_wait(done_bar, 0u, p.err, 8u) : true;
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after_sync();
            float* part = p.partial + (size_t)blockIdx.x * kWgRows * kWgCols;
            // accumulator a: lanes = rows 0..127 (dy = -1, 0); accumulator b: lanes 0..63 = rows 128..191 (dy = +1), lanes 64..72 =
            // the class sums (their columns 64..127: the unshifted dZ)
#pragma unroll 1
            for (int a = 0; a < 2; ++a) {
                if (a == 1 && q == 3) break;
                const bool classes = a == 1 && q == 2;
                float* prow = part + (size_t)(a * 128 + q * 32 + lane) * kWgCols;
#pragma unroll 1
                for (int c = half * 3; c < half * 3 + 3; ++c) {     // 32 columns at a time, three per warp of the pair
                    if (classes && c != 2 && c != 3) continue;
                    uint32_t r[32];
                    if (kb1 > kb0) {
                        tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * kWgCols + c * 32), r);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = 0u;
                    }
                    float* dst = prow + c * 32;
                    if (classes) dst = p.class_part + ((size_t)blockIdx.x * 9 + lane) * kC + (c - 2) * 32;
                    if (!classes || lane < 9) {
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            *reinterpret_cast<uint4*>(dst + v * 4) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                    }
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// out[(cout * 9 + dy * 3 + dx) * ct + cin] = beta * out + sign * (sum over the slices, in ascending order, of
// partial[slice][dy * 64 + cin][dx * 64 + cout]).  A block takes 128 consecutive elements of the [192][192] matrix; its eight
// warps add every eighth slice each, and the eight sums are added in a fixed order.  Eighteen more blocks add the slices' class
// sums the same way into `class_sums` (behind the slices' own); the one of them that finishes last (a counter that it sets back
// to zero) turns the sums into the gradients of the bias and of the appended time channel's weights.
constexpr int kWgMatrixBlocks = kWgRows * kWgCols / 128, kWgClassBlocks = 9 * kC / 32;

__global__ void __launch_bounds__(256) conv_wgrad_halo_reduce_kernel(const float* __restrict__ partial, int slices, int ct, float* __restrict__ out,
                                                                       float beta, float sign, float* __restrict__ class_part, float tau,
                                                                       float* __restrict__ wt_out, float* __restrict__ bias_out,
                                                                       unsigned* __restrict__ counter) {
    __shared__ float4 sm4[8 * 32];
    float* sm = reinterpret_cast<float*>(sm4);
    __shared__ bool last;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (blockIdx.x < kWgMatrixBlocks) {
        // four consecutive elements of the matrix per lane (16-byte loads, four of them in flight), slices in ascending order
        const float4* src = reinterpret_cast<const float4*>(partial);
        const size_t stride = (size_t)kWgRows * kWgCols / 4;
        const int e4 = blockIdx.x * 32 + lane;
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        auto add = [&](const float4& v) { s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w; };
        int z = w;
        for (; z + 24 < slices; z += 32) {
            const float4 v0 = src[(size_t)z * stride + e4], v1 = src[(size_t)(z + 8) * stride + e4];
            const float4 v2 = src[(size_t)(z + 16) * stride + e4], v3 = src[(size_t)(z + 24) * stride + e4];
            add(v0); add(v1); add(v2); add(v3);
        }
        for (; z < slices; z += 8) add(src[(size_t)z * stride + e4]);
        sm4[w * 32 + lane] = s;
        __syncthreads();
        if (w == 0) {
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int k = 0; k < 8; ++k) { const float4 v = sm4[k * 32 + lane]; t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w; }
            const float tv[4] = {t.x, t.y, t.z, t.w};
            const int e = e4 * 4, row = e / kWgCols, col = e - row * kWgCols;      // the four elements share a row (192 = 48 * 4)
            const int dy = row / kC, cin = row - dy * kC;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int dx = (col + i) / kC, cout = col + i - dx * kC;
                float* o = out + ((size_t)cout * 9 + dy * 3 + dx) * ct + cin;
                *o = (beta != 0.f ? *o : 0.f) + sign * tv[i];
            }
        }
        return;
    }
    const int e = (blockIdx.x - kWgMatrixBlocks) * 32 + lane;                     // element of the class sums
    float s = 0.f;
    for (int z = w; z < slices; z += 8) s += class_part[(size_t)z * 9 * kC + e];
    sm[w * 32 + lane] = s;
    __syncthreads();
    float t = 0.f;
    if (w == 0) {
#pragma unroll
        for (int k = 0; k < 8; ++k) t += sm[k * 32 + lane];
    }
    float* class_sums = class_part + (size_t)slices * 9 * kC;
    if (w == 0) {
        class_sums[e] = sign * t;
        __threadfence();
    }
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(counter, 1u) == (unsigned)(kWgClassBlocks - 1);
    __syncthreads();
    if (!last) return;
    __threadfence();
    for (int i = threadIdx.x; i < 9 * kC; i += blockDim.x) sm[i] = __ldcg(class_sums + i);
    __syncthreads();
    conv_class_finish(sm, kC, ct, tau, wt_out, bias_out, beta);
    if (threadIdx.x == 0) *counter = 0u;
}

template <typename T>
bool launch_halo(const CUtensorMap& tx, const CUtensorMap& tw, const ConvParams& p, cudaStream_t st) {
    static bool attr_set[kMaxDevices] = {false};
    const int dev = current_device();
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(conv3x3_halo_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        attr_set[dev] = true;
    }
    const int grid = p.tiles < sm_count() ? p.tiles : sm_count();
    conv3x3_halo_kernel<T><<<grid, kThreads, kSmemBytes, st>>>(tx, tw, p);
    return true;
}

}  // namespace

bool conv_halo_eligible(mpode_dtype dt, const GemmArgs& g) {
    if (dt != MPODE_BF16 && dt != MPODE_F16) return false;
    if (g.conv_on != 1 || (g.epi != EPI_FWD && g.epi != EPI_DGRAD) || g.out2 != nullptr) return false;
    if (g.conv_cd != kC || g.conv_ct != kC || g.N != kC || g.K != 9 * kC || g.b_rs != 9 * kC || g.b_ks != 1 || g.ldo != kC) return false;
    // image rows no wider than a warp: the horizontal neighbours of a pixel are lanes of the same epilogue warp
    if (g.conv_w < 8 || g.conv_w > 32 || (32 % g.conv_w) != 0 || g.conv_h < 2 || g.conv_h % (128 / g.conv_w) != 0) return false;
    if (g.M % (g.conv_h * g.conv_w) != 0) return false;
    if (g.epi == EPI_FWD && g.conv_tbias == nullptr) return false;
    if (g.hprev != nullptr && g.ldh != kC) return false;
    if (((uintptr_t)g.A | (uintptr_t)g.B | (uintptr_t)g.out | (uintptr_t)g.hprev | (uintptr_t)g.kap_out | (uintptr_t)g.kap_v) & 15) return false;
    if (g.kap_out != nullptr && (g.epi != EPI_DGRAD || g.hprev != nullptr || g.kap_v == nullptr)) return false;
    return g.err != nullptr;
}

bool launch_conv_halo(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* launches) {
    ConvParams p{};
    p.pixels = g.M; p.H = g.conv_h; p.W = g.conv_w;
    p.rows = 128 / g.conv_w;
    p.stage_bytes = (p.rows + 2) * g.conv_w * 128;
    p.stages = kRingBytes / p.stage_bytes;
    if (p.stages > kMaxStages) p.stages = kMaxStages;
    if (p.stages < 2) return false;
    p.tiles = g.M / BM;
    p.epi = g.epi; p.act = g.act; p.out = g.out; p.tbias = g.conv_tbias; p.hprev = g.hprev; p.flag = g.flag; p.err = g.err;
    if (g.epi == EPI_DGRAD && g.hprev == nullptr && g.kap_out != nullptr) {
        p.kap_out = g.kap_out; p.kap_v = g.kap_v; p.kap_bv = g.kap_bv; p.kap_c = g.kap_c;
    }
    CUtensorMap tx, tw;
    if (!get_tensor_map_nhwc(g.A, g.M / (g.conv_h * g.conv_w), g.conv_h, g.conv_w, kC, p.rows + 2, dt, &tx)) return false;
    if (!get_tensor_map(g.B, kC, 9 * kC, 9 * kC, kC, dt, &tw)) return false;
    const bool ok = dt == MPODE_BF16 ? launch_halo<__nv_bfloat16>(tx, tw, p, st) : launch_halo<__half>(tx, tw, p, st);
    if (ok && launches) ++*launches;
    return ok;
}

// ---------------------------------------------------------------- weight gradient: host side
static void wgrad_halo_plan(int B, int H, int W, WgradParams* p, int* grid) {
    p->H = H; p->W = W;
    p->kb_rows = 64 / W;
    p->kblocks = (int)((long long)B * H * W / 64);
    *grid = p->kblocks < sm_count() ? p->kblocks : sm_count();
    p->per_cta = (p->kblocks + *grid - 1) / *grid;
    *grid = (p->kblocks + p->per_cta - 1) / p->per_cta;
    p->a_bytes = (p->kb_rows + 2) * W * 128;
    p->stage_bytes = p->a_bytes + 4 * 8192;          // the image block, three dZ blocks, the indicator block
    p->stages = kWgRingBytes / p->stage_bytes;
    if (p->stages > kMaxStages) p->stages = kMaxStages;
}

size_t conv_wgrad_halo_scratch_bytes(int B, int H, int W) {
    WgradParams p{};
    int grid;
    wgrad_halo_plan(B, H, W, &p, &grid);
    return (size_t)grid * kWgRows * kWgCols * sizeof(float);
}

bool conv_wgrad_halo_eligible(mpode_dtype dt, int B, int H, int W, int C, const void* dz, const void* x, const float* partial,
                              size_t partial_bytes, const unsigned* err) {
    if (dt != MPODE_BF16 && dt != MPODE_F16) return false;
    if (C != kC || W < 8 || W > 32 || (32 % W) != 0 || H < 2 || H % (64 / W) != 0) return false;
    if (((uintptr_t)dz | (uintptr_t)x | (uintptr_t)partial) & 15) return false;
    if ((long long)B * H * W < 512 || (long long)B * H * W > 0x7fffffffLL || err == nullptr || partial == nullptr) return false;
    return conv_wgrad_halo_scratch_bytes(B, H, W) <= partial_bytes;
}

int conv_wgrad_halo_slices(int B, int H, int W) {
    WgradParams p{};
    int grid;
    wgrad_halo_plan(B, H, W, &p, &grid);
    return grid;
}

bool launch_conv_wgrad_halo(mpode_dtype dt, const void* dz, const void* x, const void* indicator, int B, int H, int W, int ct, float* out,
                            float* bias_out, float tau, float beta, float* partial, float* class_part, unsigned* counter, unsigned* err,
                            cudaStream_t st, long long* launches, float sign) {
    WgradParams p{};
    int grid;
    wgrad_halo_plan(B, H, W, &p, &grid);
    if (p.stages < 2) return false;
    p.partial = partial; p.class_part = class_part; p.err = err;
    CUtensorMap tx, tz, ti;
    if (!get_tensor_map_nhwc(x, B, H, W, kC, p.kb_rows + 2, dt, &tx)) return false;
    if (!get_tensor_map_nhwc(dz, B, H, W, kC, p.kb_rows, dt, &tz)) return false;
    if (!get_tensor_map(indicator, (long long)H * W, kC, kC, 64, dt, &ti)) return false;
    constexpr int smem_bytes = kWgRingBytes + 1024 + 512;
    static bool attr_set[kMaxDevices][2] = {};
    const int dev = current_device(), fi = dt == MPODE_BF16 ? 1 : 0;
    if (!attr_set[dev][fi]) {
        cudaError_t e = dt == MPODE_BF16
            ? cudaFuncSetAttribute(conv3x3_wgrad_halo_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes)
            : cudaFuncSetAttribute(conv3x3_wgrad_halo_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
        if (e != cudaSuccess) { cudaGetLastError(); return false; }
        attr_set[dev][fi] = true;
    }
    if (dt == MPODE_BF16) conv3x3_wgrad_halo_kernel<__nv_bfloat16><<<grid, 320, smem_bytes, st>>>(tx, tz, ti, p);
    else conv3x3_wgrad_halo_kernel<__half><<<grid, 320, smem_bytes, st>>>(tx, tz, ti, p);
    if (launches) ++*launches;
    conv_wgrad_halo_reduce_kernel<<<kWgMatrixBlocks + kWgClassBlocks, 256, 0, st>>>(partial, grid, ct, out, beta, sign, class_part, tau,
                                                                                    ct > kC ? out : nullptr, bias_out, counter);
    if (launches) ++*launches;
    return true;
}

}  // namespace mpode
