// Velocity-layer contractions on the 5th-generation tensor cores (sm_100a): C[M, N] = A[M, K] * B[N, K]^T with both
// operands K-major in global memory, fp32 accumulation in tensor memory, and the layer epilogue fused:
//   forward  : out = Q16(act(acc + b + tau * w_t))                      (Alg. 1 increment, one rounding per layer)
//   backward : out = Q16(act'(H_prev) * acc), non-finite outputs flagged (Eq. (vjp), Alg. 2 finiteness test)
//   flow with a trace estimate (Sec. 6.1): tiles that hold 64 tangent rows and the primal rows of the same samples, so that
//     the tangent activation G = Q16(act'(H) * U) and the backward step through an activation (which mixes the primal and the
//     tangent cotangent of a sample) are epilogue work; the two warps that hold a sample's two rows exchange 16-column pieces
//     through shared memory and meet at named barriers
//
// Persistent, warp-specialised CTA (one per SM): warp 0 issues TMA tile loads into a ring of 128B-swizzled
// shared-memory stages, warp 1 issues tcgen05.mma (128 x BN x 16 per instruction) into one of two TMEM
// accumulators, warps 2..9 drain the other accumulator with tcgen05.ld and run the epilogue, so the epilogue of
// tile i overlaps the main loop of tile i+1.  Every mbarrier wait is bounded in time; a wait that gives up sets an
// error word and the kernel winds down without trapping.
#include <cuda.h>

#include "common.cuh"
#include "gemm_tc.h"
#include "tc_ptx.cuh"
#include "tc_epilogue.cuh"
#include "tensormap.h"

namespace mpode {
using namespace tc;
namespace {

// Widest tiles (BN = 256): one CTA per SM, eight epilogue warps (two per TMEM lane quadrant, each half of the columns).
// Narrower tiles (BN <= 128: the convolutions, thin layers): half the shared memory, four epilogue warps and a small register
// footprint, so that two CTAs share an SM and one's loads and epilogue hide behind the other's MMAs.
template <int BN> struct Shape {
    static constexpr int kEpiWarps = BN <= 128 ? 4 : 8;
    static constexpr int kThreads = 64 + 32 * kEpiWarps;          // warp 0 TMA, warp 1 MMA, the rest epilogue
    static constexpr int kSmemBudget = BN <= 128 ? 98304 : 196608;   // bytes of operand stages
    static constexpr int kCtasPerSm = BN <= 128 ? 2 : 1;
};

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
    // implicit 3x3 convolution (stride 1, zero padding 1) over an NHWC image with 64 channels: rows of A are pixels, the
    // k-block index is the tap, and the tile's 128 pixels are 128 / conv_w whole image rows fetched with one 4-D bulk load
    // at the tap's offset (out-of-image pixels read as zero)
    int conv, conv_h, conv_w, conv_c;   // conv_c: channels of the image (a multiple of 64; a k-block is 64 channels of one tap)
    const float* tbias;         // EPI_FWD with conv: [9][N] bias table per position class
    int direct; float beta;     // weight gradient with one slice: write out = beta * out + acc directly
    // flow with a trace estimate: a tile is 64 primal rows and the 64 tangent rows m_split further down (GemmArgs::cnf_pair)
    int pair; void* pair_out; const void* uprev;
};

constexpr int kPairRowWords = 20;                                  // one lane's exchange row: 16 words and padding (16-byte multiples)

template <int BN> struct TileCfg {
    static constexpr int kStageBytes = BM * BK * 2 + BN * BK * 2;
    static constexpr int kStages = Shape<BN>::kSmemBudget / kStageBytes;
    static constexpr int kTmemCols = 2 * BN;            // two accumulators; 128, 256 or 512 columns (powers of two)
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 4 * BN * 4 /*bias, one copy per epilogue warp*/ + 256 /*barriers*/ +
                                      (Shape<BN>::kEpiWarps / 2) * 2 * 32 * kPairRowWords * 4 /*two sets of exchange rows per warp pair (paired tiles)*/;
};

// WG = false: C[M, N] = A[M, K] B[N, K]^T, operands K-major in memory, low-format output with fused epilogue.
// WG = true : C[M, N] = sum_r A[r, M] B[r, N] (weight gradient: the reduction index r runs over the batch rows of two
//             row-major activations), fp32 partial sums per reduction slice, reduced afterwards in a fixed order.
// PAIR: the paired tiles of the flow with a trace estimate (GemmArgs::cnf_pair, 1 forward / 2 backward), variants of their own so
// that each keeps to its register budget (a spill costs a trip to L2 here: almost all of the L1 is shared memory).
template <typename T, int BN, bool WG, int PAIR = 0>
__global__ void __launch_bounds__(Shape<BN>::kThreads, Shape<BN>::kCtasPerSm)
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
    uint32_t* xbuf = (uint32_t*)((uint8_t*)bars + 256);   // [warp pairs][2][32 lanes][kPairRowWords]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int n_work = n_tiles * p.splits;
    const int kb_total = (p.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&tfull_bar[a], 1); mbar_init(&tempty_bar[a], Shape<BN>::kEpiWarps); }
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
                    const uint32_t a_dst = smem_u32(sA + (size_t)s * BM * BK * 2), b_dst = smem_u32(sB + (size_t)s * BN * BK * 2);
                    if (WG && p.conv) {
                        // convolution weight gradient, transposed: rows of the output are (tap, input channel), the reduction
                        // runs over pixels.  A k-block is 64 pixels = 64 / W whole image rows, read at the tap's offset (zero
                        // outside the image); the tile's 128 rows are two taps, the ninth tap has no partner.
                        const int p0 = kb * BK;
                        const int img = p0 / (p.conv_h * p.conv_w), y0 = (p0 / p.conv_w) % p.conv_h;
                        const int n_a = m0 + 64 < p.M ? 2 : 1;        // the tile's rows are (tap, channel) pairs: two 64-channel pieces, or one
                        mbar_arrive_expect_tx(&full_bar[s], (uint32_t)((n_a + BN / 64) * 8192));
                        for (int c = 0; c < n_a; ++c) {
                            const int row = m0 + c * 64, tap = row / p.conv_c, ch0 = row % p.conv_c;
                            tma_load_4d(a_dst + c * 8192, &tmA, &full_bar[s], ch0, tap % 3 - 1, y0 + tap / 3 - 1, img);
                        }
#pragma unroll
                        for (int c = 0; c < BN / 64; ++c) tma_load_2d(b_dst + c * 8192, &tmB, &full_bar[s], n0 + c * 64, kb * BK);
                        if (++s == S) { s = 0; phase ^= 1u; }
                        continue;
                    }
                    mbar_arrive_expect_tx(&full_bar[s], (uint32_t)Cfg::kStageBytes);
                    if (!WG && p.conv) {
                        const int img = m0 / (p.conv_h * p.conv_w), y0 = (m0 / p.conv_w) % p.conv_h;
                        const int nch = p.conv_c / 64, tap = kb / nch;
                        tma_load_4d(a_dst, &tmA, &full_bar[s], (kb % nch) * 64, tap % 3 - 1, y0 + tap / 3 - 1, img);
                        tma_load_2d(b_dst, &tmB, &full_bar[s], kb * BK, n0);
                    } else if (PAIR != 0) {
                        // 64 tangent rows, then the primal rows of the same samples (the map's box is 64 rows high).  The primal
                        // rows have the heavier epilogue: they go to the TMEM lane quadrants 2 and 3, whose warps share no
                        // scheduler with the warps that issue the bulk loads and the MMAs.
                        tma_load_2d(a_dst, &tmA, &full_bar[s], kb * BK, p.m_split + m0 / 2);
                        tma_load_2d(a_dst + 8192, &tmA, &full_bar[s], kb * BK, m0 / 2);
                        tma_load_2d(b_dst, &tmB, &full_bar[s], kb * BK, n0);
                    } else if (!WG) {
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
        constexpr int kColsPerWarp = BN / (Shape<BN>::kEpiWarps / 4);
        float* sb_warp = sbias + (warp - 2) * kColsPerWarp;   // this warp's slice of the effective bias b + tau * w_t
        bool bad = false;
        bool ok = true;
        int it = 0;
        for (int w = blockIdx.x; w < n_work && ok; w += gridDim.x, ++it) {
            const int acc = it & 1;
            const uint32_t use = (uint32_t)(it >> 1);
            const int tile = w % n_tiles, z = w / n_tiles;
            const int m0 = (tile / p.tiles_n) * BM, n0 = (tile % p.tiles_n) * BN + half * kColsPerWarp;
            if (!WG && p.epi == EPI_FWD && !p.conv) {
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
            // paired tiles: the two warps that hold a sample's primal and tangent rows go on, or give up, together
            constexpr bool pair = PAIR != 0;
            const int pair_id = 1 + (q & 1) + 2 * half;
            if (pair) ok = pair_all(pair_id, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const bool tangent = pair && q < 2;
            // row of the operand, or with paired tiles the sample (tile rows 0..63 tangent rows, 64..127 their primal rows)
            const int m = pair ? m0 / 2 + (q & 1) * 32 + lane : m0 + q * 32 + lane;
            const bool row_ok = pair ? m < p.m_split : m < p.M;
            const bool second = pair ? tangent : (p.out2 != nullptr) && (m >= p.m_split);
            T* orow = second ? (T*)p.out2 + (long long)(pair ? m : m - p.m_split) * p.ldo : (T*)p.out + (long long)m * p.ldo;
            const T* hrow = (p.hprev != nullptr) ? (const T*)p.hprev + (long long)m * p.ldh : nullptr;
            const T* urow = (p.uprev != nullptr) ? (const T*)p.uprev + (long long)m * p.ldh : nullptr;
            uint32_t* xrow0 = xbuf + ((pair_id - 1) * 64 + lane) * kPairRowWords;      // this lane's row in the two sets
            uint32_t* xrow1 = xrow0 + 32 * kPairRowWords;
            const uint32_t tcol = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + half * kColsPerWarp);
            // convolution forward: the appended time channel is zero in the padding, so its contribution (folded into a bias
            // per position class) depends on which taps are inside the image at this pixel
            int cls = 0;
            if (!WG && !PAIR && p.conv && p.epi == EPI_FWD) {
                const int y = (m / p.conv_w) % p.conv_h, x = m % p.conv_w;
                cls = 3 * (y == 0 ? 0 : (y == p.conv_h - 1 ? 2 : 1)) + (x == 0 ? 0 : (x == p.conv_w - 1 ? 2 : 1));
            }
#pragma unroll 1
            for (int c = 0; c < kColsPerWarp / 32; ++c) {
                uint32_t r[32];
                // operands of the epilogue that live in global memory are requested before the accumulator is waited for
                uint4 hv[4], uv[4];
                float bl[32];
                if (!WG && row_ok && n0 + c * 32 < p.N) {
                    if (p.epi == EPI_DGRAD) load_h_chunk<T>(hrow, n0 + c * 32, p.N, hv);
                    if (PAIR == 2 && !tangent) load_h_chunk<T>(urow, n0 + c * 32, p.N, uv);
                    if (!PAIR && p.conv && p.epi == EPI_FWD) {
                        const float* tb = p.tbias + (long long)cls * p.N + n0 + c * 32;
#pragma unroll
                        for (int v = 0; v < 8; ++v)   // N is a multiple of 8 and the table 16-byte aligned
                            reinterpret_cast<float4*>(bl)[v] = (n0 + c * 32 + v * 4 < p.N) ? __ldg(reinterpret_cast<const float4*>(tb) + v)
                                                                                           : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
                __syncwarp();   // tcgen05.ld is warp-collective: reconverge after the guarded body of the last chunk
                tmem_ld_32x32(tcol + (uint32_t)(c * 32), r);
                const int nb = n0 + c * 32;
                if (WG && p.direct) {
                    // one reduction slice and an output whose rows are 16-byte aligned: out = beta * out + acc without scratch
                    if (row_ok && nb < p.N) {
                        float* orow32 = (float*)p.out + (long long)m * p.ldo + nb;
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            if (nb + v * 4 < p.N) {
                                float4 o = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]), __uint_as_float(r[4 * v + 2]),
                                                       __uint_as_float(r[4 * v + 3]));
                                if (p.beta != 0.f) {
                                    const float4 old = *reinterpret_cast<const float4*>(orow32 + v * 4);
                                    o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                                }
                                *reinterpret_cast<float4*>(orow32 + v * 4) = o;
                            }
                        }
                    }
                } else if (WG) {
                    if (row_ok && nb < p.N) {
                        float* prow = p.partial + ((long long)z * p.M + m) * p.N + nb;
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            if (nb + v * 4 < p.N)   // N is a multiple of 8
                                *reinterpret_cast<uint4*>(prow + v * 4) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                    }
                } else if (pair) {
                    // The warp that produces what its partner needs writes one of two sets of exchange rows and the two meet at
                    // a barrier; with two sets the producer runs up to one set ahead.  Both warps pass every barrier of every
                    // chunk, whatever their rows and columns.
                    const bool live = row_ok && nb < p.N;
                    if constexpr (PAIR == 1) {
                        uint32_t* xrow = (c & 1) ? xrow1 : xrow0;
                        if (!tangent) {
                            if (live) {
                                const float* sb = sb_warp + c * 32;
                                switch (p.act) {
                                    case MPODE_ACT_SOFTPLUS: epilogue_chunk<T, MPODE_ACT_SOFTPLUS, true>(r, sb, false, false, hv, orow, nb, p.N, xrow); break;
                                    case MPODE_ACT_RELU: epilogue_chunk<T, MPODE_ACT_RELU, true>(r, sb, false, false, hv, orow, nb, p.N, xrow); break;
                                    case MPODE_ACT_TANH: epilogue_chunk<T, MPODE_ACT_TANH, true>(r, sb, false, false, hv, orow, nb, p.N, xrow); break;
                                    default: epilogue_chunk<T, MPODE_ACT_NONE, true>(r, sb, false, false, hv, orow, nb, p.N, xrow); break;
                                }
                            }
                            __syncwarp();
                            pair_sync(pair_id);
                        } else {
                            pair_sync(pair_id);
                            if (live) {
                                T* grow = p.pair_out != nullptr ? (T*)p.pair_out + (long long)m * p.ldo : nullptr;
                                switch (p.act) {
                                    case MPODE_ACT_SOFTPLUS: tangent_chunk<T, MPODE_ACT_SOFTPLUS>(r, xrow, orow, grow, nb, p.N); break;
                                    case MPODE_ACT_RELU: tangent_chunk<T, MPODE_ACT_RELU>(r, xrow, orow, grow, nb, p.N); break;
                                    case MPODE_ACT_TANH: tangent_chunk<T, MPODE_ACT_TANH>(r, xrow, orow, grow, nb, p.N); break;
                                    default: tangent_chunk<T, MPODE_ACT_NONE>(r, xrow, orow, grow, nb, p.N); break;
                                }
                            }
                            __syncwarp();
                        }
                    } else {
                        // gbar crosses in two sets of 16 columns; each warp works on a half as soon as it has what it needs
                        uint32_t packed[16];
                        float gb[16];
                        if (tangent) {
                            if (live) {
#pragma unroll
                                for (int v = 0; v < 4; ++v) *reinterpret_cast<uint4*>(xrow0 + 4 * v) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                            }
                            __syncwarp();
                            pair_sync(pair_id);
                            if (live) {
#pragma unroll
                                for (int v = 0; v < 4; ++v)
                                    *reinterpret_cast<uint4*>(xrow1 + 4 * v) = make_uint4(r[16 + 4 * v], r[17 + 4 * v], r[18 + 4 * v], r[19 + 4 * v]);
                            }
                            __syncwarp();
                            pair_sync(pair_id);
                        }
#define MPODE_CNF_HALF(HF)                                                                                                            \
    do {                                                                                                                              \
        if (!tangent) {                                                                                                               \
            pair_sync(pair_id);                                                                                                       \
            if (live) {                                                                                                               \
                const uint32_t* xr = (HF) ? xrow1 : xrow0;                                                                            \
                _Pragma("unroll") for (int v = 0; v < 4; ++v) *reinterpret_cast<float4*>(gb + 4 * v) =                                \
                    *reinterpret_cast<const float4*>(xr + 4 * v);                                                                     \
            }                                                                                                                         \
        }                                                                                                                             \
        if (live) {                                                                                                                   \
            switch (p.act) {                                                                                                          \
                case MPODE_ACT_SOFTPLUS: bad |= cnf_backward_half<T, MPODE_ACT_SOFTPLUS, HF>(r, tangent, gb, hv, uv, packed, nb, p.N); break; \
                case MPODE_ACT_RELU: bad |= cnf_backward_half<T, MPODE_ACT_RELU, HF>(r, tangent, gb, hv, uv, packed, nb, p.N); break; \
                case MPODE_ACT_TANH: bad |= cnf_backward_half<T, MPODE_ACT_TANH, HF>(r, tangent, gb, hv, uv, packed, nb, p.N); break; \
                default: bad |= cnf_backward_half<T, MPODE_ACT_NONE, HF>(r, tangent, gb, hv, uv, packed, nb, p.N); break;              \
            }                                                                                                                         \
        }                                                                                                                             \
        __syncwarp();                                                                                                                 \
    } while (0)
                        MPODE_CNF_HALF(0);
                        MPODE_CNF_HALF(1);
#undef MPODE_CNF_HALF
                        if (live) store_chunk<T>(orow, nb, p.N, packed);
                        __syncwarp();
                    }
                } else if (p.epi == EPI_RAW32) {
                    if (row_ok && nb < p.N) {      // the wide accumulator itself (consumed by an elementwise kernel)
                        float* prow = (float*)p.out + (long long)m * p.ldo + nb;
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            if (nb + v * 4 < p.N)
                                *reinterpret_cast<uint4*>(prow + v * 4) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                    }
                } else if (row_ok && nb < p.N) {
                    const float* sb = sb_warp + c * 32;
                    const bool with_h = hrow != nullptr;
                    if (p.epi == EPI_FWD && p.conv) {      // bias from the registers filled above
                        switch (p.act) {
                            case MPODE_ACT_SOFTPLUS: epilogue_chunk<T, MPODE_ACT_SOFTPLUS, true>(r, bl, second, false, hv, orow, nb, p.N); break;
                            case MPODE_ACT_RELU: epilogue_chunk<T, MPODE_ACT_RELU, true>(r, bl, second, false, hv, orow, nb, p.N); break;
                            case MPODE_ACT_TANH: epilogue_chunk<T, MPODE_ACT_TANH, true>(r, bl, second, false, hv, orow, nb, p.N); break;
                            default: epilogue_chunk<T, MPODE_ACT_NONE, true>(r, bl, second, false, hv, orow, nb, p.N); break;
                        }
                    } else if (p.epi == EPI_FWD) {
                        switch (p.act) {
                            case MPODE_ACT_SOFTPLUS: epilogue_chunk<T, MPODE_ACT_SOFTPLUS, true>(r, sb, second, false, hv, orow, nb, p.N); break;
                            case MPODE_ACT_RELU: epilogue_chunk<T, MPODE_ACT_RELU, true>(r, sb, second, false, hv, orow, nb, p.N); break;
                            case MPODE_ACT_TANH: epilogue_chunk<T, MPODE_ACT_TANH, true>(r, sb, second, false, hv, orow, nb, p.N); break;
                            default: epilogue_chunk<T, MPODE_ACT_NONE, true>(r, sb, second, false, hv, orow, nb, p.N); break;
                        }
                    } else {
                        switch (p.act) {
                            case MPODE_ACT_SOFTPLUS: bad |= epilogue_chunk<T, MPODE_ACT_SOFTPLUS, false>(r, sb, false, with_h, hv, orow, nb, p.N); break;
                            case MPODE_ACT_RELU: bad |= epilogue_chunk<T, MPODE_ACT_RELU, false>(r, sb, false, with_h, hv, orow, nb, p.N); break;
                            case MPODE_ACT_TANH: bad |= epilogue_chunk<T, MPODE_ACT_TANH, false>(r, sb, false, with_h, hv, orow, nb, p.N); break;
                            default: bad |= epilogue_chunk<T, MPODE_ACT_NONE, false>(r, sb, false, with_h, hv, orow, nb, p.N); break;
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

// ---------------------------------------------------------------- host side: launch
template <typename T, int BN, bool WG, int PAIR = 0>
bool launch_tc(const CUtensorMap& ta, const CUtensorMap& tb, TcParams& p, cudaStream_t st) {
    using Cfg = TileCfg<BN>;
    static bool attr_set[kMaxDevices] = {false};
    const int dev = current_device();
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(gemm_tc_kernel<T, BN, WG, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess)
            return false;
        attr_set[dev] = true;
    }
    p.tiles_m = (p.M + BM - 1) / BM;                 // paired tiles: M = 2 m_split, m_split a multiple of 64
    p.tiles_n = (p.N + BN - 1) / BN;
    int work = p.tiles_m * p.tiles_n * p.splits;
    const int max_ctas = sm_count() * Shape<BN>::kCtasPerSm;
    int grid = work < max_ctas ? work : max_ctas;
    gemm_tc_kernel<T, BN, WG, PAIR><<<grid, Shape<BN>::kThreads, Cfg::kSmemBytes, st>>>(ta, tb, p);
    return true;
}

}  // namespace

bool tc_eligible(mpode_dtype dt, const GemmArgs& g) {
    if (dt != MPODE_BF16 && dt != MPODE_F16) return false;
    if (g.epi != EPI_FWD && g.epi != EPI_DGRAD && g.epi != EPI_RAW32) return false;
    if (g.epi == EPI_RAW32 && (g.conv_on != 0 || g.out2 != nullptr)) return false;
    if (g.conv_on == 2 || g.split_k > 1) return false;
    if (g.conv_on == 1) {
        // tensor-core convolution: channels in pieces of 64 (a k-block is one piece of one tap), tiles of whole image rows
        if (g.conv_cd % 64 != 0 || g.conv_cd > 512 || g.conv_ct != g.conv_cd || g.K != 9 * g.conv_cd || g.out2 != nullptr) return false;
        if (g.conv_w < 8 || g.conv_w > 128 || (128 % g.conv_w) != 0 || g.conv_h < 2 || g.conv_h % (128 / g.conv_w) != 0) return false;
        if (g.M % (g.conv_h * g.conv_w) != 0) return false;
        if (g.epi == EPI_FWD && g.conv_tbias == nullptr) return false;
        if (g.b_ks != 1 || g.N % 8 != 0 || g.b_rs % 8 != 0 || g.ldo % 8 != 0) return false;
        if (g.hprev != nullptr && g.ldh % 8 != 0) return false;
        if (((uintptr_t)g.A | (uintptr_t)g.B | (uintptr_t)g.out | (uintptr_t)g.hprev) & 15) return false;
        return g.err != nullptr;
    }
    if (g.cnf_pair != 0) {
        if (g.conv_on != 0 || g.out2 == nullptr || g.m_split <= 0 || g.m_split % 64 != 0 || g.M != 2 * g.m_split) return false;
        if (g.cnf_pair == 1 && g.epi != EPI_FWD) return false;
        if (g.cnf_pair == 2 && (g.epi != EPI_DGRAD || g.hprev == nullptr || g.uprev == nullptr || ((uintptr_t)g.uprev & 15))) return false;
        if (g.pair_out != nullptr && ((uintptr_t)g.pair_out & 15)) return false;
    }
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
    if (g.cnf_pair != 0 && bn == 64) bn = 128;      // the paired tiles come 128 and 256 columns wide
    CUtensorMap ta, tb;
    if (g.conv_on == 1) {
        if (!get_tensor_map_nhwc(g.A, g.M / (g.conv_h * g.conv_w), g.conv_h, g.conv_w, g.conv_cd, 128 / g.conv_w, dt, &ta)) return false;
    } else if (!get_tensor_map(g.A, g.M, g.K, g.a_rs, g.cnf_pair != 0 ? 64 : BM, dt, &ta)) {
        return false;
    }
    if (!get_tensor_map(g.B, g.N, g.K, g.b_rs, bn, dt, &tb)) return false;
    TcParams p{};
    p.conv = g.conv_on == 1; p.conv_h = g.conv_h; p.conv_w = g.conv_w; p.conv_c = g.conv_cd; p.tbias = g.conv_tbias;
    p.M = g.M; p.N = g.N; p.K = g.K; p.epi = g.epi;
    p.out = g.out; p.ldo = g.ldo; p.out2 = g.out2; p.m_split = g.m_split;
    p.bias = g.bias; p.wt = g.wt; p.tau = g.tau; p.act = g.act;
    p.hprev = g.hprev; p.ldh = g.ldh; p.flag = g.flag; p.err = g.err;
    p.pair = g.cnf_pair; p.pair_out = g.pair_out; p.uprev = g.uprev;
    p.splits = 1; p.kb_per_split = (g.K + BK - 1) / BK; p.partial = nullptr;
    bool ok;
    if (g.cnf_pair != 0) {
        if (dt == MPODE_BF16 && g.cnf_pair == 1)
            ok = bn == 256 ? launch_tc<__nv_bfloat16, 256, false, 1>(ta, tb, p, st) : launch_tc<__nv_bfloat16, 128, false, 1>(ta, tb, p, st);
        else if (dt == MPODE_BF16)
            ok = bn == 256 ? launch_tc<__nv_bfloat16, 256, false, 2>(ta, tb, p, st) : launch_tc<__nv_bfloat16, 128, false, 2>(ta, tb, p, st);
        else if (g.cnf_pair == 1)
            ok = bn == 256 ? launch_tc<__half, 256, false, 1>(ta, tb, p, st) : launch_tc<__half, 128, false, 1>(ta, tb, p, st);
        else
            ok = bn == 256 ? launch_tc<__half, 256, false, 2>(ta, tb, p, st) : launch_tc<__half, 128, false, 2>(ta, tb, p, st);
    } else if (dt == MPODE_BF16) {
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
    int sms = sm_count();
    // estimated time in microseconds: waves of work items at ~0.5 us per k-block of a 128 x 256 tile, plus (with more
    // than one slice) the pass that reads the slices back and adds them
    int best = 1;
    double best_t = 1e30;
    for (int s = 1; s <= 16 && s <= kb_total; ++s) {
        int work = tiles * s;
        int waves = (work + sms - 1) / sms;
        int per_s = (kb_total + s - 1) / s;
        double t = (double)waves * per_s * 0.5 * bn / 256.0;
        if (s > 1) t += (double)(s + 2) * M * N * 4.0 / 3.0e6 + 5.0;
        if (t < best_t) { best_t = t; best = s; }
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


bool launch_wgrad_tc(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* launches) {
    int bn, splits, per;
    wgrad_plan(g.M, g.N, g.K, &bn, &splits, &per);
    CUtensorMap ta, tb;
    if (!get_tensor_map(g.A, g.K, g.M, g.a_ks, 64, dt, &ta)) return false;
    if (!get_tensor_map(g.B, g.K, g.N, g.b_ks, 64, dt, &tb)) return false;
    TcParams p{};
    p.M = g.M; p.N = g.N; p.K = g.K; p.epi = EPI_WGRAD; p.err = g.err;
    p.splits = splits; p.kb_per_split = per; p.partial = g.partial;
    p.direct = splits == 1 && g.ldo % 4 == 0 && (((uintptr_t)g.out) & 15) == 0;
    p.out = g.out; p.ldo = g.ldo; p.beta = g.beta;
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
    if (!p.direct) launch_splitk_reduce(g.partial, splits, g.M, g.N, (float*)g.out, g.ldo, g.beta, st, launches);
    return true;
}

// ---------------------------------------------------------------- convolution weight gradient
bool conv_wgrad_tc_eligible(mpode_dtype dt, int B, int H, int W, int C, const void* dz, const void* x, const float* partial,
                            size_t partial_bytes, const unsigned* err) {
    if (dt != MPODE_BF16 && dt != MPODE_F16) return false;
    if (C % 64 != 0 || C > 512 || W < 8 || W > 64 || (64 % W) != 0 || H < 2 || H % (64 / W) != 0) return false;
    if (((uintptr_t)dz | (uintptr_t)x | (uintptr_t)partial) & 15) return false;
    if ((long long)B * H * W < 512 || err == nullptr || partial == nullptr) return false;
    return conv_wgrad_tc_scratch_bytes(B, H, W, C) <= partial_bytes;
}

// Output tiles are 128 (tap, channel) rows by `bn` output channels: 256 wide where the layer has that many (the operand reads of
// a 64-wide MMA cost more shared-memory bandwidth than the tensor pipe can use), and the pixels are cut into slices so that
// tiles x slices fills the SMs.
static int conv_wgrad_bn(int C) { return C % 256 == 0 ? 256 : 64; }

static void conv_wgrad_plan(long long pixels, int C, int* splits, int* per) {
    const int kb_total = (int)(pixels / 64);
    const int bn = conv_wgrad_bn(C);
    const int tiles = ((9 * C + 127) / 128) * (C / bn);
    int s = ((bn == 256 ? 1 : 2) * sm_count() + tiles / 2) / tiles;        // two CTAs share an SM for the narrow tiles
    if (s > 64) s = 64;
    if (s > kb_total / 8) s = kb_total / 8;
    if (s < 1) s = 1;
    *per = (kb_total + s - 1) / s;
    *splits = (kb_total + *per - 1) / *per;
}

size_t conv_wgrad_tc_scratch_bytes(int B, int H, int W, int C) {
    int splits, per;
    conv_wgrad_plan((long long)B * H * W, C, &splits, &per);
    return (size_t)splits * 9 * C * C * sizeof(float);
}

bool launch_conv_wgrad_tc(mpode_dtype dt, const void* dz, const void* x, int B, int H, int W, int C, int ct, float* out, float beta,
                          float* partial, unsigned* err, cudaStream_t st, long long* launches, float sign) {
    const long long pixels = (long long)B * H * W;
    int splits, per;
    conv_wgrad_plan(pixels, C, &splits, &per);
    CUtensorMap ta, tb;
    if (!get_tensor_map_nhwc(x, B, H, W, C, 64 / W, dt, &ta)) return false;
    if (!get_tensor_map(dz, pixels, C, C, 64, dt, &tb)) return false;
    TcParams p{};
    p.M = 9 * C; p.N = C; p.K = (int)pixels; p.epi = EPI_WGRAD; p.err = err;
    p.splits = splits; p.kb_per_split = per; p.partial = partial;
    p.conv = 1; p.conv_h = H; p.conv_w = W; p.conv_c = C;
    bool ok;
    if (conv_wgrad_bn(C) == 256) ok = dt == MPODE_BF16 ? launch_tc<__nv_bfloat16, 256, true>(ta, tb, p, st) : launch_tc<__half, 256, true>(ta, tb, p, st);
    else ok = dt == MPODE_BF16 ? launch_tc<__nv_bfloat16, 64, true>(ta, tb, p, st) : launch_tc<__half, 64, true>(ta, tb, p, st);
    if (!ok) return false;
    if (launches) ++*launches;
    launch_conv_wgrad_reduce(partial, splits, C, ct, out, beta, st, launches, sign);
    return true;
}

}  // namespace mpode
