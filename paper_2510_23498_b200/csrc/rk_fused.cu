// Fused Runge-Kutta step kernel (sm_100a): a persistent, warp-specialised CTA per SM walks the phase table of
// rk_fused.h.  Every phase is one velocity-layer contraction on the 5th-generation tensor cores (TMA-fed shared-memory
// ring, tcgen05.mma into one of two TMEM accumulators, epilogue warps draining the other one) whose epilogue also
// does the memory-bound step of the method that follows it:
//   forward    : stage input Y_{j+1}, fp32 state update and low-precision trajectory store (Alg. 1)
//   backward   : activation-derivative products, stage cotangents kappa_j, overflow flag (Eq. (vjp), Alg. 2)
//   parameters : fp32 partial sums of the weight gradient over slices of the batch
// Tiles are dealt round-robin to the CTAs in one global order; a tile whose operand rows are produced by the phase
// before it waits on that row block's completion counter (bounded wait, error word on give-up, never a trap).
#include "rk_fused.h"

#include <stdio.h>

#include "profiler.h"
#include "tc_ptx.cuh"
#include "tensormap.h"

namespace mpode {
using namespace tc;
namespace {

constexpr int kEpiWarps = 8;                        // kColGroups per TMEM lane quadrant, each takes its share of the tile's columns
constexpr int kColGroups = kEpiWarps / 4;
constexpr int kStrip = 256 / kColGroups;            // widest column range of one epilogue warp
// warp 0: TMA producer, 1: MMA issuer, 2: publisher, then (backward program only) the loader of the stored layer outputs,
// then the epilogue warps
constexpr int kChunk = 16;                          // accumulator columns an epilogue warp handles at a time
constexpr int kABytes = BM * BK * 2;                // 16 KB
constexpr int kBBytes = 256 * BK * 2;               // 32 KB (widest tile)
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kHUnitBytes = 2 * BM * 64 * 2;        // one unit of stored layer outputs: 128 rows x 128 columns (two 64-column boxes)
// The backward program stages the stored layer outputs H (the operand of the activation-derivative product) through two
// shared-memory units filled by bulk loads while the tile's contraction runs; it pays for them with one ring stage.
template <bool BWD> struct Cfg {
    static constexpr int kFirstEpiWarp = BWD ? 4 : 3;
    static constexpr int kThreads = 32 * (kFirstEpiWarp + kEpiWarps);
    static constexpr int kMaxRegs = BWD ? 160 : 168;            // registers are handed out per four warps: 12 warps x 32 x 168 is what fits
    static constexpr int kStages = BWD ? 3 : 4;
    static constexpr int kHBytes = BWD ? 2 * kHUnitBytes : 0;
    static constexpr int kSmemBytes = kStages * kStageBytes + kHBytes + 1024 + kEpiWarps * kStrip * 4 + 256;
};
constexpr int kTmemCols = 512;                      // two accumulators of up to 256 columns

// Tiles of phase `ph`: row blocks x column tiles, or (weight gradient) output tiles x batch slices.
__device__ __forceinline__ int phase_tiles(const RkPhase& ph, int rb) {
    return ph.epi == RK_EPI_WGRAD ? ph.tiles_m * ph.tiles_n * ph.splits : rb * ph.tiles_n;
}

// Static deal of tiles to CTAs.  A phase belongs to one of three queues: 0 = the first `chain_ctas` CTAs (the
// latency-bound per-row-block chains), 1 = the remaining CTAs (bulk work: weight gradients), 2 = all CTAs.  Within a
// queue the tiles of successive phases are dealt round-robin, each queue keeping its own running count, so every role
// of a CTA (producer, issuer, publisher, epilogue) enumerates the same tiles in the same order.
struct Sched {
    long long base[3];
    int cta, G, G0;
    __device__ Sched(int cta_, int G_, int chain) : cta(cta_), G(G_), G0(chain > 0 && chain < G_ ? chain : 0) { base[0] = base[1] = base[2] = 0; }
    // first tile of a phase with nt tiles for this CTA (nt = none) and the stride to its next one
    __device__ int first(int queue, int nt, int& stride) {
        int Gq = G, cq = cta;
        if (G0 == 0) queue = 2;
        else if (queue == 0) { Gq = G0; cq = cta < G0 ? cta : -1; }
        else if (queue == 1) { Gq = G - G0; cq = cta >= G0 ? cta - G0 : -1; }
        const long long b = base[queue];
        base[queue] = b + nt;
        stride = Gq;
        if (cq < 0) return nt;
        return (int)(((long long)cq - b % Gq + Gq) % Gq);
    }
};

// 16 consecutive low-format elements of one row, moved as two 16-byte groups; group v is present iff col0 + 8 v < N
// (N is a multiple of 8).  Loads bypass L1: the data may have been written by another SM during this launch.
template <typename T>
__device__ __forceinline__ void load16_cg(const T* row, int col0, int N, uint32_t (&w)[8]) {
    if ((N & 15) == 0) {      // whole 32-byte sectors per lane (N = 0 marks a lane outside the matrix: zeros)
        if (col0 < N) {
            asm volatile("ld.global.cg.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                         : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                         : "l"(row + col0));
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) w[i] = 0u;
        }
        return;
    }
#pragma unroll
    for (int v = 0; v < 2; ++v) {
        uint4 q = make_uint4(0, 0, 0, 0);
        if (col0 + v * 8 < N) q = __ldcg(reinterpret_cast<const uint4*>(row + col0 + v * 8));
        w[4 * v] = q.x; w[4 * v + 1] = q.y; w[4 * v + 2] = q.z; w[4 * v + 3] = q.w;
    }
}
// Rows whose length is a multiple of 16 elements take one 32-byte store per lane (a whole sector); otherwise two
// guarded 16-byte stores.
template <typename T>
__device__ __forceinline__ void store16(T* row, int col0, int N, const uint32_t (&w)[8]) {
    if ((N & 15) == 0) {
        if (col0 < N)
            asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(row + col0), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                         "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                         : "memory");
        return;
    }
#pragma unroll
    for (int v = 0; v < 2; ++v)
        if (col0 + v * 8 < N)
            *reinterpret_cast<uint4*>(row + col0 + v * 8) = make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
}
template <typename T> __device__ __forceinline__ float lo_f(uint32_t w) { return Low<T>::to_f(from_bits<T>((unsigned short)(w & 0xFFFFu))); }
template <typename T> __device__ __forceinline__ float hi_f(uint32_t w) { return Low<T>::to_f(from_bits<T>((unsigned short)(w >> 16))); }

// acc[i] = fma(c, x[i], acc[i]) over the 16 elements packed in w
template <typename T>
__device__ __forceinline__ void axpy16(float c, const uint32_t (&w)[8], float (&acc)[16]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        acc[2 * i] = fmaf(c, lo_f<T>(w[i]), acc[2 * i]);
        acc[2 * i + 1] = fmaf(c, hi_f<T>(w[i]), acc[2 * i + 1]);
    }
}

// Accumulator load in two halves (issue, then wait).  The wait names the destination registers as read-write operands: no
// use of them can be scheduled before it.
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld16_wait(uint32_t (&r)[16]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                   "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
                 :
                 : "memory");
}
// 16 consecutive elements of one row of a 128-byte-swizzled [rows][64] box in shared memory (16-byte slots j0, j0 + 1)
__device__ __forceinline__ void lds_swizzled16(uint32_t box_addr, int row, int j0, uint32_t (&w)[8]) {
    const uint32_t rowa = box_addr + (uint32_t)row * 128u;
    const uint32_t a0 = rowa + (uint32_t)(((j0) ^ (row & 7)) << 4), a1 = rowa + (uint32_t)(((j0 + 1) ^ (row & 7)) << 4);
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(a0));
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "r"(a1));
}

template <typename T, int ACT>
__device__ __forceinline__ void hidden_chunk(const uint32_t (&r)[16], const float* sb, T* orow, int nb, int N) {
    uint32_t packed[8];
#pragma unroll
    for (int i = 0; i < 16; i += 2)
        packed[i >> 1] = cvt_pack<T>(fast_act<ACT>(__uint_as_float(r[i]) + sb[i]), fast_act<ACT>(__uint_as_float(r[i + 1]) + sb[i + 1]));
    store16<T>(orow, nb, N, packed);
}

template <typename T, int ACT>
__device__ __forceinline__ bool dgrad_chunk(const uint32_t (&r)[16], const uint32_t (&hw)[8], T* orow, int nb, int N,
                                            uint32_t (&packed)[8]) {
    const float lim = OverflowLimit<T>::value();
    bool bad = false;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float v0 = __uint_as_float(r[2 * i]) * fast_act_deriv<ACT>(lo_f<T>(hw[i]));
        float v1 = __uint_as_float(r[2 * i + 1]) * fast_act_deriv<ACT>(hi_f<T>(hw[i]));
        bad |= (nb + 2 * i < N) && !(fabsf(v0) < lim);
        bad |= (nb + 2 * i + 1 < N) && !(fabsf(v1) < lim);
        packed[i] = cvt_pack<T>(v0, v1);
    }
    store16<T>(orow, nb, N, packed);
    return bad;
}

// BWD = false: programs of hidden-layer and stage-output phases (forward loop, recompute); BWD = true: programs of
// input-gradient, psi and weight-gradient phases.  Each instantiation carries only its own epilogues.
template <typename T, bool BWD>
__global__ void __maxnreg__(Cfg<BWD>::kMaxRegs)
rk_fused_kernel(const __grid_constant__ RkMaps maps, const RkParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    constexpr int kStages = Cfg<BWD>::kStages;
    constexpr int kFirstEpiWarp = Cfg<BWD>::kFirstEpiWarp;
    uint8_t* sA = smem;                                    // kStages x [128][64] (or 2 MN-major blocks)
    uint8_t* sB = smem + (size_t)kStages * kABytes;        // kStages x [<=256][64] (or <= 4 MN-major blocks)
    uint8_t* sH = smem + (size_t)kStages * kStageBytes;    // backward: 2 units of stored layer outputs, [2 boxes][128][64] each
    float* sbias = (float*)(sH + Cfg<BWD>::kHBytes);       // [kEpiWarps][kStrip]
    uint64_t* bars = (uint64_t*)(sbias + kEpiWarps * kStrip);
    uint64_t* full_bar = bars;
    uint64_t* empty_bar = bars + kStages;
    uint64_t* tfull_bar = bars + 2 * kStages;
    uint64_t* tempty_bar = bars + 2 * kStages + 2;
    uint64_t* tstored_bar = bars + 2 * kStages + 4;       // every epilogue warp has issued its stores of the tile
    uint64_t* hfull_bar = bars + 2 * kStages + 6;         // [2] a unit of stored layer outputs has landed
    uint64_t* hempty_bar = bars + 2 * kStages + 8;        // [2] every epilogue warp is done with the unit
    uint32_t* tmem_holder = (uint32_t*)(bars + 2 * kStages + 10);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = (int)gridDim.x, cta = (int)blockIdx.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&tfull_bar[a], 1);
            mbar_init(&tempty_bar[a], kEpiWarps + 1);   // epilogue warps + the publisher
            mbar_init(&tstored_bar[a], kEpiWarps);
            mbar_init(&hfull_bar[a], 1);
            mbar_init(&hempty_bar[a], kEpiWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_holder, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *(volatile uint32_t*)tmem_holder;
    const int kb_rows = (p.B + BK - 1) / BK;               // k-blocks of one stage slot when the batch is the reduction index

    if (warp == 0) {
        // ------------------------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            Sched sch(cta, G, p.chain_ctas);
            for (int it = 0; it < p.n_steps && ok; ++it) {
                const int step = p.step0 + it * p.step_dir;
                for (int q = 0; q < p.n_phases && ok; ++q) {
                    const RkPhase ph = p.phases[q];
                    const int nt = phase_tiles(ph, p.rb);
                    const CUtensorMap* ta = &maps.m[ph.a_map];
                    const CUtensorMap* tb = &maps.m[ph.b_map];
                    int tstep;
                    for (int t = sch.first(ph.queue, nt, tstep); t < nt && ok; t += tstep) {
                        if (ph.epi != RK_EPI_WGRAD) {
                            const int m = t / ph.tiles_n, n = t - m * ph.tiles_n;
                            if (ph.dep_phase >= 0 && it + 1 - ph.dep_prev_iter > 0) {
                                const unsigned target = (unsigned)(it + 1 - ph.dep_prev_iter) * (unsigned)p.phases[ph.dep_phase].tiles_n + (unsigned)ph.dep_extra;
                                ok = wait_counter_ge(p.cnt + (size_t)ph.dep_phase * p.cnt_stride + m, target, p.err, 16u, p.wait_ns);
                                if (!ok) break;
                                fence_proxy_async_all();
                            }
                            if (ph.wait_wg_total > 0) {
                                const unsigned target = (unsigned)it * (unsigned)p.wg_items_per_step + (unsigned)ph.wait_wg_total;
                                ok = wait_counter_ge(p.cnt + (size_t)p.n_phases * p.cnt_stride + 1, target, p.err, 128u, p.wait_ns);
                                if (!ok) break;
                            }
                            const int zslot = ph.a_slot + ph.a_slot_step * step;
                            const int kbs = (ph.K + BK - 1) / BK;
                            const uint32_t bytes = (uint32_t)(kABytes + ph.bn * BK * 2);
                            for (int kb = 0; kb < kbs; ++kb) {
                                ok = mbar_wait(&empty_bar[s], phase ^ 1u, p.err, 1u, p.wait_ns);
                                if (!ok) break;
                                mbar_arrive_expect_tx(&full_bar[s], bytes);
                                tma_load_3d(smem_u32(sA + (size_t)s * kABytes), ta, &full_bar[s], kb * BK, m * BM, zslot);
                                tma_load_2d(smem_u32(sB + (size_t)s * kBBytes), tb, &full_bar[s], kb * BK, n * ph.bn);
                                if (++s == kStages) { s = 0; phase ^= 1u; }
                            }
                        } else {
                            // weight gradient: its operands are whole batch slices, so it waits for a tile count of the step
                            // so far, and (when it adds to a previous stage's partial sums) for that stage's same work item
                            const unsigned target = (unsigned)it * (unsigned)p.sync_tiles_per_step + (unsigned)ph.wait_total;
                            ok = wait_counter_ge(p.cnt + (size_t)p.n_phases * p.cnt_stride, target, p.err, 32u, p.wait_ns);
                            if (ok && ph.dep_phase >= 0)
                                ok = wait_counter_ge(p.cnt + (size_t)ph.dep_phase * p.cnt_stride + t, (unsigned)(it + 1), p.err, 32u, p.wait_ns);
                            if (!ok) break;
                            fence_proxy_async_all();
                            const int tiles = ph.tiles_m * ph.tiles_n;
                            const int tile = t % tiles, z = t / tiles;
                            const int m0 = (tile / ph.tiles_n) * BM, n0 = (tile % ph.tiles_n) * ph.bn;
                            const int kb0 = z * ph.kb_per_split, kb1 = min(kb_rows, kb0 + ph.kb_per_split);
                            if (ph.pack2) {
                                // ones-product items (64 output columns) move little per k-block and would be bound by the ring's
                                // round trips: two k-blocks share a stage, the cotangent boxes in the B part (32 KB), the ones in the A part
                                for (int kb = kb0; kb < kb1; kb += 2) {
                                    const int nk = min(2, kb1 - kb);
                                    ok = mbar_wait(&empty_bar[s], phase ^ 1u, p.err, 1u, p.wait_ns);
                                    if (!ok) break;
                                    mbar_arrive_expect_tx(&full_bar[s], (uint32_t)(nk * (kABytes + 8192)));
                                    const uint32_t a_dst = smem_u32(sA + (size_t)s * kABytes), b_dst = smem_u32(sB + (size_t)s * kBBytes);
                                    for (int kk = 0; kk < nk; ++kk) {
                                        const int row = (kb + kk) * BK;
                                        for (int c = 0; c < BM / 64; ++c) tma_load_3d(b_dst + kk * kABytes + c * 8192, ta, &full_bar[s], m0 + c * 64, row, ph.a_slot);
                                        tma_load_3d(a_dst + kk * 8192, tb, &full_bar[s], n0, row, ph.b_slot);
                                    }
                                    if (++s == kStages) { s = 0; phase ^= 1u; }
                                }
                                continue;
                            }
                            const uint32_t bytes = (uint32_t)(kABytes + ph.bn * BK * 2);
                            for (int kb = kb0; kb < kb1; ++kb) {
                                const int row = kb * BK;
                                ok = mbar_wait(&empty_bar[s], phase ^ 1u, p.err, 1u, p.wait_ns);
                                if (!ok) break;
                                mbar_arrive_expect_tx(&full_bar[s], bytes);
                                const uint32_t a_dst = smem_u32(sA + (size_t)s * kABytes), b_dst = smem_u32(sB + (size_t)s * kBBytes);
                                for (int c = 0; c < BM / 64; ++c) tma_load_3d(a_dst + c * 8192, ta, &full_bar[s], m0 + c * 64, row, ph.a_slot);
                                for (int c = 0; c < ph.bn / 64; ++c) tma_load_3d(b_dst + c * 8192, tb, &full_bar[s], n0 + c * 64, row, ph.b_slot);
                                if (++s == kStages) { s = 0; phase ^= 1u; }
                            }
                        }
                    }
                }
            }
            if (!ok) {   // a wait gave up: let bulk copies already in flight land before the CTA winds down
                unsigned long long t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            int k_local = 0;
            bool ok = true;
            Sched sch(cta, G, p.chain_ctas);
            for (int it = 0; it < p.n_steps && ok; ++it) {
                for (int q = 0; q < p.n_phases && ok; ++q) {
                    const RkPhase ph = p.phases[q];
                    const int nt = phase_tiles(ph, p.rb);
                    const bool wg = ph.epi == RK_EPI_WGRAD;
                    const uint32_t idesc = make_idesc(Fmt<T>::id, BM, ph.bn, wg);
                    int tstep;
                    for (int t = sch.first(ph.queue, nt, tstep); t < nt && ok; t += tstep, ++k_local) {
                        int kbs;
                        if (!wg) {
                            kbs = (ph.K + BK - 1) / BK;
                        } else {
                            const int z = t / (ph.tiles_m * ph.tiles_n);
                            const int kb0 = z * ph.kb_per_split;
                            kbs = min(kb_rows, kb0 + ph.kb_per_split) - kb0;
                        }
                        const int acc = k_local & 1;
                        const uint32_t use = (uint32_t)(k_local >> 1);
                        ok = mbar_wait(&tempty_bar[acc], (use & 1u) ^ 1u, p.err, 2u, p.wait_ns);
                        if (!ok) break;
                        tc_fence_after_sync();
                        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * 256);
                        if (wg && ph.pack2) {
                            for (int kb = 0; kb < kbs; kb += 2) {
                                const int nk = min(2, kbs - kb);
                                ok = mbar_wait(&full_bar[s], phase, p.err, 4u, p.wait_ns);
                                if (!ok) break;
                                tc_fence_after_sync();
                                const uint32_t a_addr = smem_u32(sB + (size_t)s * kBBytes), b_addr = smem_u32(sA + (size_t)s * kABytes);
                                for (int kk = 0; kk < nk; ++kk) {
                                    const uint64_t adesc = smem_desc_mn_major_sw128(a_addr + kk * kABytes), bdesc = smem_desc_mn_major_sw128(b_addr + kk * 8192);
#pragma unroll
                                    for (int k = 0; k < BK / UMMA_K; ++k)
                                        umma_f16(tmem_d, adesc + 128u * (uint64_t)k, bdesc + 128u * (uint64_t)k, idesc, (kb > 0 || kk > 0 || k > 0) ? 1u : 0u);
                                }
                                umma_commit(&empty_bar[s]);
                                if (++s == kStages) { s = 0; phase ^= 1u; }
                            }
                            if (!ok) break;
                            umma_commit(&tfull_bar[acc]);
                            continue;
                        }
                        for (int kb = 0; kb < kbs; ++kb) {
                            ok = mbar_wait(&full_bar[s], phase, p.err, 4u, p.wait_ns);
                            if (!ok) break;
                            tc_fence_after_sync();
                            const uint32_t a_addr = smem_u32(sA + (size_t)s * kABytes), b_addr = smem_u32(sB + (size_t)s * kBBytes);
                            const uint64_t adesc = wg ? smem_desc_mn_major_sw128(a_addr) : smem_desc_k_major_sw128(a_addr);
                            const uint64_t bdesc = wg ? smem_desc_mn_major_sw128(b_addr) : smem_desc_k_major_sw128(b_addr);
                            const uint64_t kstep = wg ? 128u : 2u;
#pragma unroll
                            for (int k = 0; k < BK / UMMA_K; ++k)
                                umma_f16(tmem_d, adesc + kstep * (uint64_t)k, bdesc + kstep * (uint64_t)k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                            umma_commit(&empty_bar[s]);
                            if (++s == kStages) { s = 0; phase ^= 1u; }
                        }
                        if (!ok) break;
                        umma_commit(&tfull_bar[acc]);
                    }
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------------------------ publisher
        // Releases a finished tile to the other CTAs: once all epilogue warps have issued the tile's stores it makes
        // them visible device-wide and bumps the row block's completion counter, so the epilogue warps never wait on
        // a memory fence themselves.
        if (lane == 0) {
            bool ok = true;
            int k_local = 0;
            Sched sch(cta, G, p.chain_ctas);
            for (int it = 0; it < p.n_steps && ok; ++it) {
                for (int q = 0; q < p.n_phases && ok; ++q) {
                    const RkPhase ph = p.phases[q];
                    const int nt = phase_tiles(ph, p.rb);
                    int tstep;
                    for (int t = sch.first(ph.queue, nt, tstep); t < nt && ok; t += tstep, ++k_local) {
                        const int acc = k_local & 1;
                        const uint32_t use = (uint32_t)(k_local >> 1);
                        ok = mbar_wait(&tstored_bar[acc], use & 1u, p.err, 64u, p.wait_ns);
                        if (!ok) break;
                        // one device-scope fence orders the epilogue warps' stores (observed through the shared-memory barrier)
                        // before the counter updates; the consuming CTA orders its bulk loads after its acquire
                        __threadfence();
                        if (ph.epi != RK_EPI_WGRAD) {
                            atomicAdd(p.cnt + (size_t)q * p.cnt_stride + t / ph.tiles_n, 1u);
                            atomicAdd(p.cnt + (size_t)p.n_phases * p.cnt_stride, 1u);
                        } else {
                            atomicAdd(p.cnt + (size_t)q * p.cnt_stride + t, 1u);
                            atomicAdd(p.cnt + (size_t)p.n_phases * p.cnt_stride + 1, 1u);
                        }
                        // the accumulator is reused two tiles later: holding it until this tile is published keeps the
                        // epilogue warps from ever running two phases of tstored_bar ahead of this thread
                        mbar_arrive(&tempty_bar[acc]);
                    }
                }
            }
        }
    } else if (BWD && warp == 3) {
        // ------------------------------------------------------------------------------------ loader of stored layer outputs
        // Backward program: the input-gradient epilogues multiply the accumulator by the activation derivative taken from
        // the stored layer output H.  H was written by the recompute launch, so it has no dependency inside this launch:
        // this thread streams it into two shared-memory units ahead of the epilogue warps (a 256-wide tile is two units of
        // 128 columns, a narrower tile one unit), bounded only by the units being free again.
        if (lane == 0) {
            bool ok = true;
            unsigned u = 0;
            Sched sch(cta, G, p.chain_ctas);
            for (int it = 0; it < p.n_steps && ok; ++it) {
                for (int q = 0; q < p.n_phases && ok; ++q) {
                    const RkPhase ph = p.phases[q];
                    const int nt = phase_tiles(ph, p.rb);
                    int tstep;
                    for (int t = sch.first(ph.queue, nt, tstep); t < nt && ok; t += tstep) {
                        if (ph.epi != RK_EPI_DGRAD) continue;
                        const int m = t / ph.tiles_n, n = t - m * ph.tiles_n;
                        const int units = ph.bn == 256 ? 2 : 1;
                        const int boxes = ph.bn == 256 ? 2 : (ph.bn + 63) / 64;
                        for (int uu = 0; uu < units && ok; ++uu, ++u) {
                            const int buf = (int)(u & 1u);
                            ok = mbar_wait(&hempty_bar[buf], ((u >> 1) & 1u) ^ 1u, p.err, 256u, p.wait_ns);
                            if (!ok) break;
                            mbar_arrive_expect_tx(&hfull_bar[buf], (uint32_t)(boxes * BM * 128));
                            for (int bx = 0; bx < boxes; ++bx)
                                tma_load_3d(smem_u32(sH + (size_t)buf * kHUnitBytes + (size_t)bx * BM * 128), &maps.m[ph.h_map], &hfull_bar[buf],
                                            n * ph.bn + uu * 128 + bx * 64, m * BM, ph.h_slot);
                        }
                    }
                }
            }
            if (!ok) {   // as in the producer: let bulk copies in flight land before the CTA winds down
                unsigned long long t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
    } else {
        // ------------------------------------------------------------------------------------ epilogue warps
        const int ew = warp - kFirstEpiWarp;
        const int q4 = warp & 3;                 // TMEM lane quadrant this warp may read
        const int cg = ew >> 2;                  // which half of the tile's columns (of each unit, for two-unit tiles)
        float* sb_warp = sbias + ew * kStrip;
        bool bad = false;
        bool ok = true;
        int k_local = 0;
        unsigned u_local = 0;                    // units of stored layer outputs consumed so far (same count as the loader's)
        Sched sch(cta, G, p.chain_ctas);
        for (int it = 0; it < p.n_steps && ok; ++it) {
            const int step = p.step0 + it * p.step_dir;
            const RkStepScalars* sc = p.scalars + step;
            for (int q = 0; q < p.n_phases && ok; ++q) {
                // the fields this role needs, read one by one (a whole-struct copy would live in local memory)
                const RkPhase* gp = p.phases + q;
                struct { int N, epi, layer, tiles_n, tiles_m, splits, stage, bn, out_slot, act, M, queue, accumulate; long long part_off; } ph;
                ph.N = gp->N; ph.epi = gp->epi; ph.layer = gp->layer; ph.tiles_n = gp->tiles_n; ph.tiles_m = gp->tiles_m; ph.splits = gp->splits;
                ph.stage = gp->stage; ph.bn = gp->bn; ph.out_slot = gp->out_slot; ph.act = gp->act; ph.M = gp->M; ph.queue = gp->queue;
                ph.accumulate = gp->accumulate; ph.part_off = gp->part_off;
                const int nt = ph.epi == RK_EPI_WGRAD ? ph.tiles_m * ph.tiles_n * ph.splits : p.rb * ph.tiles_n;
                const int cols_per_warp = ph.bn / kColGroups;
                const int chunks = cols_per_warp / kChunk;
                const bool two_units = BWD && ph.epi == RK_EPI_DGRAD && ph.bn == 256;
                int tstep;
                for (int t = sch.first(ph.queue, nt, tstep); t < nt && ok; t += tstep, ++k_local) {
                    const int acc = k_local & 1;
                    const uint32_t use = (uint32_t)(k_local >> 1);
                    int m0, tile_n0, zsplit = 0;
                    if (ph.epi != RK_EPI_WGRAD) {
                        const int m = t / ph.tiles_n, n = t - m * ph.tiles_n;
                        m0 = m * BM; tile_n0 = n * ph.bn;
                    } else {
                        const int tiles = ph.tiles_m * ph.tiles_n;
                        const int tile = t % tiles;
                        zsplit = t / tiles;
                        m0 = (tile / ph.tiles_n) * BM; tile_n0 = (tile % ph.tiles_n) * ph.bn;
                    }
                    // column offset of chunk c inside the tile: a warp's chunks are consecutive, except for two-unit tiles,
                    // where the first half of its chunks lies in columns [0, 128) and the second half in [128, 256)
                    auto chunk_col = [&](int c) __attribute__((always_inline)) -> int {
                        return two_units ? (c >> 2) * 128 + cg * 64 + (c & 3) * kChunk : cg * cols_per_warp + c * kChunk;
                    };
                    if (ph.epi == RK_EPI_HIDDEN || ph.epi == RK_EPI_STAGE_OUT) {
                        const T* bias = (const T*)p.bias[ph.layer];
                        const T* wt = (ph.layer == 0) ? (const T*)p.wt : nullptr;
                        const float tau = sc->tau16[ph.stage];
                        for (int c = lane; c < cols_per_warp; c += 32) {
                            const int n = tile_n0 + cg * cols_per_warp + c;
                            float b = 0.f;
                            if (n < ph.N) {
                                if (bias != nullptr) b = Low<T>::to_f(bias[n]);
                                if (wt != nullptr) b = fmaf(tau, Low<T>::to_f(wt[n]), b);
                            }
                            sb_warp[c] = b;
                        }
                        __syncwarp();
                    }
                    ok = mbar_wait(&tfull_bar[acc], use & 1u, p.err, 8u, p.wait_ns);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const int m = m0 + q4 * 32 + lane;
                    const uint32_t tcol = tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(acc * 256);

                    // everything one chunk of 16 accumulator columns needs; `r` holds the accumulator values
                    auto process = [&](const int c, const uint32_t (&r)[kChunk]) __attribute__((always_inline)) {
                        const int nb = tile_n0 + chunk_col(c);
                        if (BWD && ph.epi == RK_EPI_WGRAD) {
                            if (m < ph.M && nb < ph.N) {
                                float* prow = p.partial + ph.part_off + ((long long)zsplit * ph.M + m) * ph.N + nb;
#pragma unroll
                                for (int v = 0; v < 2; ++v) {
                                    if (nb + v * 8 < ph.N) {      // N is a multiple of 8: 32-byte pieces are whole
                                        float o[8];
#pragma unroll
                                        for (int e = 0; e < 8; ++e) o[e] = __uint_as_float(r[8 * v + e]);
                                        if (ph.accumulate) {
                                            float q[8];
                                            asm volatile("ld.global.cg.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                                                         : "=f"(q[0]), "=f"(q[1]), "=f"(q[2]), "=f"(q[3]), "=f"(q[4]), "=f"(q[5]), "=f"(q[6]), "=f"(q[7])
                                                         : "l"(prow + v * 8));
#pragma unroll
                                            for (int e = 0; e < 8; ++e) o[e] += q[e];
                                        }
                                        asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(prow + v * 8), "f"(o[0]),
                                                     "f"(o[1]), "f"(o[2]), "f"(o[3]), "f"(o[4]), "f"(o[5]), "f"(o[6]), "f"(o[7])
                                                     : "memory");
                                    }
                                }
                            }
                            return;
                        }
                        const bool valid = m < p.B && nb < ph.N;
                        if (BWD && ph.epi == RK_EPI_DGRAD) {
                            // the input gradient of layer `ph.layer` passes through the derivative of the activation below it, taken
                            // from the stored layer output in the shared-memory unit
                            const int per_unit = two_units ? 4 : chunks;
                            const unsigned uidx = u_local + (two_units ? (unsigned)(c >> 2) : 0u);
                            const int buf = (int)(uidx & 1u);
                            if ((c % per_unit) == 0) {
                                bool hok = mbar_wait(&hfull_bar[buf], (uidx >> 1) & 1u, p.err, 512u, p.wait_ns);
                                if (!__all_sync(0xffffffffu, hok)) ok = false;
                            }
                            const int x = two_units ? cg * 64 + (c & 3) * kChunk : cg * cols_per_warp + c * kChunk;   // column inside the unit
                            uint32_t hw[8];
                            lds_swizzled16(smem_u32(sH + (size_t)buf * kHUnitBytes + (size_t)(x >> 6) * BM * 128), q4 * 32 + lane, (x & 63) >> 3, hw);
                            if (valid) {
                                T* orow = (T*)p.dzslab[ph.layer] + (long long)ph.out_slot * p.dz_slot_stride[ph.layer] + (long long)m * ph.N;
                                uint32_t out[8];
                                switch (ph.act) {
                                    case MPODE_ACT_SOFTPLUS: bad |= dgrad_chunk<T, MPODE_ACT_SOFTPLUS>(r, hw, orow, nb, ph.N, out); break;
                                    case MPODE_ACT_RELU: bad |= dgrad_chunk<T, MPODE_ACT_RELU>(r, hw, orow, nb, ph.N, out); break;
                                    case MPODE_ACT_TANH: bad |= dgrad_chunk<T, MPODE_ACT_TANH>(r, hw, orow, nb, ph.N, out); break;
                                    default: bad |= dgrad_chunk<T, MPODE_ACT_NONE>(r, hw, orow, nb, ph.N, out); break;
                                }
                            }
                            if ((c % per_unit) == per_unit - 1) {      // this warp is done with the unit
                                __syncwarp();
                                if (lane == 0) mbar_arrive(&hempty_bar[buf]);
                            }
                            return;
                        }
                        if (!valid) return;
                        const float* sb = sb_warp + c * kChunk;
                        if (!BWD && ph.epi == RK_EPI_HIDDEN) {
                            T* orow = (T*)p.hslab[ph.layer + 1] + (long long)ph.out_slot * p.h_slot_stride[ph.layer + 1] + (long long)m * ph.N;
                            switch (ph.act) {
                                case MPODE_ACT_SOFTPLUS: hidden_chunk<T, MPODE_ACT_SOFTPLUS>(r, sb, orow, nb, ph.N); break;
                                case MPODE_ACT_RELU: hidden_chunk<T, MPODE_ACT_RELU>(r, sb, orow, nb, ph.N); break;
                                case MPODE_ACT_TANH: hidden_chunk<T, MPODE_ACT_TANH>(r, sb, orow, nb, ph.N); break;
                                default: hidden_chunk<T, MPODE_ACT_NONE>(r, sb, orow, nb, ph.N); break;
                            }
                        } else if (!BWD && ph.epi == RK_EPI_STAGE_OUT) {
                            // k_j, rounded once; everything after it works on the rounded values
                            const int j = ph.stage, d = p.d;
                            const long long slab = (long long)p.B * d;
                            const long long roff = (long long)m * d;
                            // the operands of what follows are requested first, all at once, so that their latencies overlap
                            uint32_t kw[RK_MAX_STAGES - 1][8], w[8];
                            float4 yy[4];
                            const bool last = j + 1 == p.stages;
                            if (!last) {
                                load16_cg<T>((const T*)p.traj + (long long)step * slab + roff, nb, d, w);
#pragma unroll
                                for (int l = 0; l < RK_MAX_STAGES - 1; ++l)
                                    if (l < j && sc->ha[j + 1][l] != 0.f) load16_cg<T>((const T*)p.kslab + l * slab + roff, nb, d, kw[l]);
                            } else if (p.y != nullptr) {
#pragma unroll
                                for (int l = 0; l < RK_MAX_STAGES - 1; ++l)
                                    if (l < j) load16_cg<T>((const T*)p.kslab + l * slab + roff, nb, d, kw[l]);
#pragma unroll
                                for (int v = 0; v < 4; ++v)
                                    if (nb + v * 4 < d) yy[v] = __ldcg(reinterpret_cast<const float4*>(p.y + (long long)m * p.D + nb + v * 4));
                            }
                            uint32_t kq[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                kq[i] = cvt_pack<T>(__uint_as_float(r[2 * i]) + sb[2 * i], __uint_as_float(r[2 * i + 1]) + sb[2 * i + 1]);
                            store16<T>((T*)p.kslab + j * slab + roff, nb, d, kq);
                            float a[kChunk];
                            if (!last) {
                                // next stage input from the stored low-precision state and the stage derivatives so far
#pragma unroll
                                for (int i = 0; i < 8; ++i) { a[2 * i] = lo_f<T>(w[i]); a[2 * i + 1] = hi_f<T>(w[i]); }
#pragma unroll
                                for (int l = 0; l < RK_MAX_STAGES - 1; ++l) {
                                    const float cf = l < j ? sc->ha[j + 1][l] : 0.f;
                                    if (cf != 0.f) axpy16<T>(cf, kw[l], a);
                                }
                                if (sc->ha[j + 1][j] != 0.f) axpy16<T>(sc->ha[j + 1][j], kq, a);
#pragma unroll
                                for (int i = 0; i < 8; ++i) w[i] = cvt_pack<T>(a[2 * i], a[2 * i + 1]);
                                store16<T>((T*)p.yslab + (j + 1) * slab + roff, nb, d, w);
                            } else if (p.y != nullptr) {
                                // y <- y + h Phi in fp32, then the low-precision copy of the new state
#pragma unroll
                                for (int i = 0; i < kChunk; ++i) a[i] = 0.f;
#pragma unroll
                                for (int l = 0; l < RK_MAX_STAGES - 1; ++l)
                                    if (l < j) axpy16<T>(sc->hb[l], kw[l], a);
                                axpy16<T>(sc->hb[j], kq, a);
                                float* yrow = p.y + (long long)m * p.D + nb;
#pragma unroll
                                for (int v = 0; v < 4; ++v) {
                                    if (nb + v * 4 < d) {
                                        float inc[4];
#pragma unroll
                                        for (int e = 0; e < 4; ++e)
                                            inc[e] = p.round_increment ? sc->h * Low<T>::to_f(Low<T>::from_f(a[4 * v + e])) : a[4 * v + e];
                                        yy[v].x += inc[0]; yy[v].y += inc[1]; yy[v].z += inc[2]; yy[v].w += inc[3];
                                        *reinterpret_cast<float4*>(yrow + v * 4) = yy[v];
                                        a[4 * v] = yy[v].x; a[4 * v + 1] = yy[v].y; a[4 * v + 2] = yy[v].z; a[4 * v + 3] = yy[v].w;
                                    }
                                }
#pragma unroll
                                for (int i = 0; i < 8; ++i) w[i] = cvt_pack<T>(a[2 * i], a[2 * i + 1]);
                                store16<T>((T*)p.traj + (long long)(step + 1) * slab + roff, nb, d, w);
                            }
                        } else if (BWD) {   // RK_EPI_PSI
                            const int j = ph.stage, d = p.d;
                            const long long slab = (long long)p.B * d, roff = (long long)m * d;
                            const float lim = OverflowLimit<T>::value();
                            // operands of the stage cotangent below, requested together
                            uint32_t pre[8];
                            if (j > 0) load16_cg<T>((const T*)p.v + roff, nb, d, pre);
                            uint32_t pq[8], w[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const float v0 = __uint_as_float(r[2 * i]), v1 = __uint_as_float(r[2 * i + 1]);
                                bad |= (nb + 2 * i < d) && !(fabsf(v0) < lim);
                                bad |= (nb + 2 * i + 1 < d) && !(fabsf(v1) < lim);
                                pq[i] = cvt_pack<T>(v0, v1);
                            }
                            store16<T>((T*)p.psislab + j * slab + roff, nb, d, pq);
                            if (j > 0) {
                                // cotangent of the stage below: kappa_{j-1} = Q16(b_{j-1} v + sum_{l >= j} (h a_{l,j-1}) psi_l)
                                float a[kChunk];
                                const float bj = sc->b[j - 1];
#pragma unroll
                                for (int i = 0; i < 8; ++i) { a[2 * i] = bj * lo_f<T>(pre[i]); a[2 * i + 1] = bj * hi_f<T>(pre[i]); }
                                if (sc->ha[j][j - 1] != 0.f) axpy16<T>(sc->ha[j][j - 1], pq, a);
                                for (int l = j + 1; l < p.stages; ++l) {     // tableaux with entries below the first subdiagonal
                                    const float cf = sc->ha[l][j - 1];
                                    if (cf != 0.f) {
                                        load16_cg<T>((const T*)p.psislab + l * slab + roff, nb, d, w);
                                        axpy16<T>(cf, w, a);
                                    }
                                }
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    bad |= (nb + 2 * i < d) && !(fabsf(a[2 * i]) < lim);
                                    bad |= (nb + 2 * i + 1 < d) && !(fabsf(a[2 * i + 1]) < lim);
                                    w[i] = cvt_pack<T>(a[2 * i], a[2 * i + 1]);
                                }
                                store16<T>((T*)p.kappaslab + (long long)((j - 1) % 3) * slab + roff, nb, d, w);
                            }
                        }
                    };

                    // (issuing the accumulator load of the next chunk before this chunk's arithmetic was measured: slower)
                    uint32_t r0[kChunk];
#pragma unroll 1
                    for (int c = 0; c < chunks; ++c) {
                        __syncwarp();
                        tmem_ld16_issue(tcol + (uint32_t)chunk_col(c), r0);
                        tmem_ld16_wait(r0);
                        process(c, r0);
                    }
                    if (BWD && ph.epi == RK_EPI_DGRAD) u_local += two_units ? 2u : 1u;
                    // accumulator drained and stores issued: hand the accumulator back, tell the publisher
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(&tempty_bar[acc]);
                        mbar_arrive(&tstored_bar[acc]);
                    }
                }
            }
        }
        warp_flag_or(p.flag, bad);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// The CTAs of one launch hand tiles to each other, so all of them must be resident together: a cooperative launch makes the
// driver guarantee that (or refuse the launch) instead of leaving it to the device being otherwise idle.
template <typename T, bool BWD>
bool launch_t(const RkMaps& maps, const RkParams& p, cudaStream_t st) {
    static bool attr_set[kMaxDevices] = {false};
    const int dev = current_device();
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(rk_fused_kernel<T, BWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<BWD>::kSmemBytes) != cudaSuccess)
            return false;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)sm_count());
    cfg.blockDim = dim3(Cfg<BWD>::kThreads);
    cfg.dynamicSmemBytes = Cfg<BWD>::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cudaError_t le = cudaLaunchKernelEx(&cfg, rk_fused_kernel<T, BWD>, maps, p);
    if (le != cudaSuccess) {
        cudaFuncAttributes fa{};
        cudaFuncGetAttributes(&fa, rk_fused_kernel<T, BWD>);
        int occ = -1;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, rk_fused_kernel<T, BWD>, Cfg<BWD>::kThreads, Cfg<BWD>::kSmemBytes);
        fprintf(stderr, "rk_fused launch failed: %s; BWD=%d threads=%d dyn_smem=%d regs=%d static_smem=%zu local=%zu maxdyn=%d maxthreads=%d occupancy=%d sms=%d\n",
                cudaGetErrorString(le), (int)BWD, Cfg<BWD>::kThreads, Cfg<BWD>::kSmemBytes, fa.numRegs, fa.sharedSizeBytes, fa.localSizeBytes,
                fa.maxDynamicSharedSizeBytes, fa.maxThreadsPerBlock, occ, sm_count());
    }
    return le == cudaSuccess;
}

}  // namespace

bool launch_rk_fused(mpode_dtype dt, bool backward, const RkMaps& maps, const RkParams& p, cudaStream_t st, long long* launches) {
    bool ok = false;
    if (dt == MPODE_BF16) ok = backward ? launch_t<__nv_bfloat16, true>(maps, p, st) : launch_t<__nv_bfloat16, false>(maps, p, st);
    else if (dt == MPODE_F16) ok = backward ? launch_t<__half, true>(maps, p, st) : launch_t<__half, false>(maps, p, st);
    if (ok && launches) ++*launches;
    if (ok && tl_counters) ++tl_counters->fused;
    return ok;
}

}  // namespace mpode
