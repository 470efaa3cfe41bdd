// Fused Runge-Kutta step kernel for dense (MLP) velocities in the 16-bit formats: one persistent launch walks a
// host-built table of phases (one velocity-layer contraction each, with its fused epilogue) for a range of time
// steps.  Tiles of different phases are ordered by per-row-block completion counters in global memory instead of
// kernel boundaries, so the tensor pipe never drains between layers, stages or steps.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace mpode {

constexpr int RK_MAX_MAPS = 20;
constexpr int RK_MAX_PHASES = 40;
constexpr int RK_MAX_STAGES = 4;

enum RkEpilogue : int {
    RK_EPI_HIDDEN = 0,     // H = Q16(act(acc + b + tau w_t))                               (Alg. 1: increment, hidden layer)
    RK_EPI_STAGE_OUT = 1,  // k_j = Q16(acc + b); then the next stage input Y_{j+1} = Q16(ybar + sum_l (h a_{j+1,l}) k_l),
                           // or after the last stage y += sum_l (h b_l) k_l and traj[i+1] = Q16(y)  (Alg. 1: accumulate, store)
    RK_EPI_DGRAD = 2,      // dZ = Q16(act'(H) * acc), non-finite values raise the flag          (Eq. (vjp))
    RK_EPI_PSI = 3,        // psi_j = Q16(acc); then kappa_{j-1} = Q16(b_{j-1} v + sum_{l>=j} (h a_{l,j-1}) psi_l)
    RK_EPI_WGRAD = 4       // fp32 partial sums of dW over one slice of the batch rows
};

// One contraction C[M = batch rows, N] = A[M, K] B[N, K]^T (or, for RK_EPI_WGRAD, C[M, N] = sum_r A[r, M] B[r, N]).
struct RkPhase {
    int a_map, b_map;          // indices into RkMaps::m
    int a_slot, a_slot_step;   // third TMA coordinate of A: a_slot + a_slot_step * (absolute step index)
    int b_slot;                // RK_EPI_WGRAD: third coordinate of B (stage slot); otherwise unused
    int N, K, bn, tiles_n;
    int epi, act, stage;
    int queue;                 // which CTAs work on this phase: 0 = the chain CTAs, 1 = the others, 2 = all (see RkParams::chain_ctas)
    // What a tile of this phase waits for (all of it earlier in the table's order, so the static schedule cannot lock):
    int dep_phase;             // -1, or the phase that produces this tile's operand rows
    int dep_mode;              // 0: all column tiles of dep_phase in the same row block; 1: the same work item of dep_phase
    int dep_prev_iter;         // 1: dep_phase of the previous step of the launch (nothing to wait for in the first one)
    int dep_extra;             // added to the awaited count; 0 except in the test of the bounded waits (a count that is never reached)
    int wait_total;            // > 0: this many tiles of the current step (weight-gradient tiles not counted) are complete
    int wait_wg_total;         // > 0: this many weight-gradient work items of the current step are complete (they were the
                               // last readers of the buffer slot this phase overwrites)
    int out_slot;              // slot of the output slab this phase writes (hidden layers, dZ)
    int h_slot;                // RK_EPI_DGRAD: slot of the stored layer output whose activation derivative is applied
    int h_map;                 // RK_EPI_DGRAD: tensor map of that layer's output slab, boxes of [128 rows][64 columns]
    int layer;                 // velocity layer (selects bias / output slab)
    // RK_EPI_WGRAD only
    int tiles_m, splits, kb_per_split;          // output tiles along M, batch slices, k-blocks per slice
    int accumulate;            // 1: add to the partial sums already there (a later stage of the same step)
    int pack2;                 // 1: 64-column items whose ring stages hold two k-blocks each (the ones-products)
    long long part_off;        // element offset of this phase's [splits][M][N] partial sums in the fp32 scratch
    int M;                     // output rows (wgrad); batch rows otherwise come from RkParams::B
};

struct RkStepScalars {         // per time step, computed on the host in double and rounded once
    float tau16[RK_MAX_STAGES];                 // Q16(t_i + c_j h)
    float ha[RK_MAX_STAGES][RK_MAX_STAGES];     // h a_jl
    float hb[RK_MAX_STAGES];                    // h b_j (b_j when the increment is rounded first)
    float b[RK_MAX_STAGES];                     // b_j
    float a[RK_MAX_STAGES][RK_MAX_STAGES];      // a_jl and c_j themselves (time-grid gradient)
    float c[RK_MAX_STAGES];
    float h;
    float pad_[3];
};

struct RkMaps { CUtensorMap m[RK_MAX_MAPS]; };

struct RkParams {
    int B, rb, d, D, stages;
    int n_phases, n_steps, step0, step_dir;     // steps step0, step0 + step_dir, ... (n_steps of them)
    int round_increment;
    int chain_ctas;                             // 0: every phase is dealt to all CTAs; else the first chain_ctas CTAs serve queue 0
    int sync_tiles_per_step;                    // tiles per step that are not weight-gradient tiles
    int wg_items_per_step;                      // weight-gradient work items per step
    const RkPhase* phases;                      // device [n_phases]
    const RkStepScalars* scalars;               // device, indexed by absolute step
    unsigned* cnt;                              // device [n_phases][cnt_stride] completion counters + 2 totals (tiles, weight-
                                                // gradient items), zero at launch
    int cnt_stride;                             // >= row blocks and >= work items of any weight-gradient phase
    unsigned* flag;                             // non-finite flag (may be null)
    unsigned* err;                              // bounded-wait failure word
    unsigned long long wait_ns;                 // how long a wait may last before it gives up
    // buffers the epilogues touch directly (low format unless noted)
    const void* bias[8]; const void* wt;        // Q16(b_l), Q16 of the first layer's time column
    void* hslab[8]; long long h_slot_stride[8]; int w[9];   // hidden outputs H_l: [slots][B][w_l]
    void* dzslab[8]; long long dz_slot_stride[8];   // dZ_l: two stage slots of [B][w_l]
    void* kslab; void* yslab; void* psislab;    // [stages][B][d]
    void* kappaslab;                            // [3][B][d]: kappa_j lives in slot j % 3
    const void* v;                              // Q16(S a) [B][d]
    void* traj;                                 // [(N+1)][B][d]
    float* y;                                   // fp32 [B][D]
    float* partial;                             // fp32 scratch of the weight-gradient phases
};

// Launches the kernel on `st` with one CTA per SM; `backward` selects the instantiation that carries the input-gradient,
// psi and weight-gradient epilogues (a program must not mix the two families).  Returns false if it cannot be launched.
bool launch_rk_fused(mpode_dtype dt, bool backward, const RkMaps& maps, const RkParams& p, cudaStream_t st, long long* launches);

}  // namespace mpode
