// The built-in velocity networks as sequences of contraction + fused-epilogue launches.
#include <vector>

#include "conv_tc.h"
#include "gemm_tc.h"
#include "hyper_cnf.h"
#include "profiler.h"
#include "tensormap.h"
#include "tiny_mlp.h"
#include "velocity.h"

namespace mpode {

int launch_contraction(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* L);   // dispatch.cu: returns the kernel taken

namespace {

inline char* at(void* ws, size_t off) { return (char*)ws + off; }

void plan_common(Layout& lay, int B, int d, int D, size_t p, mpode_dtype dt, int ybuf_rows_factor, bool own_kappa = true) {
    const size_t es = low_size(dt);
    lay.scal = lay.take(256);
    // one slab per family, stage slots back to back (the fused kernels address a slot through a 3-D tensor map)
    const size_t slot = (size_t)B * d * es;
    const size_t k0 = lay.take(4 * slot), y0 = lay.take(4 * ybuf_rows_factor * slot), p0 = lay.take(4 * slot);
    for (int j = 0; j < 4; ++j) {
        lay.kbuf[j] = k0 + j * slot;
        lay.ybuf[j] = y0 + j * ybuf_rows_factor * slot;
        lay.psi[j] = p0 + j * slot;
    }
    lay.v = lay.take((size_t)B * d * es);
    if (own_kappa) lay.kappa = lay.take((size_t)B * d * es);
    if (D > d) {
        for (int j = 0; j < 4; ++j) lay.klbuf[j] = lay.take((size_t)B * es);
        lay.vl = lay.take((size_t)B * es);
        lay.kappal = lay.take((size_t)B * es);
    }
    lay.dg = lay.take(p * sizeof(float));
}

// words 24 .. 55 of the scalar slice: the last-block counters of the one-launch column sums
unsigned* colsum_counters(void* ws, const Layout* lay) { return (unsigned*)((char*)ws + lay->scal) + 24; }

GemmArgs base_args(void* ws, const Layout* lay) {
    GemmArgs g{};
    g.split_k = 1;
    g.err = (unsigned*)((char*)ws + lay->scal) + 2;   // third word of the scalar slice
    return g;
}

// ---------------------------------------------------------------------------------------------------- MLP
class MlpVelocity : public Velocity {
public:
    MlpVelocity(const mpode_velocity_desc& v, int B, mpode_dtype dt, int max_steps) : B_(B), dt_(dt), act_(v.act),
        time_(v.append_time != 0), bias_(v.has_bias != 0), L_(v.n_layers), max_steps_(max_steps),
        w_(v.widths, v.widths + v.n_layers + 1) {
        size_t off = 0;
        for (int l = 0; l < L_; ++l) {
            int in_full = w_[l] + ((time_ && l == 0) ? 1 : 0);
            woff_.push_back(off);
            off += (size_t)w_[l + 1] * in_full;
            boff_.push_back(off);
            if (bias_) off += w_[l + 1];
        }
        p_ = off;
    }
    size_t param_count() const override { return p_; }

    bool supports_time_gradient() const override { return true; }

    void plan(Layout& lay) override {
        const size_t es = low_size(dt_);
        keep_k_ = lay.time_gradient;          // the time-grid gradient reads every k_j after the vector-Jacobian products
        fused_ok_ = fused_shape_ok();
        plan_common(lay, B_, w_[0], w_[0], p_, dt_, 1, !fused_ok_);
        if (fused_ok_) {     // kappa_j of three consecutive stages (slot j % 3); the layer-by-layer path uses the first slot
            kappaslab_ = lay.take((size_t)3 * B_ * w_[0] * es);
            lay.kappa = kappaslab_;
        }
        int maxw = 0;
        for (int l = 0; l < L_; ++l) {
            W16_.push_back(lay.take((size_t)w_[l + 1] * w_[l] * es));
            W16T_.push_back(lay.take((size_t)w_[l + 1] * w_[l] * es));
            b16_.push_back(bias_ ? lay.take((size_t)w_[l + 1] * es) : 0);
            maxw = w_[l + 1] > maxw ? w_[l + 1] : maxw;
        }
        wt16_ = time_ ? lay.take((size_t)w_[1] * es) : 0;
        hslab_.assign(L_, 0);
        for (int l = 1; l < L_; ++l) hslab_[l] = lay.take((size_t)4 * B_ * w_[l] * es);   // H_l of the four stages
        for (int j = 0; j < 4; ++j) {
            std::vector<size_t> hs(L_, 0);
            for (int l = 1; l < L_; ++l) hs[l] = hslab_[l] + (size_t)j * B_ * w_[l] * es;
            H_.push_back(hs);
        }
        // dZ_l: one buffer, or for the fused backward two stage slots (its weight gradients lag one stage behind the
        // input-gradient chain).  The second slot goes into the k_j slab where it fits: that slab is idle while the
        // vector-Jacobian products run.
        dzslab_.assign(L_ + 1, 0);
        dz_stride_.assign(L_ + 1, 0);
        dZ_.assign(L_, 0);
        size_t k_free = 4 * (size_t)B_ * w_[0] * es, k_at = lay.kbuf[0];
        for (int l = 1; l < L_; ++l) {
            const size_t slot = (size_t)B_ * w_[l] * es;
            if (fused_ok_ && slot <= k_free && !keep_k_) {
                dzslab_[l] = k_at;                              // slot 0 in the k slab (lower address), slot 1 its own buffer
                dZ_[l] = lay.take(slot);
                dz_stride_[l] = (long long)((dZ_[l] - k_at) / es);
                k_at += (slot + 255) & ~(size_t)255; k_free = k_free >= ((slot + 255) & ~(size_t)255) ? k_free - ((slot + 255) & ~(size_t)255) : 0;
            } else {
                dzslab_[l] = lay.take((fused_ok_ ? 2 : 1) * slot);
                dZ_[l] = dzslab_[l];
                dz_stride_[l] = (long long)B_ * w_[l];
            }
        }
        colsum_ = lay.take((size_t)64 * maxw * sizeof(float));
        tiny_ok_ = tiny_shape_ok();
        if (tiny_ok_) {
            tiny_scal_ = lay.take((size_t)max_steps_ * sizeof(RkStepScalars));
            tiny_log_ = lay.take(((size_t)4 * max_steps_ + 8) * sizeof(int));   // scale log, status words, t' [max_steps + 1]
        }
        size_t wg = 0;
        if (fused_ok_) {
            rb_ = (B_ + 127) / 128;
            plan_wgrad();
            // bias / time-column gradients are column sums of the cotangents: the weight-gradient machinery computes them as
            // dZ^T * 1 against a block of ones, into [stage][slice][width][8] partial sums (only column 0 is read back)
            size_t cp = 0;
            for (int j = 0; j < 4; ++j)
                for (int l = 1; l <= L_; ++l) { col_off_[j][l] = (long long)cp; cp += (size_t)wg_splits_ * w_[l] * kOnesKeep; }
            colpart_elems_ = cp;
            wg = (wg_part_elems_ + cp) * sizeof(float);      // the column-sum partials sit right behind the weight partials
            ones_ = lay.take((size_t)B_ * 64 * es);
            f_scalars_ = lay.take((size_t)max_steps_ * sizeof(RkStepScalars));
            for (int k = 0; k < 3; ++k) f_phases_[k] = lay.take((size_t)RK_MAX_PHASES * sizeof(RkPhase));
            cnt_stride_ = rb_ > wg_items_max_ ? rb_ : wg_items_max_;
            f_cnt_ = lay.take(((size_t)RK_MAX_PHASES * cnt_stride_ + 2) * sizeof(unsigned));
        } else if (dt_ != MPODE_F32) {      // slice partial sums of the tensor-core weight gradient
            for (int l = 0; l < L_; ++l) {
                size_t b = wgrad_tc_scratch_bytes(w_[l + 1], w_[l], B_);
                wg = b > wg ? b : wg;
            }
        }
        wgpart_ = lay.take(wg);
        wgpart_bytes_ = wg;
    }

    // Weight-gradient tiling of the fused backward: every layer's dW tiles (128 x bn) times a common number of batch
    // slices, chosen so that all layers together give about one work item per SM.
    void plan_wgrad() {
        long long tiles = 0;
        for (int l = 0; l < L_; ++l) {
            wg_bn_[l] = w_[l] >= 256 ? 256 : (w_[l] >= 128 ? 128 : 64);
            tiles += (long long)((w_[l + 1] + 127) / 128) * ((w_[l] + wg_bn_[l] - 1) / wg_bn_[l]);
        }
        const int kb_rows = (B_ + 63) / 64;
        int splits = (int)((sm_count() + tiles / 2) / tiles);
        if (splits > 16) splits = 16;
        if (splits > (kb_rows + 3) / 4) splits = (kb_rows + 3) / 4;
        if (splits < 1) splits = 1;
        wg_kb_per_split_ = (kb_rows + splits - 1) / splits;
        wg_splits_ = (kb_rows + wg_kb_per_split_ - 1) / wg_kb_per_split_;
        wg_part_elems_ = 0;
        wg_items_max_ = 0;
        for (int l = 0; l < L_; ++l) {
            wg_part_off_[l] = (long long)wg_part_elems_;
            wg_part_elems_ += (size_t)wg_splits_ * w_[l + 1] * w_[l];
            int items = ((w_[l + 1] + 127) / 128) * ((w_[l] + wg_bn_[l] - 1) / wg_bn_[l]) * wg_splits_;
            wg_items_max_ = items > wg_items_max_ ? items : wg_items_max_;
        }
    }

    void prepare(cudaStream_t st, void* ws, const float* theta, const signed char*, long long* L) override {
        for (int l = 0; l < L_; ++l) {
            int in_full = w_[l] + ((time_ && l == 0) ? 1 : 0);
            launch_quantize_matrix(dt_, theta + woff_[l], in_full, w_[l + 1], w_[l], at(ws, W16_[l]), at(ws, W16T_[l]), st, L);
            if (time_ && l == 0)
                launch_quantize_matrix(dt_, theta + woff_[l] + w_[l], in_full, w_[l + 1], 1, at(ws, wt16_), nullptr, st, L);
            if (bias_) launch_quantize_matrix(dt_, theta + boff_[l], w_[l + 1], 1, w_[l + 1], at(ws, b16_[l]), nullptr, st, L);
        }
    }

    void forward(cudaStream_t st, void* ws, int j, const void* yin, float tau16, long long* L) override {
        const void* X = yin;
        for (int l = 0; l < L_; ++l) {
            GemmArgs g = base_args(ws, lay_);
            g.A = X; g.a_rs = w_[l]; g.a_ks = 1;
            g.B = at(ws, W16_[l]); g.b_rs = w_[l]; g.b_ks = 1;
            g.M = B_; g.N = w_[l + 1]; g.K = w_[l];
            g.epi = EPI_FWD;
            g.out = (l == L_ - 1) ? at(ws, lay_->kbuf[j]) : at(ws, H_[j][l + 1]);
            g.ldo = w_[l + 1];
            g.bias = bias_ ? at(ws, b16_[l]) : nullptr;
            g.wt = (time_ && l == 0) ? at(ws, wt16_) : nullptr;
            g.tau = tau16;
            g.act = (l == L_ - 1) ? MPODE_ACT_NONE : act_;
            launch_contraction(dt_, g, st, L);
            X = g.out;
        }
    }

    void vjp(cudaStream_t st, void* ws, int j, const void* yin, float tau16, void* psi_out, float* dg, float beta,
             unsigned* flag, long long* L) override {
        const void* dZ = at(ws, lay_->kappa);
        for (int l = L_ - 1; l >= 0; --l) {
            const void* X = (l == 0) ? yin : at(ws, H_[j][l]);
            int in_full = w_[l] + ((time_ && l == 0) ? 1 : 0);
            {   // weight gradient: dW_l[n, k] (+)= sum_m dZ[m, n] X[m, k]
                GemmArgs g = base_args(ws, lay_);
                g.A = dZ; g.a_rs = 1; g.a_ks = w_[l + 1];
                g.B = X; g.b_rs = 1; g.b_ks = w_[l];
                g.M = w_[l + 1]; g.N = w_[l]; g.K = B_;
                g.epi = EPI_WGRAD; g.out = dg + woff_[l]; g.ldo = in_full; g.beta = beta;
                g.partial = wgrad_tc_scratch_bytes(g.M, g.N, g.K) <= wgpart_bytes_ ? (float*)at(ws, wgpart_) : nullptr;
                launch_contraction(dt_, g, st, L);
            }
            if (bias_ || (time_ && l == 0)) {
                const int R = launch_colsum(dt_, dZ, B_, w_[l + 1], (float*)at(ws, colsum_), bias_ ? dg + boff_[l] : nullptr, 1,
                                            (time_ && l == 0) ? dg + woff_[l] + w_[l] : nullptr, in_full, tau16, beta, st, L, colsum_counters(ws, lay_));
                if (lay_->time_gradient && time_ && l == 0) {      // d tau_j = w_t . colsum(dZ_1)
                    StageTimeArgs ta{};
                    ta.colsum = (const float*)at(ws, colsum_); ta.off[0] = 0; ta.terms = 1; ta.rows = R; ta.M = w_[1]; ta.stride = 1;
                    ta.wt = at(ws, wt16_); ta.dtau = (float*)at(ws, lay_->tdots) + 2 * kDotBlocks + j;
                    launch_stage_time_cot(dt_, ta, st, L);
                }
            }
            {   // input gradient: dX[m, k] = sum_n dZ[m, n] W_l[n, k], then the activation derivative of the layer below
                GemmArgs g = base_args(ws, lay_);
                g.A = dZ; g.a_rs = w_[l + 1]; g.a_ks = 1;
                g.B = at(ws, W16T_[l]); g.b_rs = w_[l + 1]; g.b_ks = 1;
                g.M = B_; g.N = w_[l]; g.K = w_[l + 1];
                g.epi = EPI_DGRAD; g.flag = flag;
                g.out = (l == 0) ? psi_out : at(ws, dZ_[l]);
                g.ldo = w_[l];
                g.hprev = (l == 0) ? nullptr : at(ws, H_[j][l]);
                g.ldh = w_[l];
                g.act = act_;
                launch_contraction(dt_, g, st, L);
                dZ = g.out;
            }
        }
    }


    // ---- whole-solve kernels for very small networks (any format)
    virtual bool tiny_shape_ok() const { return tiny_mlp_supported(B_, w_[0], L_ >= 2 ? w_[1] : 0, L_, (int)p_); }
    TinyParams tiny_params(void* ws, const FusedSolve& fs, const float* theta) const {
        TinyParams t{};
        t.B = B_; t.d = w_[0]; t.h = w_[1]; t.stages = fs.stages; t.n_steps = fs.n_steps;
        t.act = act_; t.time = time_ ? 1 : 0; t.bias = bias_ ? 1 : 0;
        t.theta = theta; t.scal = (const RkStepScalars*)at(ws, tiny_scal_); t.traj = const_cast<void*>(fs.traj);
        t.round_increment = fs.round_increment;
        return t;
    }
    bool whole_forward(cudaStream_t st, void* ws, const FusedSolve& fs, const float* theta, const float* y0, float* yT,
                       long long* L) override {
        if (!tiny_ok_ || fs.stages > RK_MAX_STAGES || fs.n_steps > max_steps_) return false;
        cudaMemcpyAsync(at(ws, tiny_scal_), fs.scalars.data(), (size_t)fs.n_steps * sizeof(RkStepScalars), cudaMemcpyHostToDevice, st);
        TinyParams t = tiny_params(ws, fs, theta);
        t.y0 = y0; t.yT = yT;
        launch_tiny_forward(dt_, t, st, L);
        if (tl_counters) ++tl_counters->whole;
        return true;
    }
    bool whole_backward(cudaStream_t st, void* ws, const FusedSolve& fs, WholeBackward& wb, long long* L) override {
        if (!tiny_ok_ || fs.stages > RK_MAX_STAGES || fs.n_steps > max_steps_) return false;
        const int N = fs.n_steps;
        cudaMemcpyAsync(at(ws, tiny_scal_), fs.scalars.data(), (size_t)N * sizeof(RkStepScalars), cudaMemcpyHostToDevice, st);
        int* logs = (int*)at(ws, tiny_log_);
        cudaMemsetAsync(logs, 0, ((size_t)4 * max_steps_ + 8) * sizeof(int), st);
        TinyParams t = tiny_params(ws, fs, wb.theta);
        t.dLdyT = wb.dLdyT; t.a = wb.a; t.g = wb.g; t.accumulate = wb.accumulate;
        t.scaling = wb.scaling; t.k_max = wb.k_max; t.growth_rule = wb.growth_rule; t.pbits = wb.pbits;
        t.e0 = wb.e0; t.e0_from_norm = wb.e0_from_norm;
        t.log_exp = logs; t.log_attempts = logs + max_steps_; t.log_doubled = logs + 2 * max_steps_; t.status = logs + 3 * max_steps_;
        t.cot = wb.cot;
        t.tprime = wb.dt_host != nullptr ? (float*)(logs + 3 * max_steps_ + 4) : nullptr;
        launch_tiny_backward(dt_, t, st, L);
        if (tl_counters) ++tl_counters->whole;
        std::vector<int> h((size_t)3 * max_steps_ + 4);
        cudaMemcpyAsync(h.data(), logs, h.size() * sizeof(int), cudaMemcpyDeviceToHost, st);
        if (wb.dt_host != nullptr) cudaMemcpyAsync(wb.dt_host, t.tprime, (size_t)(N + 1) * sizeof(float), cudaMemcpyDeviceToHost, st);
        cudaStreamSynchronize(st);
        const int* stp = h.data() + 3 * max_steps_;
        wb.status = stp[0]; wb.first_failed_step = wb.status == MPODE_ERR_SCALE_FAILED ? stp[1] : -1; wb.retries = stp[2];
        for (int i = 0; i < N; ++i) {
            if (wb.exp_used) wb.exp_used[i] = h[i];
            if (wb.attempts) wb.attempts[i] = h[max_steps_ + i];
            if (wb.doubled) wb.doubled[i] = (unsigned char)h[2 * max_steps_ + i];
        }
        return true;
    }

    // ---- fused Runge-Kutta path (16-bit formats, every width a multiple of 8)
    virtual bool fused_shape_ok() const {
        if (dt_ != MPODE_BF16 && dt_ != MPODE_F16) return false;
        if (L_ > 4) return false;
        for (int w : w_) if (w % 8 != 0) return false;
        return true;
    }
    // output-tile width of a contraction with N columns: wide tiles for the tensor pipe, narrower ones when that
    // wastes fewer padded columns or when wide tiles would leave SMs without work
    int choose_bn(int N) const {
        int bn = 64;
        long long best_pad = -1;
        for (int c : {256, 128, 64}) {
            long long pad = (long long)((N + c - 1) / c) * c;
            if (best_pad < 0 || pad < best_pad) { best_pad = pad; bn = c; }
        }
        auto tiles = [&](int c) { return (long long)rb_ * ((N + c - 1) / c); };
        if (bn == 256 && tiles(256) < sm_count()) bn = 128;
        if (bn == 128 && tiles(128) < sm_count() / 2) bn = 64;
        return bn;
    }

    bool fused_forward(cudaStream_t st, void* ws, const FusedSolve& fs, long long* L) override {
        if (!fused_ok_ || fs.stages > RK_MAX_STAGES || fs.n_steps > max_steps_) return false;
        if (((uintptr_t)fs.traj & 31) != 0) return false;       // the epilogues move 32-byte pieces of trajectory rows
        const int s = fs.stages, d = w_[0];
        if (s * L_ > RK_MAX_PHASES) return false;
        RkMaps maps;
        int nm = 0;
        const int m_traj = nm++, m_y = nm++;
        if (!get_tensor_map_3d(fs.traj, fs.n_steps + 1, B_, d, (long long)B_ * d, d, 128, dt_, &maps.m[m_traj])) return false;
        if (!get_tensor_map_3d(at(ws, lay_->ybuf[0]), 4, B_, d, (long long)B_ * d, d, 128, dt_, &maps.m[m_y])) return false;
        int m_h[8] = {0}, m_w[8] = {0}, bn[8] = {0};
        for (int l = 1; l < L_; ++l) {
            m_h[l] = nm++;
            if (!get_tensor_map_3d(at(ws, hslab_[l]), 4, B_, w_[l], (long long)B_ * w_[l], w_[l], 128, dt_, &maps.m[m_h[l]])) return false;
        }
        for (int l = 0; l < L_; ++l) {
            bn[l] = choose_bn(w_[l + 1]);
            m_w[l] = nm++;
            if (!get_tensor_map(at(ws, W16_[l]), w_[l + 1], w_[l], w_[l], bn[l], dt_, &maps.m[m_w[l]])) return false;
        }
        std::vector<RkPhase> ph;
        for (int j = 0; j < s; ++j)
            for (int l = 0; l < L_; ++l) {
                RkPhase q{};
                q.a_map = l == 0 ? (j == 0 ? m_traj : m_y) : m_h[l];
                q.a_slot = (l == 0 && j > 0) ? j : 0;          // hidden outputs are consumed at once: one slot serves all stages
                q.a_slot_step = (l == 0 && j == 0) ? 1 : 0;
                q.b_map = m_w[l];
                q.N = w_[l + 1]; q.K = w_[l]; q.bn = bn[l]; q.tiles_n = (q.N + q.bn - 1) / q.bn;
                q.epi = l == L_ - 1 ? RK_EPI_STAGE_OUT : RK_EPI_HIDDEN;
                q.act = act_; q.stage = j; q.layer = l; q.out_slot = 0;
                q.dep_phase = ph.empty() ? s * L_ - 1 : (int)ph.size() - 1;      // the chain is linear: previous phase,
                q.dep_prev_iter = ph.empty() ? 1 : 0;                             // wrapping to the last one of the step before
                ph.push_back(q);
            }
        if (fs.starve && ph.size() > 1) ph[1].dep_extra = 1;
        RkParams p{};
        fill_common_params(p, ws, fs, (int)ph.size());
        p.n_steps = fs.n_steps; p.step0 = 0; p.step_dir = 1;
        p.y = fs.y;
        p.flag = nullptr;
        p.phases = (const RkPhase*)at(ws, f_phases_[0]);
        cudaMemcpyAsync(at(ws, f_phases_[0]), ph.data(), ph.size() * sizeof(RkPhase), cudaMemcpyHostToDevice, st);
        cudaMemcpyAsync(at(ws, f_scalars_), fs.scalars.data(), (size_t)fs.n_steps * sizeof(RkStepScalars), cudaMemcpyHostToDevice, st);
        cudaMemsetAsync(at(ws, f_cnt_), 0, ((size_t)ph.size() * cnt_stride_ + 2) * sizeof(unsigned), st);
        return timed_launch(0, (double)fs.n_steps * s * layer_flops(), maps, p, st, L);
    }

    double layer_flops() const {     // one evaluation of the velocity over the batch
        double f = 0;
        for (int l = 0; l < L_; ++l) f += 2.0 * B_ * (double)w_[l] * w_[l + 1];
        return f;
    }
    bool timed_launch(int klass, double flops, const RkMaps& maps, const RkParams& p, cudaStream_t st, long long* L) {
        Profiler* pr = tl_profiler;
        if (pr && pr->enabled) pr->begin(klass, flops, st);
        bool ok = launch_rk_fused(dt_, klass == 3, maps, p, st, L);
        if (pr && pr->enabled) pr->end(st);
        return ok;
    }

    // ---- fused backward: per step one launch that recomputes the stages (keeping every layer output) and one launch
    // per attempt for the vector-Jacobian products and weight gradients.  begin() builds both phase tables.
    bool fused_backward_begin(cudaStream_t st, void* ws, const FusedSolve& fs, long long* L) override {
        (void)L;
        if (!fused_ok_ || fs.stages > RK_MAX_STAGES || fs.n_steps > max_steps_) return false;
        if (((uintptr_t)fs.traj & 31) != 0) return false;
        const int s = fs.stages, d = w_[0];
        b_stages_ = s;
        // ---------------- recompute program: stage inputs live in the Y slab (slot 0 = copy of the stored state)
        {
            int nm = 0;
            const int m_y = nm++;
            if (!get_tensor_map_3d(at(ws, lay_->ybuf[0]), 4, B_, d, (long long)B_ * d, d, 128, dt_, &maps_r_.m[m_y])) return false;
            int m_h[8] = {0}, m_w[8] = {0}, bn[8] = {0};
            for (int l = 1; l < L_; ++l) {
                m_h[l] = nm++;
                if (!get_tensor_map_3d(at(ws, hslab_[l]), 4, B_, w_[l], (long long)B_ * w_[l], w_[l], 128, dt_, &maps_r_.m[m_h[l]])) return false;
            }
            for (int l = 0; l < L_; ++l) {
                bn[l] = choose_bn(w_[l + 1]);
                m_w[l] = nm++;
                if (!get_tensor_map(at(ws, W16_[l]), w_[l + 1], w_[l], w_[l], bn[l], dt_, &maps_r_.m[m_w[l]])) return false;
            }
            std::vector<RkPhase> ph;
            for (int j = 0; j < s; ++j)
                for (int l = 0; l < L_; ++l) {
                    if (j == s - 1 && l == L_ - 1 && !keep_k_) continue;   // k_s is not needed to differentiate the step
                    RkPhase q{};
                    q.a_map = l == 0 ? m_y : m_h[l];
                    q.a_slot = j; q.a_slot_step = 0;
                    q.b_map = m_w[l];
                    q.N = w_[l + 1]; q.K = w_[l]; q.bn = bn[l]; q.tiles_n = (q.N + q.bn - 1) / q.bn;
                    q.epi = l == L_ - 1 ? RK_EPI_STAGE_OUT : RK_EPI_HIDDEN;
                    q.act = act_; q.stage = j; q.layer = l; q.out_slot = j;
                    q.dep_phase = (int)ph.size() - 1;
                    ph.push_back(q);
                }
            n_phases_r_ = (int)ph.size();
            if (n_phases_r_ > RK_MAX_PHASES) return false;
            if (n_phases_r_ > 0)
                cudaMemcpyAsync(at(ws, f_phases_[1]), ph.data(), ph.size() * sizeof(RkPhase), cudaMemcpyHostToDevice, st);
        }
        // ---------------- VJP program: stages in reverse; the weight gradients of a stage follow the input-gradient
        // chain of the stage below it, so that their operands (whole batch slices) are complete when they start
        {
            int nm = 0;
            const int m_kap = nm++;
            if (!get_tensor_map_3d(at(ws, kappaslab_), 3, B_, d, (long long)B_ * d, d, 128, dt_, &maps_v_.m[m_kap])) return false;
            int m_dz[8] = {0}, m_wt[8] = {0}, m_hs[8] = {0}, bn[8] = {0};
            for (int l = 1; l < L_; ++l) {
                m_dz[l] = nm++;
                if (!get_tensor_map_3d(at(ws, dzslab_[l]), 2, B_, w_[l], dz_stride_[l], w_[l], 128, dt_, &maps_v_.m[m_dz[l]])) return false;
                m_hs[l] = nm++;     // stored layer outputs H_l (4 stage slots), staged into shared memory for the derivative product
                if (!get_tensor_map_3d(at(ws, hslab_[l]), 4, B_, w_[l], (long long)B_ * w_[l], w_[l], 128, dt_, &maps_v_.m[m_hs[l]])) return false;
            }
            for (int l = 0; l < L_; ++l) {       // input gradient of layer l: N = w_l, K = w_{l+1}, operand W_l^T [w_l][w_{l+1}]
                bn[l] = choose_bn(w_[l]);
                m_wt[l] = nm++;
                if (!get_tensor_map(at(ws, W16T_[l]), w_[l], w_[l + 1], w_[l + 1], bn[l], dt_, &maps_v_.m[m_wt[l]])) return false;
            }
            // weight-gradient operands, read with the batch as the reduction index: boxes of [64 rows][64 columns]
            int m_ga[8] = {0}, m_gb[8] = {0};
            for (int l = 0; l < L_; ++l) {
                m_ga[l] = nm++;     // dZ_{l+1} (2 slots), kappa for the last layer (3 slots)
                const bool last = l == L_ - 1;
                const void* a_ptr = last ? at(ws, kappaslab_) : at(ws, dzslab_[l + 1]);
                if (!get_tensor_map_3d(a_ptr, last ? 3 : 2, B_, w_[l + 1], last ? (long long)B_ * d : dz_stride_[l + 1], w_[l + 1], 64, dt_,
                                       &maps_v_.m[m_ga[l]])) return false;
                m_gb[l] = nm++;     // layer input: Y slab for the first layer, H_l otherwise, 4 slots
                const void* b_ptr = l == 0 ? at(ws, lay_->ybuf[0]) : at(ws, hslab_[l]);
                if (!get_tensor_map_3d(b_ptr, 4, B_, w_[l], (long long)B_ * w_[l], w_[l], 64, dt_, &maps_v_.m[m_gb[l]])) return false;
            }
            const int m_ones = nm++;
            if (!get_tensor_map_3d(at(ws, ones_), 1, B_, 64, (long long)B_ * 64, 64, 64, dt_, &maps_v_.m[m_ones])) return false;
            launch_fill_low(dt_, at(ws, ones_), 1.f, (long long)B_ * 64, st, L);
            if (nm > RK_MAX_MAPS) return false;
            std::vector<RkPhase> ph;
            int chain_prev = -1, sync_tiles = 0;
            int wg_prev[8];
            for (int l = 0; l < 8; ++l) wg_prev[l] = -1;
            int tiles_through_stage[RK_MAX_STAGES] = {0}, wg_items_through_stage[RK_MAX_STAGES] = {0}, wg_items = 0;
            auto push_wgrad = [&](int j) {
                for (int l = 0; l < L_; ++l) {
                    RkPhase q{};
                    q.epi = RK_EPI_WGRAD;
                    q.a_map = m_ga[l]; q.a_slot = l == L_ - 1 ? j % 3 : (j & 1);
                    q.b_map = m_gb[l]; q.b_slot = j;
                    q.M = w_[l + 1]; q.N = w_[l]; q.K = B_; q.bn = wg_bn_[l];
                    q.tiles_m = (q.M + 127) / 128; q.tiles_n = (q.N + q.bn - 1) / q.bn;
                    q.splits = wg_splits_; q.kb_per_split = wg_kb_per_split_;
                    q.part_off = wg_part_off_[l];
                    q.accumulate = j == s - 1 ? 0 : 1;
                    q.dep_phase = wg_prev[l]; q.dep_mode = 1;
                    q.wait_total = tiles_through_stage[j];
                    q.layer = l; q.stage = j;
                    q.queue = j == 0 ? 2 : 1;          // the last stage's items have nothing left to overlap with: all CTAs
                    wg_prev[l] = (int)ph.size();
                    wg_items += q.tiles_m * q.tiles_n * q.splits;
                    ph.push_back(q);
                    if (bias_ || (time_ && l == 0)) {
                        // column sums of the same cotangent (bias and time-column gradients of layer l): one 64-wide tile per
                        // 128 output rows against the block of ones, kept per stage (the time column weighs each stage by its tau)
                        RkPhase b = q;
                        b.b_map = m_ones; b.b_slot = 0;
                        b.N = kOnesKeep; b.bn = 64; b.tiles_n = 1;
                        b.part_off = (long long)(wg_part_elems_) + col_off_[j][l + 1];
                        b.accumulate = 0; b.dep_phase = -1; b.pack2 = 1;
                        wg_items += b.tiles_m * b.splits;
                        ph.push_back(b);
                    }
                }
                wg_items_through_stage[j] = wg_items;
            };
            for (int j = s - 1; j >= 0; --j) {
                for (int l = L_ - 1; l >= 0; --l) {
                    RkPhase q{};
                    q.a_map = l == L_ - 1 ? m_kap : m_dz[l + 1];
                    q.a_slot = l == L_ - 1 ? j % 3 : (j & 1); q.a_slot_step = 0;
                    // this stage overwrites the dZ slots of stage j + 2 (and, after psi_j, the kappa slot of stage j + 2):
                    // their last readers are that stage's weight-gradient items
                    if (j + 2 <= s - 1) q.wait_wg_total = wg_items_through_stage[j + 2];
                    q.b_map = m_wt[l];
                    q.N = w_[l]; q.K = w_[l + 1]; q.bn = bn[l]; q.tiles_n = (q.N + q.bn - 1) / q.bn;
                    q.epi = l == 0 ? RK_EPI_PSI : RK_EPI_DGRAD;
                    q.act = act_; q.stage = j; q.layer = l; q.out_slot = j & 1; q.h_slot = j; q.h_map = l >= 1 ? m_hs[l] : 0;
                    q.queue = j == s - 1 ? 2 : 0;      // no weight-gradient work exists yet during the first stage's chain
                    q.dep_phase = chain_prev;
                    chain_prev = (int)ph.size();
                    sync_tiles += rb_ * q.tiles_n;
                    ph.push_back(q);
                }
                tiles_through_stage[j] = sync_tiles;
                if (j < s - 1) push_wgrad(j + 1);
            }
            push_wgrad(0);
            n_phases_v_ = (int)ph.size();
            sync_tiles_v_ = sync_tiles;
            wg_items_v_ = wg_items;
            if (n_phases_v_ > RK_MAX_PHASES) return false;
            cudaMemcpyAsync(at(ws, f_phases_[2]), ph.data(), ph.size() * sizeof(RkPhase), cudaMemcpyHostToDevice, st);
        }
        scal_host_ = fs.scalars;
        cudaMemcpyAsync(at(ws, f_scalars_), fs.scalars.data(), (size_t)fs.n_steps * sizeof(RkStepScalars), cudaMemcpyHostToDevice, st);
        return true;
    }

    void fused_recompute(cudaStream_t st, void* ws, const FusedSolve& fs, int step, long long* L) override {
        const size_t es = low_size(dt_);
        const size_t slot = (size_t)B_ * w_[0] * es;
        cudaMemcpyAsync(at(ws, lay_->ybuf[0]), (const char*)fs.traj + (size_t)step * slot, slot, cudaMemcpyDeviceToDevice, st);
        if (n_phases_r_ == 0) return;
        RkParams p{};
        fill_common_params(p, ws, fs, n_phases_r_);
        p.phases = (const RkPhase*)at(ws, f_phases_[1]);
        p.n_steps = 1; p.step0 = step; p.step_dir = 1;
        p.y = nullptr; p.flag = nullptr;
        cudaMemsetAsync(at(ws, f_cnt_), 0, ((size_t)n_phases_r_ * cnt_stride_ + 2) * sizeof(unsigned), st);
        timed_launch(0, b_stages_ * layer_flops() - (keep_k_ ? 0.0 : 2.0 * B_ * (double)w_[L_ - 1] * w_[L_]), maps_r_, p, st, L);
    }

    // CTAs given to the latency-bound input-gradient chains while the others run weight-gradient items
    int chain_ctas() const {
        return b_stages_ > 1 ? (sm_count() * 19) / 37 : 0;   // measured best on B200 for the MLP block (76 of 148)
    }

    void* fused_kappa_last(void* ws) const override {
        return at(ws, kappaslab_) + (size_t)((b_stages_ - 1) % 3) * B_ * w_[0] * low_size(dt_);
    }

    void fused_vjp(cudaStream_t st, void* ws, const FusedSolve& fs, int step, float* out, float beta, float coef, unsigned* flag,
                   long long* L, cudaEvent_t after_kernel, cudaStream_t st_finish) override {
        const int s = b_stages_, d = w_[0];
        const RkStepScalars& sc = scal_host_[step];
        RkParams p{};
        fill_common_params(p, ws, fs, n_phases_v_);
        p.phases = (const RkPhase*)at(ws, f_phases_[2]);
        p.n_steps = 1; p.step0 = step; p.step_dir = 1;
        p.sync_tiles_per_step = sync_tiles_v_;
        p.wg_items_per_step = wg_items_v_;
        p.chain_ctas = chain_ctas();
        p.flag = flag;
        p.v = at(ws, lay_->v);
        p.kappaslab = at(ws, kappaslab_);
        for (int l = 1; l < L_; ++l) { p.dzslab[l] = at(ws, dzslab_[l]); p.dz_slot_stride[l] = dz_stride_[l]; }
        p.partial = (float*)at(ws, wgpart_);
        cudaMemsetAsync(at(ws, f_cnt_), 0, ((size_t)n_phases_v_ * cnt_stride_ + 2) * sizeof(unsigned), st);
        timed_launch(3, 2.0 * s * layer_flops(), maps_v_, p, st, L);
        if (after_kernel != nullptr) cudaEventRecord(after_kernel, st);
        if (st_finish != nullptr && after_kernel != nullptr) {
            cudaStreamWaitEvent(st_finish, after_kernel, 0);
            st = st_finish;
        }
        if (lay_->time_gradient && time_) {      // d tau_j = w_t . colsum_j(dZ_1), from the stored ones-products of the first layer
            StageTimeArgs ta{};
            ta.colsum = (const float*)at(ws, wgpart_) + wg_part_elems_;
            for (int j = 0; j < s; ++j) ta.off[j] = col_off_[j][1];
            ta.terms = s; ta.rows = wg_splits_; ta.M = w_[1]; ta.stride = kOnesKeep;
            ta.wt = at(ws, wt16_); ta.dtau = (float*)at(ws, lay_->tdots) + 2 * kDotBlocks;
            launch_stage_time_cot(dt_, ta, st, L);
        }
        // slices of the batch and row blocks summed in a fixed order, all layers in one launch
        GradFinishArgs ga{};
        ga.n_layers = L_; ga.out = out; ga.beta = beta; ga.coef = coef;
        for (int l = 0; l < L_; ++l) {
            GradFinishLayer& g = ga.layer[l];
            const int in_full = w_[l] + ((time_ && l == 0) ? 1 : 0);
            g.partial = (const float*)at(ws, wgpart_) + wg_part_off_[l];
            g.splits = wg_splits_; g.M = w_[l + 1]; g.N = w_[l];
            g.w_off = (long long)woff_[l]; g.ldo = in_full;
            g.colpart = (const float*)at(ws, wgpart_) + wg_part_elems_;
            g.terms = s; g.rows = wg_splits_;
            for (int j = 0; j < s; ++j) { g.col_off[j] = col_off_[j][l + 1]; g.tau[j] = sc.tau16[j]; }
            g.bias_off = bias_ ? (long long)boff_[l] : -1;
            g.time_off = (time_ && l == 0) ? (long long)(woff_[0] + w_[0]) : -1;
        }
        launch_grad_finish(ga, st, L);
    }

    void fill_common_params(RkParams& p, void* ws, const FusedSolve& fs, int n_phases) const {
        p.B = B_; p.rb = rb_; p.d = w_[0]; p.D = w_[0]; p.stages = fs.stages;
        p.n_phases = n_phases;
        p.round_increment = fs.round_increment;
        p.scalars = (const RkStepScalars*)at(ws, f_scalars_);
        p.cnt = (unsigned*)at(ws, f_cnt_);
        p.cnt_stride = cnt_stride_;
        p.err = (unsigned*)at(ws, lay_->scal) + 2;
        p.wait_ns = fs.wait_ns;
        for (int l = 0; l < L_; ++l) p.bias[l] = bias_ ? at(ws, b16_[l]) : nullptr;
        p.wt = time_ ? at(ws, wt16_) : nullptr;
        for (int l = 0; l <= L_; ++l) p.w[l] = w_[l];
        for (int l = 1; l < L_; ++l) { p.hslab[l] = at(ws, hslab_[l]); p.h_slot_stride[l] = (long long)B_ * w_[l]; }
        p.kslab = at(ws, lay_->kbuf[0]); p.yslab = at(ws, lay_->ybuf[0]); p.psislab = at(ws, lay_->psi[0]);
        p.traj = const_cast<void*>(fs.traj);
    }

    void bind(const Layout* lay) { lay_ = lay; }

protected:
    int B_;
    mpode_dtype dt_;
    int act_;
    bool time_, bias_;
    int L_;
    int max_steps_;
    std::vector<int> w_;
    std::vector<size_t> woff_, boff_, W16_, W16T_, b16_, dZ_;
    std::vector<std::vector<size_t>> H_;
    std::vector<size_t> hslab_, dzslab_;
    std::vector<long long> dz_stride_;
    size_t wt16_ = 0, colsum_ = 0, wgpart_ = 0, wgpart_bytes_ = 0, p_ = 0;
    size_t f_scalars_ = 0, f_phases_[3] = {0, 0, 0}, f_cnt_ = 0, kappaslab_ = 0;
    size_t tiny_scal_ = 0, tiny_log_ = 0;
    bool tiny_ok_ = false;
    bool fused_ok_ = false;
    bool keep_k_ = false;
    int rb_ = 0, cnt_stride_ = 0;
    int wg_bn_[8] = {0}, wg_splits_ = 1, wg_kb_per_split_ = 1, wg_items_max_ = 0;
    long long wg_part_off_[8] = {0};
    size_t wg_part_elems_ = 0;
    int n_phases_v_ = 0, n_phases_r_ = 0, sync_tiles_v_ = 0, wg_items_v_ = 0;
    static constexpr int kOnesKeep = 8;   // columns of the ones-product that are stored (one 32-byte piece per row)
    long long col_off_[4][9] = {{0}};
    size_t colpart_elems_ = 0, ones_ = 0;
    RkMaps maps_r_, maps_v_;
    std::vector<RkStepScalars> scal_host_;
    int b_stages_ = 0;
    const Layout* lay_ = nullptr;
};

// ---------------------------------------------------------------------------------------------------- CNF
// Primal rows and tangent rows share every weight, so each layer runs as one contraction over 2B rows:
// rows [0, B) carry the state, rows [B, 2B) the forward-mode tangent started at the probe (Sec. 6.1).
class CnfVelocity : public MlpVelocity {
public:
    CnfVelocity(const mpode_velocity_desc& v, int B, mpode_dtype dt, int max_steps) : MlpVelocity(v, B, dt, max_steps) {}
    bool fused_shape_ok() const override { return false; }
    bool tiny_shape_ok() const override { return false; }
    bool supports_time_gradient() const override { return false; }

    void plan(Layout& lay) override {
        const size_t es = low_size(dt_);
        const int d = w_[0];
        plan_common(lay, B_, d, d + 1, p_, dt_, 2);
        int maxw = 0;
        for (int l = 0; l < L_; ++l) {
            W16_.push_back(lay.take((size_t)w_[l + 1] * w_[l] * es));
            W16T_.push_back(lay.take((size_t)w_[l + 1] * w_[l] * es));
            b16_.push_back(bias_ ? lay.take((size_t)w_[l + 1] * es) : 0);
            maxw = w_[l + 1] > maxw ? w_[l + 1] : maxw;
        }
        wt16_ = time_ ? lay.take((size_t)w_[1] * es) : 0;
        for (int j = 0; j < 4; ++j) {
            std::vector<size_t> hg(L_, 0), u(L_, 0);
            for (int l = 1; l < L_; ++l) {
                hg[l] = lay.take((size_t)2 * B_ * w_[l] * es);   // [H_l; G_l]
                u[l] = lay.take((size_t)B_ * w_[l] * es);        // U_l
            }
            H_.push_back(hg);
            U_.push_back(u);
        }
        uL_ = lay.take((size_t)B_ * d * es);
        cot_.assign(L_ + 1, 0);
        for (int l = 1; l <= L_; ++l) cot_[l] = lay.take((size_t)2 * B_ * w_[l] * es);   // [zeta_l; ubar_l]
        // fp32 [hbar; gbar] of the backward step through an activation: not needed where the tensor-core epilogue takes that
        // step (tiles of sample pairs; every such contraction is eligible when the widths are multiples of 8 and at least 64)
        pair_bwd_ = pair_tiles();
        for (int l = 1; l <= L_; ++l) pair_bwd_ = pair_bwd_ && w_[l] >= 64 && w_[l] % 8 == 0;
        wide_ = pair_bwd_ ? 0 : lay.take((size_t)2 * B_ * maxw * sizeof(float));
        colsum_ = lay.take((size_t)64 * maxw * sizeof(float));
        size_t wg = 0;
        for (int l = 0; l < L_; ++l) {
            size_t b = wgrad_tc_scratch_bytes(w_[l + 1], w_[l], 2 * B_);
            wg = b > wg ? b : wg;
        }
        wgpart_ = lay.take(wg);
    }

    bool needs_input_copy() const override { return true; }
    size_t kappa_offset(const Layout&) const override { return cot_[L_]; }

    void prepare(cudaStream_t st, void* ws, const float* theta, const signed char* probe, long long* L) override {
        MlpVelocity::prepare(st, ws, theta, probe, L);
        probe_ = probe;
        const size_t es = low_size(dt_);
        const long long n = (long long)B_ * w_[0];
        for (int j = 0; j < 4; ++j) launch_cnf_probe_to_low(dt_, probe, at(ws, lay_->ybuf[j]) + n * es, n, st, L);
    }

    void forward(cudaStream_t st, void* ws, int j, const void* yin, float tau16, long long* L) override {
        const size_t es = low_size(dt_);
        const void* X = yin;   // [Y_j; eps], 2B rows
        for (int l = 0; l < L_; ++l) {
            bool last = (l == L_ - 1);
            GemmArgs g = base_args(ws, lay_);
            g.A = X; g.a_rs = w_[l]; g.a_ks = 1;
            g.B = at(ws, W16_[l]); g.b_rs = w_[l]; g.b_ks = 1;
            g.M = 2 * B_; g.N = w_[l + 1]; g.K = w_[l];
            g.epi = EPI_FWD;
            g.out = last ? at(ws, lay_->kbuf[j]) : at(ws, H_[j][l + 1]);
            g.out2 = last ? at(ws, uL_) : at(ws, U_[j][l + 1]);
            g.m_split = B_;
            g.ldo = w_[l + 1];
            g.bias = bias_ ? at(ws, b16_[l]) : nullptr;
            g.wt = (time_ && l == 0) ? at(ws, wt16_) : nullptr;
            g.tau = tau16;
            g.act = last ? MPODE_ACT_NONE : act_;
            // tensor-core kernel: tiles of sample pairs, whose epilogue also writes G_l = Q16(sigma'(H_l) * U_l)
            const long long n = (long long)B_ * w_[l + 1];
            g.cnf_pair = pair_tiles() ? 1 : 0;
            g.pair_out = (g.cnf_pair && !last) ? at(ws, H_[j][l + 1]) + n * es : nullptr;
            const int path = launch_contraction(dt_, g, st, L);
            if (!last) {
                if (!(path == 1 && g.cnf_pair))
                    launch_cnf_tangent_act(dt_, act_, at(ws, H_[j][l + 1]), at(ws, U_[j][l + 1]), at(ws, H_[j][l + 1]) + n * es, n, st, L);
                X = at(ws, H_[j][l + 1]);
            }
        }
        launch_cnf_trace(dt_, probe_, at(ws, uL_), at(ws, lay_->klbuf[j]), B_, w_[0], st, L);
    }

    void vjp(cudaStream_t st, void* ws, int j, const void* yin, float tau16, void* psi_out, float* dg, float beta,
             unsigned* flag, long long* L) override {
        const size_t es = low_size(dt_);
        const int d = w_[0];
        // cot_[L] = [kappa_z; ubar_L]: the driver wrote kappa_z into the first half
        launch_cnf_ubar_last(dt_, at(ws, lay_->kappal), probe_, at(ws, cot_[L_]) + (size_t)B_ * d * es, B_, d, flag, st, L);
        const void* C = at(ws, cot_[L_]);
        for (int l = L_ - 1; l >= 0; --l) {
            const void* Xpair = (l == 0) ? yin : at(ws, H_[j][l]);
            int in_full = w_[l] + ((time_ && l == 0) ? 1 : 0);
            {   // dW_l = zeta^T X + ubar^T G: one contraction over the 2B stacked rows
                GemmArgs g = base_args(ws, lay_);
                g.A = C; g.a_rs = 1; g.a_ks = w_[l + 1];
                g.B = Xpair; g.b_rs = 1; g.b_ks = w_[l];
                g.M = w_[l + 1]; g.N = w_[l]; g.K = 2 * B_;
                g.epi = EPI_WGRAD; g.out = dg + woff_[l]; g.ldo = in_full; g.beta = beta;
                g.partial = (float*)at(ws, wgpart_);
                launch_contraction(dt_, g, st, L);
            }
            if (bias_ || (time_ && l == 0))   // bias and time column see the primal rows only
                launch_colsum(dt_, C, B_, w_[l + 1], (float*)at(ws, colsum_), bias_ ? dg + boff_[l] : nullptr, 1,
                              (time_ && l == 0) ? dg + woff_[l] + w_[l] : nullptr, in_full, tau16, beta, st, L, colsum_counters(ws, lay_));
            if (l > 0) {
                const long long n = (long long)B_ * w_[l];
                GemmArgs g = base_args(ws, lay_);
                g.A = C; g.a_rs = w_[l + 1]; g.a_ks = 1;
                g.B = at(ws, W16T_[l]); g.b_rs = w_[l + 1]; g.b_ks = 1;
                g.M = 2 * B_; g.N = w_[l]; g.K = w_[l + 1];
                bool done = false;
                if (pair_tiles()) {      // [hbar; gbar] through the activation in the epilogue of the tensor-core kernel
                    GemmArgs f = g;
                    f.epi = EPI_DGRAD; f.cnf_pair = 2; f.m_split = B_; f.act = act_; f.flag = flag;
                    f.hprev = at(ws, H_[j][l]); f.ldh = w_[l]; f.uprev = at(ws, U_[j][l]);
                    f.out = at(ws, cot_[l]); f.out2 = at(ws, cot_[l]) + n * es; f.ldo = w_[l];
                    done = tc_eligible(dt_, f) && launch_contraction(dt_, f, st, L) == 1;
                }
                if (!done && pair_bwd_) {
                    // no scratch was planned for the two-kernel form: report through the error word that the driver reads back
                    cudaMemsetAsync(g.err, 0xff, sizeof(unsigned), st);
                } else if (!done) {
                    g.epi = EPI_RAW32; g.out = at(ws, wide_); g.ldo = w_[l];
                    launch_contraction(dt_, g, st, L);
                    float* wide = (float*)at(ws, wide_);
                    launch_cnf_backprop_act(dt_, act_, at(ws, H_[j][l]), at(ws, U_[j][l]), wide, wide + n, at(ws, cot_[l]),
                                            at(ws, cot_[l]) + n * es, n, flag, st, L);
                }
                C = at(ws, cot_[l]);
            } else {
                GemmArgs g = base_args(ws, lay_);
                g.A = C; g.a_rs = w_[1]; g.a_ks = 1;
                g.B = at(ws, W16T_[0]); g.b_rs = w_[1]; g.b_ks = 1;
                g.M = B_; g.N = w_[0]; g.K = w_[1];
                g.epi = EPI_DGRAD; g.flag = flag; g.out = psi_out; g.ldo = w_[0];
                launch_contraction(dt_, g, st, L);
            }
        }
    }

private:
    // whole tiles of 64 sample pairs, 16-bit formats
    bool pair_tiles() const { return dt_ != MPODE_F32 && B_ % 64 == 0; }
    bool pair_bwd_ = false;
    std::vector<std::vector<size_t>> U_;
    std::vector<size_t> cot_;
    size_t uL_ = 0, wide_ = 0;
    const signed char* probe_ = nullptr;
};

// ---------------------------------------------------------------------------------------------------- conv
class ConvVelocity : public Velocity {
public:
    ConvVelocity(const mpode_velocity_desc& v, int B, mpode_dtype dt, int /*max_steps*/) : B_(B), dt_(dt), H_(v.H), W_(v.W), C_(v.C),
        act_(v.act) {
        n1_ = (size_t)C_ * 9 * (C_ + 1);
        n2_ = (size_t)C_ * 9 * C_;
        o_w1_ = 0; o_b1_ = n1_; o_w2_ = n1_ + C_; o_b2_ = n1_ + C_ + n2_;
        p_ = n1_ + C_ + n2_ + C_;
    }
    size_t param_count() const override { return p_; }

    void plan(Layout& lay) override {
        const size_t es = low_size(dt_);
        const size_t pix = (size_t)B_ * H_ * W_;
        plan_common(lay, B_, H_ * W_ * C_, H_ * W_ * C_, p_, dt_, 1);
        w1_ = lay.take(n1_ * es);
        w1t_ = lay.take(n2_ * es);      // [C][9 flipped][C]: data channels only
        w2_ = lay.take(n2_ * es);
        w2t_ = lay.take(n2_ * es);
        b1_ = lay.take((size_t)C_ * es);
        b2_ = lay.take((size_t)C_ * es);
        for (int j = 0; j < 4; ++j) h1_[j] = lay.take(pix * C_ * es);
        dz1_ = lay.take(pix * C_ * es);
        w1d_ = lay.take(n2_ * es);                              // first conv without the time channel: [C][9][C]
        for (int j = 0; j < 4; ++j) tb1_[j] = lay.take((size_t)9 * C_ * sizeof(float));
        tb2_ = lay.take((size_t)9 * C_ * sizeof(float));
        split_ = 1;
        while (split_ < 64 && (size_t)split_ * 2 * 4096 <= pix) split_ *= 2;   // >= 4096 pixels per slice
        partial_bytes_ = (size_t)split_ * n1_ * sizeof(float);
        if (dt_ != MPODE_F32 && C_ == 64 && conv_wgrad_tc_scratch_bytes(B_, H_, W_, C_) > partial_bytes_)
            partial_bytes_ = conv_wgrad_tc_scratch_bytes(B_, H_, W_, C_);
        if (dt_ != MPODE_F32 && C_ == 64 && W_ >= 8 && W_ <= 32 && conv_wgrad_halo_scratch_bytes(B_, H_, W_) > partial_bytes_)
            partial_bytes_ = conv_wgrad_halo_scratch_bytes(B_, H_, W_);
        partial_ = lay.take(partial_bytes_);
        tws_ = lay.take(((size_t)8 * 148 + 1) * 9 * C_ * sizeof(float));
        colsum_ = lay.take((size_t)64 * C_ * sizeof(float));
        ind_ = lay.take((size_t)H_ * W_ * 64 * es);             // position-class indicator table of one image
    }

    void prepare(cudaStream_t st, void* ws, const float* theta, const signed char*, long long* L) override {
        if (dt_ != MPODE_F32) launch_conv_class_indicator(dt_, H_, W_, at(ws, ind_), st, L);
        launch_quantize_conv_weights(dt_, theta + o_w1_, C_, C_ + 1, C_ + 1, at(ws, w1_), nullptr, st, L);
        launch_quantize_conv_weights(dt_, theta + o_w1_, C_, C_ + 1, C_, nullptr, at(ws, w1t_), st, L);
        launch_quantize_conv_weights(dt_, theta + o_w1_, C_, C_ + 1, C_, at(ws, w1d_), nullptr, st, L);
        launch_quantize_conv_weights(dt_, theta + o_w2_, C_, C_, C_, at(ws, w2_), at(ws, w2t_), st, L);
        launch_quantize_matrix(dt_, theta + o_b1_, C_, 1, C_, at(ws, b1_), nullptr, st, L);
        launch_quantize_matrix(dt_, theta + o_b2_, C_, 1, C_, at(ws, b2_), nullptr, st, L);
        launch_conv_class_bias(dt_, at(ws, b2_), nullptr, C_, 0.f, C_, (float*)at(ws, tb2_), st, L);
    }

    GemmArgs conv_args(void* ws, const void* x, int ct, float tau, const void* w, int k, int epi) const {
        GemmArgs g = base_args(ws, lay_);
        g.A = x; g.conv_on = 1; g.conv_h = H_; g.conv_w = W_; g.conv_cd = C_; g.conv_ct = ct; g.conv_tau = tau;
        g.B = w; g.b_rs = k; g.b_ks = 1;
        g.M = B_ * H_ * W_; g.N = C_; g.K = k;
        g.epi = epi; g.ldo = C_;
        return g;
    }

    void forward(cudaStream_t st, void* ws, int j, const void* yin, float tau16, long long* L) override {
        // tensor-core form of the first convolution: 64 data channels per tap, the time channel folded into a bias per
        // position class; when the shape does not allow it, the general kernel takes the 65-channel form
        GemmArgs g = conv_args(ws, yin, C_, 0.f, at(ws, w1d_), 9 * C_, EPI_FWD);
        g.conv_tbias = (const float*)at(ws, tb1_[j]);
        g.bias = at(ws, b1_); g.act = act_; g.out = at(ws, h1_[j]);
        if (tc_eligible(dt_, g)) {
            launch_conv_class_bias(dt_, at(ws, b1_), at(ws, w1_), C_ + 1, tau16, C_, (float*)at(ws, tb1_[j]), st, L);
        } else {
            g = conv_args(ws, yin, C_ + 1, tau16, at(ws, w1_), 9 * (C_ + 1), EPI_FWD);
            g.bias = at(ws, b1_); g.act = act_; g.out = at(ws, h1_[j]);
        }
        launch_contraction(dt_, g, st, L);
        g = conv_args(ws, at(ws, h1_[j]), C_, 0.f, at(ws, w2_), 9 * C_, EPI_FWD);
        g.conv_tbias = (const float*)at(ws, tb2_);
        g.bias = at(ws, b2_); g.act = MPODE_ACT_NONE; g.out = at(ws, lay_->kbuf[j]);
        launch_contraction(dt_, g, st, L);
    }

    // weight gradient of one convolution (and of its appended time channel when ct > C) plus its bias gradient
    void wgrad(cudaStream_t st, void* ws, const void* dz, const void* x, int ct, float tau, float* out, float* bias_out, float beta,
               long long* L) const {
        unsigned* err = (unsigned*)((char*)ws + lay_->scal) + 2;
        Profiler* pr = tl_profiler;
        const bool timed = pr != nullptr && pr->enabled;
        float* partial = (float*)at(ws, partial_);
        float* class_scratch = (float*)at(ws, tws_);
        const bool halo = conv_wgrad_halo_eligible(dt_, B_, H_, W_, C_, dz, x, partial, partial_bytes_, err);
        const bool tc_form = halo || conv_wgrad_tc_eligible(dt_, B_, H_, W_, C_, dz, x, partial, partial_bytes_, err);
        // tensor-core forms: from one image block per 64 pixels where the shape allows (that kernel also sums the cotangent per
        // position class), else tap by tap
        bool on_tc = false, classes_done = false;
        unsigned* counter = (unsigned*)((char*)ws + lay_->scal) + 16;   // a word of the scalar slice: zero between kernels
        if (tc_form && timed) pr->begin(2, 2.0 * B_ * H_ * W_ * 9.0 * C_ * C_, st);
        if (halo && launch_conv_wgrad_halo(dt_, dz, x, at(ws, ind_), B_, H_, W_, ct, out, bias_out, tau, beta, partial, class_scratch, counter, err, st, L)) {
            on_tc = classes_done = true;
        } else if (tc_form) {
            on_tc = conv_wgrad_tc_eligible(dt_, B_, H_, W_, C_, dz, x, partial, partial_bytes_, err) &&
                    launch_conv_wgrad_tc(dt_, dz, x, B_, H_, W_, C_, ct, out, beta, partial, err, st, L);
        }
        if (tc_form && timed) pr->end(st);
        if (on_tc) {
            if (tl_counters) ++tl_counters->tc;
            // the appended time channel is not an operand of the tensor-core form: its weights' gradient is a sum of the
            // cotangent over the pixels where the tap is inside the image
            if (!classes_done)
                launch_conv_class_grads(dt_, dz, B_, H_, W_, C_, ct, tau, class_scratch, ct > C_ ? out : nullptr, bias_out, beta, st, L);
            return;
        }
        launch_colsum(dt_, dz, B_ * H_ * W_, C_, (float*)at(ws, colsum_), bias_out, 1, nullptr, 0, 0.f, beta, st, L, colsum_counters(ws, lay_));
        GemmArgs g = base_args(ws, lay_);
        g.A = dz; g.a_rs = 1; g.a_ks = C_;
        g.B = x; g.conv_on = 2; g.conv_h = H_; g.conv_w = W_; g.conv_cd = C_; g.conv_ct = ct; g.conv_tau = tau;
        g.M = C_; g.N = 9 * ct; g.K = B_ * H_ * W_;
        g.epi = EPI_WGRAD; g.out = out; g.ldo = 9 * ct; g.beta = beta;
        g.split_k = split_; g.partial = (float*)at(ws, partial_);
        launch_contraction(dt_, g, st, L);
    }

    void vjp(cudaStream_t st, void* ws, int j, const void* yin, float tau16, void* psi_out, float* dg, float beta,
             unsigned* flag, long long* L) override {
        const void* dz2 = at(ws, lay_->kappa);
        const int pix = B_ * H_ * W_;
        wgrad(st, ws, dz2, at(ws, h1_[j]), C_, 0.f, dg + o_w2_, dg + o_b2_, beta, L);
        GemmArgs g = conv_args(ws, dz2, C_, 0.f, at(ws, w2t_), 9 * C_, EPI_DGRAD);
        g.hprev = at(ws, h1_[j]); g.ldh = C_; g.act = act_; g.flag = flag; g.out = at(ws, dz1_);
        launch_contraction(dt_, g, st, L);
        wgrad(st, ws, at(ws, dz1_), yin, C_ + 1, tau16, dg + o_w1_, dg + o_b1_, beta, L);
        g = conv_args(ws, at(ws, dz1_), C_, 0.f, at(ws, w1t_), 9 * C_, EPI_DGRAD);
        g.flag = flag; g.out = psi_out;
        // the previous stage's cotangent kappa = Q16(b v + c psi) in the same epilogue where the kernel has that output, else by
        // the elementwise kernel
        const KappaNext kn = next_;
        next_.out = nullptr;
        if (kn.out != nullptr) { g.kap_out = kn.out; g.kap_v = kn.v; g.kap_bv = kn.bv; g.kap_c = kn.c; }
        const int path = launch_contraction(dt_, g, st, L);
        if (kn.out != nullptr && path != 2) {
            Terms t{};
            t.n = 1; t.p[0] = psi_out; t.c[0] = kn.c;
            launch_kappa(dt_, kn.v, kn.bv, t, kn.out, (long long)pix * C_, flag, st, L);
        }
    }

    bool can_write_next_kappa() const override { return dt_ != MPODE_F32; }
    void set_next_kappa(const KappaNext& n) override { next_ = n; }

    void bind(const Layout* lay) { lay_ = lay; }

private:
    int B_;
    mpode_dtype dt_;
    int H_, W_, C_;
    int act_;
    size_t n1_, n2_, o_w1_, o_b1_, o_w2_, o_b2_, p_;
    size_t w1_ = 0, w1t_ = 0, w2_ = 0, w2t_ = 0, b1_ = 0, b2_ = 0, h1_[4] = {0}, dz1_ = 0, partial_ = 0, colsum_ = 0;
    size_t w1d_ = 0, tb1_[4] = {0}, tb2_ = 0, tws_ = 0, partial_bytes_ = 0, ind_ = 0;
    KappaNext next_{};
    int split_ = 1;
    const Layout* lay_ = nullptr;
};

// ---------------------------------------------------------------------------------------------------- parabolic conv layer
// f = -W^T N(relu(W y + b)) (Sec. 6.3, Eq. (NODE_STL10)): two convolutions with the same weights.  The transposed convolution is
// a convolution with the flipped, transposed weights; the minus signs are carried by negated copies of the rounded weights
// (Q16(-w) = -Q16(w)), so that every operator output is rounded once, as in the other velocities.
class ParabolicVelocity : public Velocity {
public:
    ParabolicVelocity(const mpode_velocity_desc& v, int B, mpode_dtype dt, int /*max_steps*/) : B_(B), dt_(dt), H_(v.H), W_(v.W), C_(v.C),
        pieces_(v.n_intervals), norm_(v.instance_norm != 0) {
        nw_ = (size_t)C_ * 9 * C_;
        per_ = nw_ + C_;
        p_ = per_ * pieces_;
    }
    size_t param_count() const override { return p_; }
    void set_step(int step, int n_steps) override { piece_ = (int)((long long)step * pieces_ / n_steps); }

    void plan(Layout& lay) override {
        const size_t es = low_size(dt_);
        const size_t pix = (size_t)B_ * H_ * W_;
        plan_common(lay, B_, H_ * W_ * C_, H_ * W_ * C_, p_, dt_, 1);
        for (int i = 0; i < pieces_; ++i) {
            w_.push_back(lay.take(nw_ * es));        // W                (S = relu(conv(y, W) + b))
            wn_.push_back(lay.take(nw_ * es));       // -W               (dZ = -conv(kappa, W))
            wt_.push_back(lay.take(nw_ * es));       // W flipped, transposed  (psi = W^T dU)
            wtn_.push_back(lay.take(nw_ * es));      // -(W flipped, transposed)  (k = -W^T Z)
            b_.push_back(lay.take((size_t)C_ * es));
            tb_.push_back(lay.take((size_t)9 * C_ * sizeof(float)));
        }
        tb0_ = lay.take((size_t)9 * C_ * sizeof(float));
        for (int j = 0; j < 4; ++j) {
            s_[j] = lay.take(pix * C_ * es);
            z_[j] = norm_ ? lay.take(pix * C_ * es) : s_[j];
            r_[j] = lay.take((size_t)B_ * C_ * sizeof(float));
        }
        dz_ = lay.take(pix * C_ * es);
        du_ = lay.take(pix * C_ * es);
        split_ = 1;
        while (split_ < 64 && (size_t)split_ * 2 * 4096 <= pix) split_ *= 2;
        partial_bytes_ = (size_t)split_ * nw_ * sizeof(float);
        if (dt_ != MPODE_F32 && C_ % 64 == 0 && conv_wgrad_tc_scratch_bytes(B_, H_, W_, C_) > partial_bytes_)
            partial_bytes_ = conv_wgrad_tc_scratch_bytes(B_, H_, W_, C_);
        partial_ = lay.take(partial_bytes_);
        colsum_ = lay.take((size_t)64 * C_ * sizeof(float));
    }

    void prepare(cudaStream_t st, void* ws, const float* theta, const signed char*, long long* L) override {
        for (int i = 0; i < pieces_; ++i) {
            const float* wsrc = theta + (size_t)i * per_;
            launch_quantize_conv_weights(dt_, wsrc, C_, C_, C_, at(ws, w_[i]), at(ws, wt_[i]), st, L);
            launch_quantize_conv_weights(dt_, wsrc, C_, C_, C_, at(ws, wn_[i]), at(ws, wtn_[i]), st, L, -1.f);
            launch_quantize_matrix(dt_, wsrc + nw_, C_, 1, C_, at(ws, b_[i]), nullptr, st, L);
            launch_conv_class_bias(dt_, at(ws, b_[i]), nullptr, C_, 0.f, C_, (float*)at(ws, tb_[i]), st, L);
        }
        cudaMemsetAsync(at(ws, tb0_), 0, (size_t)9 * C_ * sizeof(float), st);
    }

    GemmArgs conv_args(void* ws, const void* x, const void* w, int epi) const {
        GemmArgs g = base_args(ws, lay_);
        g.A = x; g.conv_on = 1; g.conv_h = H_; g.conv_w = W_; g.conv_cd = C_; g.conv_ct = C_; g.conv_tau = 0.f;
        g.B = w; g.b_rs = 9 * C_; g.b_ks = 1;
        g.M = B_ * H_ * W_; g.N = C_; g.K = 9 * C_;
        g.epi = epi; g.ldo = C_;
        return g;
    }

    void forward(cudaStream_t st, void* ws, int j, const void* yin, float, long long* L) override {
        GemmArgs g = conv_args(ws, yin, at(ws, w_[piece_]), EPI_FWD);
        g.conv_tbias = (const float*)at(ws, tb_[piece_]);
        g.bias = at(ws, b_[piece_]); g.act = MPODE_ACT_RELU; g.out = at(ws, s_[j]);
        launch_contraction(dt_, g, st, L);
        if (norm_) launch_instnorm_fwd(dt_, at(ws, s_[j]), at(ws, z_[j]), (float*)at(ws, r_[j]), B_, H_ * W_, C_, 1e-5f, st, L);
        g = conv_args(ws, at(ws, z_[j]), at(ws, wtn_[piece_]), EPI_FWD);
        g.conv_tbias = (const float*)at(ws, tb0_);
        g.act = MPODE_ACT_NONE; g.out = at(ws, lay_->kbuf[j]);
        launch_contraction(dt_, g, st, L);
    }

    // out = beta * out + sign * dW with dW[cout][tap][cin] = sum over pixels of dz[p][cout] x[p + tap][cin]
    void wgrad(cudaStream_t st, void* ws, const void* dz, const void* x, float* out, float beta, float sign, long long* L) const {
        unsigned* err = (unsigned*)((char*)ws + lay_->scal) + 2;
        if (conv_wgrad_tc_eligible(dt_, B_, H_, W_, C_, dz, x, (const float*)at(ws, partial_), partial_bytes_, err)) {
            Profiler* pr = tl_profiler;
            const bool timed = pr != nullptr && pr->enabled;
            if (timed) pr->begin(2, 2.0 * B_ * H_ * W_ * 9.0 * C_ * C_, st);
            const bool done = launch_conv_wgrad_tc(dt_, dz, x, B_, H_, W_, C_, C_, out, beta, (float*)at(ws, partial_), err, st, L, sign);
            if (timed) pr->end(st);
            if (done) {
                if (tl_counters) ++tl_counters->tc;
                return;
            }
        }
        // CUDA-core path: the general kernel computes out <- beta * out + dW; a minus sign is put around it,
        // -(beta * (-out) + dW) = beta * out - dW
        GemmArgs g = base_args(ws, lay_);
        g.A = dz; g.a_rs = 1; g.a_ks = C_;
        g.B = x; g.conv_on = 2; g.conv_h = H_; g.conv_w = W_; g.conv_cd = C_; g.conv_ct = C_; g.conv_tau = 0.f;
        g.M = C_; g.N = 9 * C_; g.K = B_ * H_ * W_;
        g.epi = EPI_WGRAD; g.out = out; g.ldo = 9 * C_; g.beta = beta;
        g.split_k = split_; g.partial = (float*)at(ws, partial_);
        if (sign < 0.f) launch_scale(out, -1.f, (long long)nw_, st, L);
        launch_contraction(dt_, g, st, L);
        if (sign < 0.f) launch_scale(out, -1.f, (long long)nw_, st, L);
    }

    void vjp(cudaStream_t st, void* ws, int j, const void* yin, float, void* psi_out, float* dg, float beta, unsigned* flag,
             long long* L) override {
        const void* kap = at(ws, lay_->kappa);
        float* dw = dg + (size_t)piece_ * per_;
        float* db = dw + nw_;
        if (beta == 0.f) launch_fill(dg, 0.f, (long long)p_, st, L);      // first stage of the attempt: the other pieces' slices are zero
        // dZ = -conv(kappa, W): the transpose of k = -W^T Z
        GemmArgs g = conv_args(ws, kap, at(ws, wn_[piece_]), EPI_DGRAD);
        g.flag = flag; g.out = at(ws, dz_);
        launch_contraction(dt_, g, st, L);
        wgrad(st, ws, at(ws, z_[j]), kap, dw, 1.f, -1.f, L);               // k = -W^T Z as a function of W
        launch_instnorm_bwd(dt_, at(ws, dz_), at(ws, z_[j]), at(ws, s_[j]), (const float*)at(ws, r_[j]), at(ws, du_), B_, H_ * W_, C_,
                            MPODE_ACT_RELU, norm_ ? 1 : 0, flag, st, L);
        wgrad(st, ws, at(ws, du_), yin, dw, 1.f, 1.f, L);                  // S = relu(W y + b) as a function of W
        launch_colsum(dt_, at(ws, du_), B_ * H_ * W_, C_, (float*)at(ws, colsum_), db, 1, nullptr, 0, 0.f, 1.f, st, L, colsum_counters(ws, lay_));
        g = conv_args(ws, at(ws, du_), at(ws, wt_[piece_]), EPI_DGRAD);
        g.flag = flag; g.out = psi_out;
        launch_contraction(dt_, g, st, L);
    }

    void bind(const Layout* lay) { lay_ = lay; }

private:
    int B_;
    mpode_dtype dt_;
    int H_, W_, C_, pieces_;
    bool norm_;
    int piece_ = 0;
    size_t nw_ = 0, per_ = 0, p_ = 0;
    std::vector<size_t> w_, wn_, wt_, wtn_, b_, tb_;
    size_t tb0_ = 0, s_[4] = {0}, z_[4] = {0}, r_[4] = {0}, dz_ = 0, du_ = 0, partial_ = 0, colsum_ = 0, partial_bytes_ = 0;
    int split_ = 1;
    const Layout* lay_ = nullptr;
};

// ---------------------------------------------------------------------------------------------------- scalar example
// Example 1 of the paper: one state component, three parameters.  Both passes run as whole-solve kernels (one CTA, one thread
// per sample); there is no layer-by-layer form.
class ScalarPolyVelocity : public Velocity {
public:
    ScalarPolyVelocity(const mpode_velocity_desc&, int B, mpode_dtype dt, int max_steps) : B_(B), dt_(dt), max_steps_(max_steps) {}
    size_t param_count() const override { return 3; }
    bool supports_time_gradient() const override { return true; }
    void plan(Layout& lay) override {
        plan_common(lay, B_, 1, 1, 3, dt_, 1);
        scal_ = lay.take((size_t)max_steps_ * sizeof(RkStepScalars));
        log_ = lay.take(((size_t)4 * max_steps_ + 8) * sizeof(int));         // scale log, status words, t' [max_steps + 1]
    }
    void prepare(cudaStream_t, void*, const float*, const signed char*, long long*) override {}
    void forward(cudaStream_t, void*, int, const void*, float, long long*) override {}
    void vjp(cudaStream_t, void*, int, const void*, float, void*, float*, float, unsigned*, long long*) override {}
    TinyParams params(void* ws, const FusedSolve& fs, const float* theta) const {
        TinyParams t{};
        t.B = B_; t.d = 1; t.h = 2; t.stages = fs.stages; t.n_steps = fs.n_steps; t.poly = 1;
        t.theta = theta; t.scal = (const RkStepScalars*)at(ws, scal_); t.traj = const_cast<void*>(fs.traj);
        t.round_increment = fs.round_increment;
        return t;
    }
    bool whole_forward(cudaStream_t st, void* ws, const FusedSolve& fs, const float* theta, const float* y0, float* yT,
                       long long* L) override {
        cudaMemcpyAsync(at(ws, scal_), fs.scalars.data(), (size_t)fs.n_steps * sizeof(RkStepScalars), cudaMemcpyHostToDevice, st);
        TinyParams t = params(ws, fs, theta);
        t.y0 = y0; t.yT = yT;
        launch_tiny_forward(dt_, t, st, L);
        if (tl_counters) ++tl_counters->whole;
        return true;
    }
    bool whole_backward(cudaStream_t st, void* ws, const FusedSolve& fs, WholeBackward& wb, long long* L) override {
        const int N = fs.n_steps;
        cudaMemcpyAsync(at(ws, scal_), fs.scalars.data(), (size_t)N * sizeof(RkStepScalars), cudaMemcpyHostToDevice, st);
        int* logs = (int*)at(ws, log_);
        cudaMemsetAsync(logs, 0, ((size_t)4 * max_steps_ + 8) * sizeof(int), st);
        TinyParams t = params(ws, fs, wb.theta);
        t.dLdyT = wb.dLdyT; t.a = wb.a; t.g = wb.g; t.accumulate = wb.accumulate;
        t.scaling = wb.scaling; t.k_max = wb.k_max; t.growth_rule = wb.growth_rule; t.pbits = wb.pbits;
        t.e0 = wb.e0; t.e0_from_norm = wb.e0_from_norm;
        t.log_exp = logs; t.log_attempts = logs + max_steps_; t.log_doubled = logs + 2 * max_steps_; t.status = logs + 3 * max_steps_;
        t.cot = wb.cot;
        t.tprime = wb.dt_host != nullptr ? (float*)(logs + 3 * max_steps_ + 4) : nullptr;
        launch_tiny_backward(dt_, t, st, L);
        if (tl_counters) ++tl_counters->whole;
        std::vector<int> h((size_t)3 * max_steps_ + 4);
        cudaMemcpyAsync(h.data(), logs, h.size() * sizeof(int), cudaMemcpyDeviceToHost, st);
        if (wb.dt_host != nullptr) cudaMemcpyAsync(wb.dt_host, t.tprime, (size_t)(N + 1) * sizeof(float), cudaMemcpyDeviceToHost, st);
        cudaStreamSynchronize(st);
        const int* stp = h.data() + 3 * max_steps_;
        wb.status = stp[0]; wb.first_failed_step = wb.status == MPODE_ERR_SCALE_FAILED ? stp[1] : -1; wb.retries = stp[2];
        for (int i = 0; i < N; ++i) {
            if (wb.exp_used) wb.exp_used[i] = h[i];
            if (wb.attempts) wb.attempts[i] = h[max_steps_ + i];
            if (wb.doubled) wb.doubled[i] = (unsigned char)h[2 * max_steps_ + i];
        }
        return true;
    }
    void bind(const Layout* lay) { lay_ = lay; }

private:
    int B_;
    mpode_dtype dt_;
    int max_steps_;
    size_t scal_ = 0, log_ = 0;
    const Layout* lay_ = nullptr;
};

// ---------------------------------------------------------------------------------------------------- hypernetwork flow, exact trace
// Sec. 6.1 (two-dimensional flows): joint state [z; l], z' = (1/w) sum_j U_j(t) tanh(W_j(t) . z + b_j(t)), l' = -tr(dz'/dz) written
// out; the weight sets come from t through three fully connected layers (hyper_cnf.cu).  Layer-by-layer path only.
class HyperCnfVelocity : public Velocity {
public:
    HyperCnfVelocity(const mpode_velocity_desc& v, int B, mpode_dtype dt, int max_steps) : B_(B), dt_(dt), d_(v.d), h_(v.widths[0]),
        w_(v.widths[1]), max_steps_(max_steps) {}
    size_t param_count() const override { return hyper_param_count(h_, w_, d_); }
    void plan(Layout& lay) override {
        const size_t es = low_size(dt_);
        plan_common(lay, B_, d_, d_ + 1, param_count(), dt_, 1);
        for (int j = 0; j < 4; ++j) {
            hyp_[j] = lay.take(hyper_stage_floats(h_, w_, d_) * sizeof(float));
            units_[j] = lay.take((size_t)w_ * B_ * es);
        }
        // one set per stage of what a whole-step vector-Jacobian product keeps: unit cotangents, stage cotangents, batch sums
        for (int j = 0; j < 4; ++j) {
            sbar_[j] = lay.take((size_t)w_ * B_ * es);
            kap_[j] = lay.take((size_t)B_ * d_ * es);
            kapl_[j] = lay.take((size_t)B_ * es);
        }
        part_ = lay.take(hyper_step_scratch_floats(h_, w_, d_) * sizeof(float));
        // the hypernetwork's layers and weight sets for every stage time of a solve, and those times
        table_ = lay.take((size_t)max_steps_ * 4 * hyper_stage_floats(h_, w_, d_) * sizeof(float));
        taus_ = lay.take((size_t)max_steps_ * 4 * sizeof(float));
    }
    void prepare(cudaStream_t, void*, const float* theta, const signed char*, long long*) override { theta_ = theta; by_step_ = false; }
    void prepare_solve(cudaStream_t st, void* ws, const FusedSolve& fs, long long* L) override {
        by_step_ = hyper_step_shape_ok(h_, w_, d_, fs.stages) && fs.n_steps <= max_steps_;
        if (!by_step_) return;
        taus_host_.assign((size_t)fs.n_steps * 4, 0.f);
        for (int i = 0; i < fs.n_steps; ++i)
            for (int j = 0; j < fs.stages; ++j) taus_host_[(size_t)i * 4 + j] = fs.scalars[i].tau16[j];
        cudaMemcpyAsync(at(ws, taus_), taus_host_.data(), taus_host_.size() * sizeof(float), cudaMemcpyHostToDevice, st);
        launch_hyper_table(dt_, theta_, (const float*)at(ws, taus_), fs.n_steps * 4, h_, w_, d_, (float*)at(ws, table_), st, L);
    }
    void set_step(int step, int) override { step_ = step; }
    void forward(cudaStream_t st, void* ws, int j, const void* yin, float tau16, long long* L) override {
        launch_hyper_forward(dt_, theta_, tau16, h_, w_, d_, (float*)at(ws, hyp_[j]), yin, at(ws, units_[j]), at(ws, lay_->kbuf[j]),
                             at(ws, lay_->klbuf[j]), B_, st, L);
    }
    void vjp(cudaStream_t st, void* ws, int j, const void* yin, float tau16, void* psi_out, float* dg, float beta, unsigned* flag,
             long long* L) override {
        unsigned* counter = (unsigned*)at(ws, lay_->scal) + 17;     // a word of the scalar slice: zero between kernels
        launch_hyper_vjp(dt_, theta_, tau16, h_, w_, d_, (const float*)at(ws, hyp_[j]), yin, at(ws, units_[j]), at(ws, sbar_[0]),
                         at(ws, lay_->kappa), at(ws, lay_->kappal), psi_out, (float*)at(ws, part_), dg, beta, B_, flag, counter, st, L);
    }
    bool step_forward(cudaStream_t st, void* ws, const void* ybar, const RkStepScalars& sc, int stages, long long* L) override {
        if (!by_step_) return false;
        launch_hyper_step_forward(dt_, sc, stages, h_, w_, d_, stage_ptrs(ws), ybar, B_, st, L);
        return true;
    }
    bool step_vjp(cudaStream_t st, void* ws, const void* ybar, const RkStepScalars& sc, int stages, float* dg, unsigned* flag,
                  long long* L) override {
        if (!by_step_) return false;
        unsigned* counter = (unsigned*)at(ws, lay_->scal) + 20;     // words 20 .. 23 of the scalar slice
        launch_hyper_step_vjp(dt_, theta_, sc, stages, h_, w_, d_, stage_ptrs(ws), ybar, at(ws, lay_->v), at(ws, lay_->vl),
                              (float*)at(ws, part_), dg, B_, flag, counter, st, L);
        return true;
    }
    void bind(const Layout* lay) { lay_ = lay; }

private:
    HyperStagePtrs stage_ptrs(void* ws) const {
        HyperStagePtrs p{};
        for (int j = 0; j < 4; ++j) {
            p.hyp[j] = (float*)at(ws, table_) + ((size_t)step_ * 4 + j) * hyper_stage_floats(h_, w_, d_); p.A[j] = at(ws, units_[j]); p.k[j] = at(ws, lay_->kbuf[j]); p.kl[j] = at(ws, lay_->klbuf[j]);
            p.y[j] = at(ws, lay_->ybuf[j]); p.psi[j] = at(ws, lay_->psi[j]); p.sb[j] = at(ws, sbar_[j]); p.kap[j] = at(ws, kap_[j]);
            p.kapl[j] = at(ws, kapl_[j]);
        }
        return p;
    }
    int B_;
    mpode_dtype dt_;
    int d_, h_, w_;
    int max_steps_, step_ = 0;
    bool by_step_ = false;                 // this pass goes step by step on the table of weight sets
    std::vector<float> taus_host_;
    size_t hyp_[4] = {0}, units_[4] = {0}, sbar_[4] = {0}, kap_[4] = {0}, kapl_[4] = {0}, part_ = 0, table_ = 0, taus_ = 0;
    const float* theta_ = nullptr;
    const Layout* lay_ = nullptr;
};

// A velocity keeps a pointer to the context's layout; plan() is called exactly once, on that layout.
template <typename V>
class Bound : public V {
public:
    using V::V;
    void plan(Layout& lay) override {
        V::plan(lay);
        this->bind(&lay);
    }
};

}  // namespace

Velocity* make_velocity(const mpode_velocity_desc& desc, int batch, mpode_dtype low, int max_steps) {
    switch (desc.kind) {
        case MPODE_VEL_MLP: return new Bound<MlpVelocity>(desc, batch, low, max_steps);
        case MPODE_VEL_CNF_MLP: return new Bound<CnfVelocity>(desc, batch, low, max_steps);
        case MPODE_VEL_CONV3X3_2: return new Bound<ConvVelocity>(desc, batch, low, max_steps);
        case MPODE_VEL_PARABOLIC_CONV: return new Bound<ParabolicVelocity>(desc, batch, low, max_steps);
        case MPODE_VEL_SCALAR_POLY: return batch <= TINY_MAX_B ? new Bound<ScalarPolyVelocity>(desc, batch, low, max_steps) : nullptr;
        case MPODE_VEL_CNF_HYPER: return new Bound<HyperCnfVelocity>(desc, batch, low, max_steps);
    }
    return nullptr;
}

}  // namespace mpode
