// The built-in velocity networks as sequences of contraction + fused-epilogue launches.
#include <vector>

#include "gemm_tc.h"
#include "velocity.h"

namespace mpode {

void launch_contraction(mpode_dtype dt, const GemmArgs& g, cudaStream_t st, long long* L);  // dispatch.cu

namespace {

inline char* at(void* ws, size_t off) { return (char*)ws + off; }

void plan_common(Layout& lay, int B, int d, int D, size_t p, mpode_dtype dt, int ybuf_rows_factor) {
    const size_t es = low_size(dt);
    lay.scal = lay.take(256);
    for (int j = 0; j < 4; ++j) lay.kbuf[j] = lay.take((size_t)B * d * es);
    for (int j = 0; j < 4; ++j) lay.ybuf[j] = lay.take((size_t)ybuf_rows_factor * B * d * es);
    for (int j = 0; j < 4; ++j) lay.psi[j] = lay.take((size_t)B * d * es);
    lay.v = lay.take((size_t)B * d * es);
    lay.kappa = lay.take((size_t)B * d * es);
    if (D > d) {
        for (int j = 0; j < 4; ++j) lay.klbuf[j] = lay.take((size_t)B * es);
        lay.vl = lay.take((size_t)B * es);
        lay.kappal = lay.take((size_t)B * es);
    }
    lay.dg = lay.take(p * sizeof(float));
}

GemmArgs base_args(void* ws, const Layout* lay) {
    GemmArgs g{};
    g.split_k = 1;
    g.err = (unsigned*)((char*)ws + lay->scal) + 2;   // third word of the scalar slice
    return g;
}

// ---------------------------------------------------------------------------------------------------- MLP
class MlpVelocity : public Velocity {
public:
    MlpVelocity(const mpode_velocity_desc& v, int B, mpode_dtype dt) : B_(B), dt_(dt), act_(v.act),
        time_(v.append_time != 0), bias_(v.has_bias != 0), L_(v.n_layers), w_(v.widths, v.widths + v.n_layers + 1) {
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

    void plan(Layout& lay) override {
        const size_t es = low_size(dt_);
        plan_common(lay, B_, w_[0], w_[0], p_, dt_, 1);
        int maxw = 0;
        for (int l = 0; l < L_; ++l) {
            W16_.push_back(lay.take((size_t)w_[l + 1] * w_[l] * es));
            W16T_.push_back(lay.take((size_t)w_[l + 1] * w_[l] * es));
            b16_.push_back(bias_ ? lay.take((size_t)w_[l + 1] * es) : 0);
            maxw = w_[l + 1] > maxw ? w_[l + 1] : maxw;
        }
        wt16_ = time_ ? lay.take((size_t)w_[1] * es) : 0;
        for (int j = 0; j < 4; ++j) {
            std::vector<size_t> hs(L_, 0);
            for (int l = 1; l < L_; ++l) hs[l] = lay.take((size_t)B_ * w_[l] * es);
            H_.push_back(hs);
        }
        dZ_.assign(L_, 0);
        for (int l = 1; l < L_; ++l) dZ_[l] = lay.take((size_t)B_ * w_[l] * es);
        colsum_ = lay.take((size_t)64 * maxw * sizeof(float));
        size_t wg = 0;
        for (int l = 0; l < L_; ++l) {
            size_t b = wgrad_tc_scratch_bytes(w_[l + 1], w_[l], B_);
            wg = b > wg ? b : wg;
        }
        wgpart_ = lay.take(wg);
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
                g.partial = (float*)at(ws, wgpart_);
                launch_contraction(dt_, g, st, L);
            }
            if (bias_ || (time_ && l == 0))
                launch_colsum(dt_, dZ, B_, w_[l + 1], (float*)at(ws, colsum_), bias_ ? dg + boff_[l] : nullptr, 1,
                              (time_ && l == 0) ? dg + woff_[l] + w_[l] : nullptr, in_full, tau16, beta, st, L);
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

    void bind(const Layout* lay) { lay_ = lay; }

protected:
    int B_;
    mpode_dtype dt_;
    int act_;
    bool time_, bias_;
    int L_;
    std::vector<int> w_;
    std::vector<size_t> woff_, boff_, W16_, W16T_, b16_, dZ_;
    std::vector<std::vector<size_t>> H_;
    size_t wt16_ = 0, colsum_ = 0, wgpart_ = 0, p_ = 0;
    const Layout* lay_ = nullptr;
};

// ---------------------------------------------------------------------------------------------------- CNF
// Primal rows and tangent rows share every weight, so each layer runs as one contraction over 2B rows:
// rows [0, B) carry the state, rows [B, 2B) the forward-mode tangent started at the probe (Sec. 6.1).
class CnfVelocity : public MlpVelocity {
public:
    CnfVelocity(const mpode_velocity_desc& v, int B, mpode_dtype dt) : MlpVelocity(v, B, dt) {}

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
        wide_ = lay.take((size_t)2 * B_ * maxw * sizeof(float));
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
            launch_contraction(dt_, g, st, L);
            if (!last) {
                long long n = (long long)B_ * w_[l + 1];
                launch_cnf_tangent_act(dt_, act_, at(ws, H_[j][l + 1]), at(ws, U_[j][l + 1]),
                                       at(ws, H_[j][l + 1]) + n * es, n, st, L);
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
                              (time_ && l == 0) ? dg + woff_[l] + w_[l] : nullptr, in_full, tau16, beta, st, L);
            if (l > 0) {
                GemmArgs g = base_args(ws, lay_);
                g.A = C; g.a_rs = w_[l + 1]; g.a_ks = 1;
                g.B = at(ws, W16T_[l]); g.b_rs = w_[l + 1]; g.b_ks = 1;
                g.M = 2 * B_; g.N = w_[l]; g.K = w_[l + 1];
                g.epi = EPI_RAW32; g.out = at(ws, wide_); g.ldo = w_[l];
                launch_contraction(dt_, g, st, L);
                long long n = (long long)B_ * w_[l];
                float* wide = (float*)at(ws, wide_);
                launch_cnf_backprop_act(dt_, act_, at(ws, H_[j][l]), at(ws, U_[j][l]), wide, wide + n, at(ws, cot_[l]),
                                        at(ws, cot_[l]) + n * es, n, flag, st, L);
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
    std::vector<std::vector<size_t>> U_;
    std::vector<size_t> cot_;
    size_t uL_ = 0, wide_ = 0;
    const signed char* probe_ = nullptr;
};

// ---------------------------------------------------------------------------------------------------- conv
class ConvVelocity : public Velocity {
public:
    ConvVelocity(const mpode_velocity_desc& v, int B, mpode_dtype dt) : B_(B), dt_(dt), H_(v.H), W_(v.W), C_(v.C) {
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
        split_ = 1;
        while (split_ < 64 && (size_t)split_ * 2 * 4096 <= pix) split_ *= 2;   // >= 4096 pixels per slice
        partial_ = lay.take((size_t)split_ * n1_ * sizeof(float));
        colsum_ = lay.take((size_t)64 * C_ * sizeof(float));
    }

    void prepare(cudaStream_t st, void* ws, const float* theta, const signed char*, long long* L) override {
        launch_quantize_conv_weights(dt_, theta + o_w1_, C_, C_ + 1, C_ + 1, at(ws, w1_), nullptr, st, L);
        launch_quantize_conv_weights(dt_, theta + o_w1_, C_, C_ + 1, C_, nullptr, at(ws, w1t_), st, L);
        launch_quantize_conv_weights(dt_, theta + o_w2_, C_, C_, C_, at(ws, w2_), at(ws, w2t_), st, L);
        launch_quantize_matrix(dt_, theta + o_b1_, C_, 1, C_, at(ws, b1_), nullptr, st, L);
        launch_quantize_matrix(dt_, theta + o_b2_, C_, 1, C_, at(ws, b2_), nullptr, st, L);
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
        GemmArgs g = conv_args(ws, yin, C_ + 1, tau16, at(ws, w1_), 9 * (C_ + 1), EPI_FWD);
        g.bias = at(ws, b1_); g.act = MPODE_ACT_RELU; g.out = at(ws, h1_[j]);
        launch_contraction(dt_, g, st, L);
        g = conv_args(ws, at(ws, h1_[j]), C_, 0.f, at(ws, w2_), 9 * C_, EPI_FWD);
        g.bias = at(ws, b2_); g.act = MPODE_ACT_NONE; g.out = at(ws, lay_->kbuf[j]);
        launch_contraction(dt_, g, st, L);
    }

    void wgrad(cudaStream_t st, void* ws, const void* dz, const void* x, int ct, float tau, float* out, float beta,
               long long* L) const {
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
        wgrad(st, ws, dz2, at(ws, h1_[j]), C_, 0.f, dg + o_w2_, beta, L);
        launch_colsum(dt_, dz2, pix, C_, (float*)at(ws, colsum_), dg + o_b2_, 1, nullptr, 0, 0.f, beta, st, L);
        GemmArgs g = conv_args(ws, dz2, C_, 0.f, at(ws, w2t_), 9 * C_, EPI_DGRAD);
        g.hprev = at(ws, h1_[j]); g.ldh = C_; g.act = MPODE_ACT_RELU; g.flag = flag; g.out = at(ws, dz1_);
        launch_contraction(dt_, g, st, L);
        wgrad(st, ws, at(ws, dz1_), yin, C_ + 1, tau16, dg + o_w1_, beta, L);
        launch_colsum(dt_, at(ws, dz1_), pix, C_, (float*)at(ws, colsum_), dg + o_b1_, 1, nullptr, 0, 0.f, beta, st, L);
        g = conv_args(ws, at(ws, dz1_), C_, 0.f, at(ws, w1t_), 9 * C_, EPI_DGRAD);
        g.flag = flag; g.out = psi_out;
        launch_contraction(dt_, g, st, L);
    }

    void bind(const Layout* lay) { lay_ = lay; }

private:
    int B_;
    mpode_dtype dt_;
    int H_, W_, C_;
    size_t n1_, n2_, o_w1_, o_b1_, o_w2_, o_b2_, p_;
    size_t w1_ = 0, w1t_ = 0, w2_ = 0, w2t_ = 0, b1_ = 0, b2_ = 0, h1_[4] = {0}, dz1_ = 0, partial_ = 0, colsum_ = 0;
    int split_ = 1;
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

Velocity* make_velocity(const mpode_velocity_desc& desc, int batch, mpode_dtype low) {
    switch (desc.kind) {
        case MPODE_VEL_MLP: return new Bound<MlpVelocity>(desc, batch, low);
        case MPODE_VEL_CNF_MLP: return new Bound<CnfVelocity>(desc, batch, low);
        case MPODE_VEL_CONV3X3_2: return new Bound<ConvVelocity>(desc, batch, low);
    }
    return nullptr;
}

}  // namespace mpode
