// Host driver: the time loop of Alg. 1, the reverse loop and scale state machine of Alg. 2, workspace carving
// and the C ABI.  All arithmetic of the method runs in the kernels; the host only sequences launches and takes
// the accept / halve / double decisions of Alg. 2 from two device words (flag, ||a||_inf).
#include <math.h>
#include <string.h>

#include <mutex>
#include <string>
#include <vector>

#include "common.cuh"
#include "profiler.h"
#include "tensormap.h"
#include "hyper_cnf.h"
#include "velocity.h"

using namespace mpode;

namespace {

const double kEulerA[1] = {0.0}, kEulerB[1] = {1.0}, kEulerC[1] = {0.0};
const double kRk4A[16] = {0, 0, 0, 0, 0.5, 0, 0, 0, 0, 0.5, 0, 0, 0, 0, 1.0, 0};
const double kRk4B[4] = {1.0 / 6, 1.0 / 3, 1.0 / 3, 1.0 / 6};
const double kRk4C[4] = {0.0, 0.5, 0.5, 1.0};
const mpode_tableau kEuler = {1, kEulerA, kEulerB, kEulerC};
const mpode_tableau kRk4 = {4, kRk4A, kRk4B, kRk4C};

constexpr int kExpMin = -100, kExpMax = 100;

inline int precision_bits(mpode_dtype dt) { return dt == MPODE_F16 ? 11 : dt == MPODE_BF16 ? 8 : 24; }

// S_N = 2^floor(-log2(u_L m)) (Alg. 2, scale initialisation) in integer arithmetic: with u_L = 2^-p and m = f 2^E, f in [0.5, 1),
// floor(p - log2 m) = p - E when f > 0.5 and p - E + 1 when f = 0.5.
int initial_scale_exponent(float m, mpode_dtype dt) {
    if (m == 0.f) return 0;
    int E;
    float f = frexpf(m, &E);
    int c = (f > 0.5f) ? E : E - 1;
    int e = precision_bits(dt) - c;
    return e < kExpMin ? kExpMin : (e > kExpMax ? kExpMax : e);
}

}  // namespace

struct mpode_ctx {
    mpode_velocity_desc vel{};
    std::vector<int> widths;
    int B = 0, max_steps = 0, d = 0, D = 0;
    mpode_policy pol{};
    Velocity* v = nullptr;
    Layout lay;
    // record of the last forward
    bool have_forward = false;
    const float* theta = nullptr;
    const signed char* probe = nullptr;
    const void* traj = nullptr;
    std::vector<float> tgrid;
    int n_steps = 0;
    int stages = 0;
    double ta[16], tb[4], tc[4];
    float tc_f[4] = {0, 0, 0, 0};           // c_j as floats (source of an asynchronous copy: must outlive the call's launches)
    std::string err;
    mpode_stats stats{};
    PathCounters counters;
    unsigned long long dbg_wait_ns = 0;     // test hook: 0 = default wait limit
    int dbg_starve = 0;
    void* ws_forward = nullptr;             // workspace of the last mpode_forward (its error word is read by the next synchronising call)
    Profiler prof;
    // second stream of the unchecked fused backward: the recompute of step i - 1 runs beside the reductions of step i
    cudaStream_t side = nullptr;
    cudaEvent_t ev_ready = nullptr, ev_vjp = nullptr, ev_rec = nullptr;
    bool allow_side = true;
    // dynamic scaling: the device's scale state mirrored into mapped host memory, and one event per step parity; the host
    // queues the attempt of step i - 1 only after step i was accepted (the recompute of step i - 1 is queued before that)
    int* mirror_host = nullptr;
    int* mirror_dev = nullptr;
    cudaEvent_t ev_step[2] = {nullptr, nullptr};
};

namespace {

mpode_status fail(mpode_ctx* c, mpode_status s, const std::string& msg) {
    if (c) c->err = msg;
    return s;
}

mpode_status check_cuda(mpode_ctx* c, const char* where) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(c, MPODE_ERR_CUDA, std::string(where) + ": " + cudaGetErrorString(e));
    return MPODE_OK;
}

struct StepTimes {
    float h;
    float tau16[4];
};

StepTimes step_times(const mpode_ctx* c, int i) {
    StepTimes s;
    double t0 = (double)c->tgrid[i], t1 = (double)c->tgrid[i + 1];
    s.h = (float)(t1 - t0);
    for (int j = 0; j < c->stages; ++j) {
        float tau = (float)(t0 + c->tc[j] * (double)s.h);
        s.tau16[j] = round_scalar_to_low(tau, c->pol.low);
    }
    return s;
}

inline char* at(void* ws, size_t off) { return (char*)ws + off; }

// Step size, stage times and tableau products of one step, each formed in double and rounded to fp32 once.
RkStepScalars step_scalars(const mpode_ctx* c, int i) {
    const int s = c->stages;
    const StepTimes tm = step_times(c, i);
    RkStepScalars sc;
    memset(&sc, 0, sizeof(sc));
    sc.h = tm.h;
    for (int j = 0; j < s; ++j) {
        sc.tau16[j] = tm.tau16[j];
        sc.b[j] = (float)c->tb[j];
        sc.c[j] = (float)c->tc[j];
        for (int l = 0; l < s; ++l) sc.a[j][l] = (float)c->ta[j * s + l];
        sc.hb[j] = c->pol.round_increment ? (float)c->tb[j] : (float)((double)tm.h * c->tb[j]);
        for (int l = 0; l < s; ++l) sc.ha[j][l] = (float)((double)tm.h * c->ta[j * s + l]);
    }
    return sc;
}

FusedSolve fused_solve(const mpode_ctx* c, float* y) {
    FusedSolve fs;
    fs.n_steps = c->n_steps;
    fs.stages = c->stages;
    fs.round_increment = c->pol.round_increment;
    fs.traj = c->traj;
    fs.y = y;
    if (c->dbg_wait_ns) fs.wait_ns = c->dbg_wait_ns;
    fs.starve = c->dbg_starve;
    for (int k = 0; k < 16; ++k) fs.a[k] = c->ta[k];
    fs.scalars.resize(c->n_steps);
    for (int i = 0; i < c->n_steps; ++i) fs.scalars[i] = step_scalars(c, i);
    return fs;
}

// Evaluate all stages of step i from the stored state traj[i] (increment of Alg. 1 / recompute of Alg. 2).
void run_stages(mpode_ctx* c, cudaStream_t st, void* ws, int i, const StepTimes& tm) {
    const mpode_dtype dt = c->pol.low;
    const size_t es = low_size(dt);
    const long long nBd = (long long)c->B * c->d;
    const char* traj_i = (const char*)c->traj + (size_t)i * nBd * es;
    long long* L = &c->stats.kernel_launches;
    if (!c->v->needs_input_copy() && c->v->step_forward(st, ws, traj_i, step_scalars(c, i), c->stages, L)) return;
    for (int j = 0; j < c->stages; ++j) {
        const void* yin = traj_i;
        if (j > 0 || c->v->needs_input_copy()) {
            Terms t{};
            t.n = 0;
            for (int l = 0; l < j; ++l) {
                double a = c->ta[j * c->stages + l];
                if (a != 0.0) {
                    t.p[t.n] = at(ws, c->lay.kbuf[l]);
                    t.c[t.n] = (float)((double)tm.h * a);
                    ++t.n;
                }
            }
            launch_stage_input(dt, traj_i, t, at(ws, c->lay.ybuf[j]), nBd, st, L);
            yin = at(ws, c->lay.ybuf[j]);
        }
        c->v->forward(st, ws, j, yin, tm.tau16[j], L);
    }
}

}  // namespace

extern "C" {

const mpode_tableau* mpode_tableau_euler(void) { return &kEuler; }
const mpode_tableau* mpode_tableau_rk4(void) { return &kRk4; }

const char* mpode_status_string(mpode_status s) {
    switch (s) {
        case MPODE_OK: return "ok";
        case MPODE_ERR_INVALID_ARG: return "invalid argument";
        case MPODE_ERR_UNSUPPORTED: return "unsupported configuration";
        case MPODE_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case MPODE_ERR_CUDA: return "CUDA error";
        case MPODE_ERR_BAD_STATE: return "backward called without a forward";
        case MPODE_ERR_NONFINITE_INPUT: return "non-finite dL/dy_T";
        case MPODE_ERR_SCALE_FAILED: return "dynamic adjoint scaling failed";
        case MPODE_WARN_NONFINITE_GRAD: return "overflow: gradients returned as Inf";
    }
    return "unknown status";
}

const char* mpode_last_error(const mpode_ctx* ctx) { return ctx ? ctx->err.c_str() : ""; }

mpode_status mpode_create(mpode_ctx** out, const mpode_velocity_desc* vel, int batch, int max_steps,
                          const mpode_policy* policy) {
    if (!out || !vel || !policy || batch <= 0 || max_steps <= 0) return MPODE_ERR_INVALID_ARG;
    *out = nullptr;
    if (policy->low != MPODE_F32 && policy->low != MPODE_BF16 && policy->low != MPODE_F16) return MPODE_ERR_INVALID_ARG;
    if (policy->scaling < MPODE_SCALE_NONE || policy->scaling > MPODE_SCALE_DYNAMIC) return MPODE_ERR_INVALID_ARG;
    mpode_ctx* c = new mpode_ctx();
    c->vel = *vel;
    c->B = batch;
    c->max_steps = max_steps;
    c->pol = *policy;
    if (c->pol.k_max <= 0) c->pol.k_max = 10;
    if (vel->kind == MPODE_VEL_MLP || vel->kind == MPODE_VEL_CNF_MLP) {
        if (vel->n_layers < 1 || vel->n_layers > 8 || !vel->widths) { delete c; return MPODE_ERR_INVALID_ARG; }
        c->widths.assign(vel->widths, vel->widths + vel->n_layers + 1);
        c->vel.widths = c->widths.data();
        for (int w : c->widths) if (w <= 0) { delete c; return MPODE_ERR_INVALID_ARG; }
        if (c->widths.front() != vel->d || c->widths.back() != vel->d) { delete c; return MPODE_ERR_INVALID_ARG; }
        if (vel->kind == MPODE_VEL_CNF_MLP && (vel->n_layers < 2 || vel->act != MPODE_ACT_SOFTPLUS)) {
            delete c; return MPODE_ERR_UNSUPPORTED;
        }
    } else if (vel->kind == MPODE_VEL_CONV3X3_2) {
        if (vel->H <= 0 || vel->W <= 0 || vel->C <= 0 || vel->d != vel->H * vel->W * vel->C) { delete c; return MPODE_ERR_INVALID_ARG; }
        if ((long long)batch * vel->H * vel->W > 0x7fffffffLL / 16) { delete c; return MPODE_ERR_UNSUPPORTED; }
    } else if (vel->kind == MPODE_VEL_PARABOLIC_CONV) {
        if (vel->H <= 0 || vel->W <= 0 || vel->C <= 0 || vel->d != vel->H * vel->W * vel->C || vel->n_intervals < 1 ||
            vel->n_intervals > max_steps) { delete c; return MPODE_ERR_INVALID_ARG; }
        if ((long long)batch * vel->H * vel->W > 0x7fffffffLL / 16) { delete c; return MPODE_ERR_UNSUPPORTED; }
    } else if (vel->kind == MPODE_VEL_SCALAR_POLY) {
        if (vel->d != 1) { delete c; return MPODE_ERR_INVALID_ARG; }
    } else if (vel->kind == MPODE_VEL_CNF_HYPER) {
        // widths = {hidden width of the hypernetwork, number of weight sets w}
        if (vel->d < 1 || vel->d > 8 || vel->n_layers != 1 || vel->widths == nullptr) { delete c; return MPODE_ERR_INVALID_ARG; }
        c->widths.assign(vel->widths, vel->widths + 2);
        c->vel.widths = c->widths.data();
        if (c->widths[0] < 1 || c->widths[0] > 256 || c->widths[1] < 1 || c->widths[1] > 1024) { delete c; return MPODE_ERR_UNSUPPORTED; }
        if (!hyper_shape_ok(c->widths[0], c->widths[1], vel->d)) { delete c; return MPODE_ERR_UNSUPPORTED; }
    } else {
        delete c; return MPODE_ERR_INVALID_ARG;
    }
    c->d = vel->d;
    c->D = (vel->kind == MPODE_VEL_CNF_MLP || vel->kind == MPODE_VEL_CNF_HYPER) ? vel->d + 1 : vel->d;
    c->v = make_velocity(c->vel, c->B, c->pol.low, c->max_steps);
    if (!c->v) { delete c; return MPODE_ERR_UNSUPPORTED; }
    if (c->pol.time_gradient) {
        // the rounded increment (round_increment = 1) would need Q16 of the combined stage derivatives inside Phi^T a
        if (!c->v->supports_time_gradient() || c->pol.round_increment) { delete c->v; delete c; return MPODE_ERR_UNSUPPORTED; }
        c->lay.time_gradient = true;
    }
    c->v->plan(c->lay);
    if (c->pol.scaling == MPODE_SCALE_DYNAMIC)      // the device-side scale log: exponent, attempts (int each), doubled (byte) per step
        c->lay.slog = c->lay.take((size_t)c->max_steps * 9);
    if (c->pol.time_gradient) {
        c->lay.tprime = c->lay.take(((size_t)c->max_steps + 1) * sizeof(float));
        c->lay.tdots = c->lay.take(((size_t)2 * kDotBlocks + 12) * sizeof(float));
    }
    *out = c;
    return MPODE_OK;
}

void mpode_destroy(mpode_ctx* ctx) {
    if (!ctx) return;
    if (ctx->side) {
        cudaStreamDestroy(ctx->side);
        cudaEventDestroy(ctx->ev_ready); cudaEventDestroy(ctx->ev_vjp); cudaEventDestroy(ctx->ev_rec);
    }
    if (ctx->mirror_host) {
        cudaFreeHost(ctx->mirror_host);
        cudaEventDestroy(ctx->ev_step[0]); cudaEventDestroy(ctx->ev_step[1]);
    }
    delete ctx->v;
    delete ctx;
}

size_t mpode_param_count(const mpode_ctx* ctx) { return ctx ? ctx->v->param_count() : 0; }
size_t mpode_state_width(const mpode_ctx* ctx) { return ctx ? (size_t)ctx->D : 0; }
size_t mpode_workspace_bytes(const mpode_ctx* ctx) { return ctx ? ctx->lay.total : 0; }
size_t mpode_trajectory_bytes(const mpode_ctx* ctx, int n_steps) {
    if (!ctx || n_steps < 0) return 0;
    return (size_t)(n_steps + 1) * ctx->B * ctx->d * low_size(ctx->pol.low);
}
size_t mpode_io_bytes(const mpode_ctx* ctx) {
    if (!ctx) return 0;
    size_t p = ctx->v->param_count();
    size_t r256 = 255;
    size_t theta = (p * 4 + r256) & ~r256, st = ((size_t)ctx->B * ctx->D * 4 + r256) & ~r256;
    size_t probe = ((size_t)ctx->B * ctx->d + r256) & ~r256;
    return theta + 2 * st + probe + theta;   // theta | state in | state out | probe | dtheta
}

void mpode_get_stats(const mpode_ctx* ctx, mpode_stats* out) {
    if (!ctx || !out) return;
    *out = ctx->stats;
    out->tc_contractions = ctx->counters.tc;
    out->simt_contractions = ctx->counters.simt;
    out->fused_launches = ctx->counters.fused;
    out->whole_solve_launches = ctx->counters.whole;
}

void mpode_debug_waits(mpode_ctx* ctx, unsigned long long wait_limit_ns, int starve_forward) {
    if (!ctx) return;
    ctx->dbg_wait_ns = wait_limit_ns;
    ctx->dbg_starve = starve_forward;
}

void mpode_set_profiling(mpode_ctx* ctx, int enabled) {
    if (ctx) ctx->prof.enabled = enabled != 0;
}

mpode_status mpode_collect_profile(mpode_ctx* ctx, double* ms, long long* launches, double* flops) {
    if (!ctx || !ms || !launches || !flops) return MPODE_ERR_INVALID_ARG;
    cudaDeviceSynchronize();
    ctx->prof.collect(ms, launches, flops);
    return check_cuda(ctx, "mpode_collect_profile");
}

mpode_status mpode_forward(mpode_ctx* c, void* cuda_stream, const float* theta_dev, const float* y0_dev,
                           const float* tgrid_host, int n_steps, const mpode_tableau* tab,
                           const signed char* probe_dev, void* traj_dev, float* yT_dev, void* ws, size_t ws_bytes) {
    if (!c) return MPODE_ERR_INVALID_ARG;
    c->have_forward = false;
    if (!theta_dev || !y0_dev || !tgrid_host || !tab || !traj_dev || !yT_dev || !ws)
        return fail(c, MPODE_ERR_INVALID_ARG, "null pointer argument");
    if (n_steps < 1 || n_steps > c->max_steps) return fail(c, MPODE_ERR_INVALID_ARG, "n_steps out of range");
    if (tab->stages < 1 || tab->stages > 4 || !tab->a || !tab->b || !tab->c)
        return fail(c, MPODE_ERR_INVALID_ARG, "tableau must have 1..4 stages");
    for (int j = 0; j < tab->stages; ++j)
        for (int l = j; l < tab->stages; ++l)
            if (tab->a[j * tab->stages + l] != 0.0) return fail(c, MPODE_ERR_INVALID_ARG, "tableau is not explicit");
    for (int i = 0; i < n_steps; ++i)
        if (!(tgrid_host[i + 1] > tgrid_host[i])) return fail(c, MPODE_ERR_INVALID_ARG, "time grid must be strictly increasing");
    if (c->vel.kind == MPODE_VEL_CNF_MLP && !probe_dev) return fail(c, MPODE_ERR_INVALID_ARG, "CNF velocity needs a probe");
    if (ws_bytes < c->lay.total) return fail(c, MPODE_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    if (((uintptr_t)ws & 255) || ((uintptr_t)traj_dev & 15) || ((uintptr_t)yT_dev & 15) || ((uintptr_t)y0_dev & 15) ||
        ((uintptr_t)theta_dev & 15))
        return fail(c, MPODE_ERR_INVALID_ARG, "misaligned device pointer");

    cudaStream_t st = (cudaStream_t)cuda_stream;
    tl_profiler = &c->prof;
    c->stats = mpode_stats{};
    c->counters = PathCounters{};
    tl_counters = &c->counters;
    c->ws_forward = ws;
    c->theta = theta_dev;
    c->probe = probe_dev;
    c->traj = traj_dev;
    c->tgrid.assign(tgrid_host, tgrid_host + n_steps + 1);
    c->n_steps = n_steps;
    c->stages = tab->stages;
    memset(c->ta, 0, sizeof(c->ta));
    for (int j = 0; j < tab->stages; ++j) {
        c->tb[j] = tab->b[j];
        c->tc[j] = tab->c[j];
        for (int l = 0; l < tab->stages; ++l) c->ta[j * tab->stages + l] = tab->a[j * tab->stages + l];
    }
    const mpode_dtype dt = c->pol.low;
    const size_t es = low_size(dt);
    const long long nBd = (long long)c->B * c->d;
    long long* L = &c->stats.kernel_launches;

    cudaMemsetAsync(at(ws, c->lay.scal), 0, 256, st);
    {   // very small velocities: the whole loop in one launch of one CTA
        FusedSolve whole = fused_solve(c, yT_dev);
        if (c->v->whole_forward(st, ws, whole, theta_dev, y0_dev, yT_dev, L)) {
            mpode_status ws_ = check_cuda(c, "mpode_forward");
            if (ws_ != MPODE_OK) return ws_;
            c->have_forward = true;
            return MPODE_OK;
        }
    }
    c->v->prepare(st, ws, theta_dev, probe_dev, L);                                         // Q16(theta)
    launch_init_state(dt, y0_dev, yT_dev, traj_dev, c->B, c->d, c->D, st, L);                // y <- x, traj[0]
    // the whole loop in one persistent launch where the velocity has a fused kernel, else layer by layer
    FusedSolve fs = fused_solve(c, yT_dev);
    c->v->prepare_solve(st, ws, fs, L);
    const bool fused = c->v->fused_forward(st, ws, fs, L);
    for (int i = 0; i < n_steps && !fused; ++i) {
        StepTimes tm = step_times(c, i);
        c->v->set_step(i, n_steps);
        run_stages(c, st, ws, i, tm);
        Terms t{};
        t.n = c->stages;
        for (int j = 0; j < c->stages; ++j) {
            t.p[j] = at(ws, c->lay.kbuf[j]);
            t.c[j] = c->pol.round_increment ? (float)c->tb[j] : (float)((double)tm.h * c->tb[j]);
        }
        char* traj_next = (char*)traj_dev + (size_t)(i + 1) * nBd * es;
        launch_final_combine(dt, yT_dev, t, traj_next, c->B, c->d, c->D, c->pol.round_increment, tm.h, st, L);
        if (c->D > c->d) {
            for (int j = 0; j < c->stages; ++j) t.p[j] = at(ws, c->lay.klbuf[j]);
            launch_column_combine(dt, yT_dev, c->D, c->d, t, c->B, c->pol.round_increment, tm.h, st, L);
        }
    }
    mpode_status s = check_cuda(c, "mpode_forward");
    if (s != MPODE_OK) return s;
    c->have_forward = true;
    return MPODE_OK;
}

mpode_status mpode_backward(mpode_ctx* c, void* cuda_stream, const float* dL_dyT_dev, float* a, float* g,
                            int accumulate_dtheta, mpode_scale_log* log, void* ws, size_t ws_bytes) {
    return mpode_backward_ex(c, cuda_stream, dL_dyT_dev, nullptr, a, g, accumulate_dtheta, nullptr, log, ws, ws_bytes);
}

mpode_status mpode_backward_ex(mpode_ctx* c, void* cuda_stream, const float* dL_dyT_dev, const float* cot, float* a, float* g,
                               int accumulate_dtheta, float* dt_host, mpode_scale_log* log, void* ws, size_t ws_bytes) {
    if (!c) return MPODE_ERR_INVALID_ARG;
    if (!c->have_forward) return fail(c, MPODE_ERR_BAD_STATE, "mpode_backward needs a preceding mpode_forward");
    if (!dL_dyT_dev || !a || !g || !ws) return fail(c, MPODE_ERR_INVALID_ARG, "null pointer argument");
    if (dt_host != nullptr && !c->pol.time_gradient)
        return fail(c, MPODE_ERR_INVALID_ARG, "dL/dt needs a context created with policy.time_gradient = 1");
    if (cot != nullptr && ((uintptr_t)cot & 15)) return fail(c, MPODE_ERR_INVALID_ARG, "misaligned device pointer");
    if (ws_bytes < c->lay.total) return fail(c, MPODE_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    if (((uintptr_t)ws & 255) || ((uintptr_t)a & 15) || ((uintptr_t)g & 15) || ((uintptr_t)dL_dyT_dev & 15))
        return fail(c, MPODE_ERR_INVALID_ARG, "misaligned device pointer");
    const int N = c->n_steps, s = c->stages;
    if (log) {
        if (log->n_steps < N || !log->exp_used || !log->attempts || !log->doubled)
            return fail(c, MPODE_ERR_INVALID_ARG, "scale log arrays too small");
        log->first_failed_step = -1;
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    tl_profiler = &c->prof;
    tl_counters = &c->counters;
    const mpode_dtype dt = c->pol.low;
    const size_t es = low_size(dt);
    const long long nBd = (long long)c->B * c->d;
    const long long p = (long long)c->v->param_count();
    const bool dynamic = c->pol.scaling == MPODE_SCALE_DYNAMIC;
    const bool checked = c->pol.scaling != MPODE_SCALE_NONE;
    long long launches0 = c->stats.kernel_launches;
    long long* L = &c->stats.kernel_launches;
    c->stats.retries = 0;
    c->stats.host_syncs = 0;
    c->stats.step_waits = 0;

    {   // very small velocities: Alg. 2 with its scale decisions in one launch of one CTA
        WholeBackward wb;
        wb.theta = c->theta; wb.dLdyT = dL_dyT_dev; wb.a = a; wb.g = g; wb.accumulate = accumulate_dtheta;
        wb.scaling = (int)c->pol.scaling; wb.k_max = c->pol.k_max; wb.growth_rule = c->pol.growth_rule; wb.pbits = precision_bits(dt);
        wb.e0 = 0; wb.e0_from_norm = dynamic ? 1 : 0;
        if (c->pol.init_scale_exp_override != MPODE_NO_OVERRIDE) {
            int eo = c->pol.init_scale_exp_override;
            wb.e0 = eo < kExpMin ? kExpMin : (eo > kExpMax ? kExpMax : eo);
            wb.e0_from_norm = 0;
        }
        if (log) { wb.exp_used = log->exp_used; wb.attempts = log->attempts; wb.doubled = log->doubled; }
        wb.cot = cot; wb.dt_host = dt_host;
        FusedSolve whole = fused_solve(c, nullptr);
        if (c->v->whole_backward(st, ws, whole, wb, L)) {
            ++c->stats.host_syncs;
            c->stats.retries = wb.retries;
            mpode_status cs = check_cuda(c, "mpode_backward");
            if (cs != MPODE_OK) return cs;
            if (wb.status == MPODE_ERR_NONFINITE_INPUT) return fail(c, MPODE_ERR_NONFINITE_INPUT, "dL/dy_T is not finite");
            if (wb.status == MPODE_ERR_SCALE_FAILED) {
                if (log) log->first_failed_step = wb.first_failed_step;
                return fail(c, MPODE_ERR_SCALE_FAILED, "dynamic adjoint scaling failed at step " + std::to_string(wb.first_failed_step));
            }
            if (wb.status == MPODE_WARN_NONFINITE_GRAD) { c->err = "overflow in the unscaled backward pass"; return MPODE_WARN_NONFINITE_GRAD; }
            return MPODE_OK;
        }
    }
    unsigned* flag = (unsigned*)at(ws, c->lay.scal);
    float* amax = (float*)at(ws, c->lay.scal) + 1;
    unsigned* vjp_flag = checked ? flag : nullptr;
    float* dg = (float*)at(ws, c->lay.dg);
    // time-grid gradient: t' and its scratch (partial sums of Phi^T a, of the <psi_j, k_l> terms, dtau_j, c_j, {Phi^T a, dt, dh})
    const bool tg = dt_host != nullptr;
    float* tprime = tg ? (float*)at(ws, c->lay.tprime) : nullptr;
    float* part_phi = tg ? (float*)at(ws, c->lay.tdots) : nullptr;
    float* part_dh = tg ? part_phi + kDotBlocks : nullptr;
    float* dtau = tg ? part_phi + 2 * kDotBlocks : nullptr;
    float* cvec = tg ? dtau + 4 : nullptr;
    float* tvals = tg ? dtau + 8 : nullptr;
    if (tg) {
        cudaMemsetAsync(tprime, 0, ((size_t)N + 1) * sizeof(float), st);
        for (int j = 0; j < 4; ++j) c->tc_f[j] = j < s ? (float)c->tc[j] : 0.f;
        cudaMemcpyAsync(cvec, c->tc_f, 4 * sizeof(float), cudaMemcpyHostToDevice, st);
    }
    struct { unsigned flag; float amax; } hs;
    // dynamic scaling: log2 S, the first failed step and the bad-input mark live on the device (words 8..10 of the scalar slice);
    // the seed and the updates read the exponent there, one-thread kernels take Alg. 2's decisions, and the host reads the state
    // once, after the last step (again after every retry)
    int* sstate = (int*)at(ws, c->lay.scal) + 8;
    int* slog_exp = dynamic ? (int*)at(ws, c->lay.slog) : nullptr;
    int* slog_att = dynamic ? slog_exp + c->max_steps : nullptr;
    unsigned char* slog_dbl = dynamic ? (unsigned char*)(slog_att + c->max_steps) : nullptr;
    const int* e_dev = dynamic ? sstate : nullptr;
    if (dynamic && c->mirror_host == nullptr && c->allow_side) {        // first dynamic pass through an entry point that may allocate
        void* mh = nullptr;
        if (cudaHostAlloc(&mh, 64, cudaHostAllocMapped) == cudaSuccess) {
            void* md = nullptr;
            if (cudaHostGetDevicePointer(&md, mh, 0) == cudaSuccess &&
                cudaEventCreateWithFlags(&c->ev_step[0], cudaEventDisableTiming) == cudaSuccess &&
                cudaEventCreateWithFlags(&c->ev_step[1], cudaEventDisableTiming) == cudaSuccess) {
                c->mirror_host = (int*)mh; c->mirror_dev = (int*)md;
            } else {
                if (c->ev_step[0]) { cudaEventDestroy(c->ev_step[0]); c->ev_step[0] = nullptr; }
                cudaFreeHost(mh);
            }
        }
        cudaGetLastError();
    }
    const bool paced = dynamic && c->mirror_host != nullptr;
    int* mirror = paced ? c->mirror_dev : sstate + 4;                   // without the mapped copy the kernels mirror into spare words
    volatile int* mirror_h = c->mirror_host;

    // Alg. 2 initialisation: a <- dL/dy_N, g <- 0 (or the caller's partial), then the initial scale
    if (ws != c->ws_forward) cudaMemsetAsync(at(ws, c->lay.scal), 0, 256, st);     // a workspace no forward pass has prepared
    cudaMemsetAsync(flag, 0, 8, st);
    launch_copy_amax(dL_dyT_dev, a, (long long)c->B * c->D, amax, flag, st, L);
    if (!accumulate_dtheta) launch_fill(g, 0.f, p, st, L);
    int e = 0;
    if (c->pol.init_scale_exp_override != MPODE_NO_OVERRIDE) {
        e = c->pol.init_scale_exp_override;
        e = e < kExpMin ? kExpMin : (e > kExpMax ? kExpMax : e);
    }
    if (dynamic) {
        if (paced) { mirror_h[1] = -1; mirror_h[2] = 0; }
        launch_scale_init(flag, amax, precision_bits(dt), e, c->pol.init_scale_exp_override == MPODE_NO_OVERRIDE ? 1 : 0, kExpMin, kExpMax,
                          sstate, mirror, st, L);
    }
    c->v->prepare(st, ws, c->theta, c->probe, L);                                            // weights in low precision
    // fused kernels (one recompute launch per step, one VJP launch per attempt) where the velocity has them
    FusedSolve fs = fused_solve(c, nullptr);
    c->v->prepare_solve(st, ws, fs, L);
    const bool fused = c->v->fused_backward_begin(st, ws, fs, L);
    // Without finiteness decisions nothing of step i - 1's recompute depends on step i's adjoint.  The two fused launches of
    // every step then follow each other on the caller's stream (recompute of step i - 1 right behind the VJP launch of
    // step i, whose layer outputs it overwrites), and the small kernels between them (gradient finish, adjoint commit,
    // next seed) run beside the recompute on a second stream.
    bool overlap = fused && !checked && c->allow_side && !tg;
    if (overlap && c->side == nullptr) {
        if (cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_ready, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_vjp, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_rec, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            c->side = nullptr;
            overlap = false;
        }
    }
    cudaStream_t sr = st;                       // stream of the seed, the reductions and the commits
    if (overlap) {
        cudaEventRecord(c->ev_ready, st);
        cudaStreamWaitEvent(c->side, c->ev_ready, 0);
        sr = c->side;
        c->v->fused_recompute(st, ws, fs, N - 1, L);
    }

    int start = N - 1;                          // first step of this round of queueing (dynamic scaling: the step to repeat)
    int fail_step = -1, fail_count = 0;         // the step that failed last and how many of its attempts did
    int recomputed = -1;                        // the step whose stages the workspace holds
    int hstate[3] = {0, -1, 0};
    unsigned dev_err = 0, fwd_err = 0;          // a tensor-core kernel whose bounded wait gave up reports it in the third scalar word
    // the stages of step i again (Alg. 2, recompute), and what else depends on them but not on the attempt
    auto queue_recompute = [&](int i) {
        StepTimes tm = step_times(c, i);
        c->v->set_step(i, N);
        recomputed = i;
        if (overlap) { /* queued on the second stream */ }
        else if (fused) c->v->fused_recompute(st, ws, fs, i, L);
        else run_stages(c, st, ws, i, tm);
        if (tg) {      // Phi^T a_{i+1} with Phi = sum_j b_j k_j from the recomputed stages and the adjoint before its update
            DotPairs pr{};
            pr.n = s;
            for (int j = 0; j < s; ++j) {
                pr.x[j] = at(ws, c->lay.kbuf[j]); pr.ldx[j] = c->d; pr.y[j] = a; pr.y_f32[j] = 1; pr.ldy[j] = c->D; pr.coef[j] = (float)c->tb[j];
            }
            launch_dot_partial(dt, pr, c->B, c->d, part_phi, st, L);
        }
    };
    for (;;) {
    for (int i = start; i >= 0; --i) {
        if (recomputed != i) queue_recompute(i);     // a repeated attempt finds its step's stages still in place
        StepTimes tm = step_times(c, i);
        c->v->set_step(i, N);
        const char* traj_i = (const char*)c->traj + (size_t)i * nBd * es;
        {
            if (tg) cudaMemsetAsync(dtau, 0, 4 * sizeof(float), st);
            // velocities that write kappa_{j-1} from their own epilogues (state without extra columns) get kappa_s from the seed
            const bool kappa_in_vjp = !fused && c->D == c->d && c->v->can_write_next_kappa();
            const bool seeded_kappa = kappa_in_vjp;
            launch_seed(dt, a, e, at(ws, c->lay.v), c->D > c->d ? at(ws, c->lay.vl) : nullptr, c->B, c->d, c->D,
                        vjp_flag, sr, L, fused ? c->v->fused_kappa_last(ws) : (seeded_kappa ? at(ws, c->v->kappa_offset(c->lay)) : nullptr),
                        (float)c->tb[s - 1], e_dev);                                             // seed Q16(S a)
            // without a finiteness decision the step gradient goes straight into g <- g + (h / S) dg
            if (overlap) {
                cudaEventRecord(c->ev_rec, sr);                    // the seed of this step is ready
                cudaStreamWaitEvent(st, c->ev_rec, 0);
                c->v->fused_vjp(st, ws, fs, i, g, 1.f, (float)((double)tm.h * ldexp(1.0, -e)), vjp_flag, L, c->ev_vjp, sr);
                if (i > 0) c->v->fused_recompute(st, ws, fs, i - 1, L);
            } else if (fused && !checked) c->v->fused_vjp(st, ws, fs, i, g, 1.f, (float)((double)tm.h * ldexp(1.0, -e)), vjp_flag, L);
            else if (fused) c->v->fused_vjp(st, ws, fs, i, dg, 0.f, 1.f, vjp_flag, L);
            bool kappa_ready = seeded_kappa;          // stage s - 1: kappa = Q16(b_s v), written by the seed kernel
            const bool by_step = !fused && !tg && !c->v->needs_input_copy() &&
                                 c->v->step_vjp(st, ws, traj_i, step_scalars(c, i), s, dg, vjp_flag, L);
            for (int j = s - 1; j >= 0 && !fused && !by_step; --j) {
                Terms t{};
                t.n = 0;
                for (int l = j + 1; l < s; ++l) {
                    double alj = c->ta[l * s + j];
                    if (alj != 0.0) {
                        t.p[t.n] = at(ws, c->lay.psi[l]);
                        t.c[t.n] = (float)((double)tm.h * alj);
                        ++t.n;
                    }
                }
                void* kappa = at(ws, c->v->kappa_offset(c->lay));
                if (!kappa_ready) launch_kappa(dt, at(ws, c->lay.v), (float)c->tb[j], t, kappa, nBd, vjp_flag, st, L);
                // can this stage's vector-Jacobian product also write kappa_{j-1}?  Yes when the tableau couples stage j - 1 to
                // stage j alone (a_lj = 0 for l > j: Euler, midpoint, RK4, ...)
                kappa_ready = false;
                if (j > 0 && kappa_in_vjp) {
                    int terms = 0;
                    for (int l = j; l < s; ++l) terms += c->ta[l * s + (j - 1)] != 0.0 ? 1 : 0;
                    if (terms == 1 && c->ta[j * s + (j - 1)] != 0.0) {
                        KappaNext kn;
                        kn.out = kappa; kn.v = at(ws, c->lay.v); kn.bv = (float)c->tb[j - 1]; kn.c = (float)((double)tm.h * c->ta[j * s + (j - 1)]);
                        c->v->set_next_kappa(kn);
                        kappa_ready = true;
                    }
                }
                if (c->D > c->d) {
                    Terms none{};
                    launch_kappa(dt, at(ws, c->lay.vl), (float)c->tb[j], none, at(ws, c->lay.kappal), c->B, vjp_flag, st, L);
                }
                const void* yin = (j > 0 || c->v->needs_input_copy()) ? (const void*)at(ws, c->lay.ybuf[j]) : (const void*)traj_i;
                c->v->vjp(st, ws, j, yin, tm.tau16[j], at(ws, c->lay.psi[j]), dg, j == s - 1 ? 0.f : 1.f, vjp_flag, L);
            }
            if (tg) {      // dt = sum_j dtau_j, dh = sum_j (c_j dtau_j + sum_{l<j} a_jl <psi_j, k_l>); Q16(dt), Q16(dh) join the test
                DotPairs pr{};
                for (int j = 1; j < s; ++j)
                    for (int l = 0; l < j; ++l)
                        if (c->ta[j * s + l] != 0.0 && pr.n < 8) {
                            const int q = pr.n++;
                            pr.x[q] = at(ws, c->lay.psi[j]); pr.ldx[q] = c->d; pr.y[q] = at(ws, c->lay.kbuf[l]); pr.y_f32[q] = 0; pr.ldy[q] = c->d;
                            pr.coef[q] = (float)c->ta[j * s + l];
                        }
                launch_dot_partial(dt, pr, c->B, c->d, part_dh, st, L);
                launch_tgrad_reduce(dt, part_phi, part_dh, dtau, cvec, s, tvals, vjp_flag, st, L);
            }
            if (checked) launch_check_as_low(dt, dg, p, flag, st, L);                        // finiteness of dg
        }
        // high-precision updates of a and g with h / S (exact in fp32: a power-of-two scaling of h)
        Terms ps{};
        ps.n = s;
        for (int j = 0; j < s; ++j) { ps.p[j] = at(ws, c->lay.psi[s - 1 - j]); ps.c[j] = 1.f; }
        const float* cot_i = cot ? cot + (size_t)i * c->B * c->D : nullptr;
        if (dynamic) {
            // queued at once: they skip themselves while the flag is raised, take 2^-e from the device, and the decision kernel
            // behind them records the attempt (growth test on the new ||a||_inf) or the failure
            cudaMemsetAsync(amax, 0, 4, st);
            if (tg) launch_tgrad_update(tprime, i, tvals, tm.h, flag, st, L, e_dev);        // before a changes: it holds Phi^T a_{i+1} already
            launch_commit_a(dt, a, ps, tm.h, c->B, c->d, c->D, amax, st, L, flag, cot_i, e_dev);
            launch_commit_g(g, dg, tm.h, p, st, L, flag, e_dev);
            launch_scale_decide(flag, amax, sstate, mirror, i, i == fail_step ? fail_count + 1 : 1, c->pol.growth_rule, precision_bits(dt),
                                kExpMin, kExpMax, slog_exp, slog_att, slog_dbl, st, L);
            if (paced) cudaEventRecord(c->ev_step[i & 1], st);
            // The host learns the outcome of step i before it queues the attempt of step i - 1.  Meanwhile the device has the
            // recompute of step i - 1 to work on (it does not depend on the outcome), so the stream does not run dry; after an
            // overflow that recompute and the one of step i are what is queued again.  A step that is being repeated gets no
            // such work ahead: overflows come in runs at one step (the first, above all), and a repeat then costs one attempt.
            const bool repeat = i == start && i == fail_step;
            if (i > 0 && paced && !repeat) queue_recompute(i - 1);
            if (i > 0 || !paced) {
                bool failed;
                if (paced) {
                    cudaEventSynchronize(c->ev_step[i & 1]);
                    ++c->stats.step_waits;
                    failed = mirror_h[1] >= 0 || mirror_h[2] != 0;
                } else {
                    cudaMemcpyAsync(hstate, sstate, sizeof hstate, cudaMemcpyDeviceToHost, st);
                    cudaStreamSynchronize(st);
                    ++c->stats.host_syncs;
                    failed = hstate[1] >= 0 || hstate[2] != 0;
                }
                if (failed) break;
            }
        } else {
            float coef = (float)((double)tm.h * ldexp(1.0, -e));
            if (tg) launch_tgrad_update(tprime, i, tvals, coef, nullptr, st, L);
            launch_commit_a(dt, a, ps, coef, c->B, c->d, c->D, nullptr, sr, L, nullptr, cot_i);
            if (!(fused && !checked)) launch_commit_g(g, dg, coef, p, st, L);
            if (log) { log->attempts[i] = 1; log->exp_used[i] = e; log->doubled[i] = 0; }
        }
    }
    if (!dynamic) break;
    // one drain per round: the state and, should this have been the last round, everything else the host reads
    cudaMemcpyAsync(hstate, sstate, sizeof hstate, cudaMemcpyDeviceToHost, st);
    if (log) {
        cudaMemcpyAsync(log->exp_used, slog_exp, (size_t)N * sizeof(int), cudaMemcpyDeviceToHost, st);
        cudaMemcpyAsync(log->attempts, slog_att, (size_t)N * sizeof(int), cudaMemcpyDeviceToHost, st);
        cudaMemcpyAsync(log->doubled, slog_dbl, (size_t)N, cudaMemcpyDeviceToHost, st);
    }
    if (tg) cudaMemcpyAsync(dt_host, tprime, ((size_t)N + 1) * sizeof(float), cudaMemcpyDeviceToHost, st);
    cudaMemcpyAsync(&dev_err, flag + 2, 4, cudaMemcpyDeviceToHost, st);
    if (c->ws_forward != nullptr && c->ws_forward != ws)     // the forward pass ran on another workspace: its error word lives there
        cudaMemcpyAsync(&fwd_err, (unsigned*)at(c->ws_forward, c->lay.scal) + 2, 4, cudaMemcpyDeviceToHost, st);
    cudaStreamSynchronize(st);
    ++c->stats.host_syncs;
    {
        mpode_status cs = check_cuda(c, "mpode_backward");
        if (cs != MPODE_OK) return cs;
    }
    dev_err |= fwd_err;
    if (dev_err != 0u) return fail(c, MPODE_ERR_CUDA, "a device-side wait timed out (code " + std::to_string(dev_err) + ")");
    if (hstate[2] != 0) return fail(c, MPODE_ERR_NONFINITE_INPUT, "dL/dy_T is not finite");
    if (hstate[1] < 0) return MPODE_OK;         // every step accepted
    // the attempt at step hstate[1] was not finite: the device has halved S and committed nothing since
    if (hstate[1] == fail_step) ++fail_count; else { fail_step = hstate[1]; fail_count = 1; }
    ++c->stats.retries;
    if (fail_count >= c->pol.k_max) {
        if (log) {
            cudaMemcpy(log->exp_used + fail_step + 1, slog_exp + fail_step + 1, (size_t)(N - 1 - fail_step) * sizeof(int), cudaMemcpyDeviceToHost);
            cudaMemcpy(log->attempts + fail_step + 1, slog_att + fail_step + 1, (size_t)(N - 1 - fail_step) * sizeof(int), cudaMemcpyDeviceToHost);
            cudaMemcpy(log->doubled + fail_step + 1, slog_dbl + fail_step + 1, (size_t)(N - 1 - fail_step), cudaMemcpyDeviceToHost);
            log->attempts[fail_step] = fail_count; log->exp_used[fail_step] = hstate[0]; log->doubled[fail_step] = 0;
            log->first_failed_step = fail_step;
        }
        return fail(c, MPODE_ERR_SCALE_FAILED, "dynamic adjoint scaling failed at step " + std::to_string(fail_step));
    }
    cudaMemsetAsync(flag, 0, 4, st);
    cudaMemsetAsync(sstate + 1, 0xff, 4, st);   // no failed step
    if (paced) mirror_h[1] = -1;
    start = fail_step;
    }
    if (overlap) {      // the caller's stream continues only after the last commit on the second stream
        cudaEventRecord(c->ev_ready, sr);
        cudaStreamWaitEvent(st, c->ev_ready, 0);
    }
    mpode_status rs = MPODE_OK;
    if (c->pol.scaling == MPODE_SCALE_NONE_SAFE) {
        cudaMemcpyAsync(&hs, flag, 8, cudaMemcpyDeviceToHost, st);
        cudaStreamSynchronize(st);
        ++c->stats.host_syncs;
        if (hs.flag != 0u) {                     // Sec. 5: report the overflow through infinite gradients
            launch_fill(a, INFINITY, (long long)c->B * c->D, st, L);
            launch_fill(g, INFINITY, p, st, L);
            if (tg) launch_fill(tprime, INFINITY, (long long)N + 1, st, L);
            rs = MPODE_WARN_NONFINITE_GRAD;
            c->err = "overflow in the unscaled backward pass";
        }
    }
    (void)launches0;
    if (tg) cudaMemcpyAsync(dt_host, tprime, ((size_t)N + 1) * sizeof(float), cudaMemcpyDeviceToHost, st);
    cudaMemcpyAsync(&dev_err, flag + 2, 4, cudaMemcpyDeviceToHost, st);
    if (c->ws_forward != nullptr && c->ws_forward != ws)     // the forward pass ran on another workspace: its error word lives there
        cudaMemcpyAsync(&fwd_err, (unsigned*)at(c->ws_forward, c->lay.scal) + 2, 4, cudaMemcpyDeviceToHost, st);
    cudaStreamSynchronize(st);
    ++c->stats.host_syncs;
    mpode_status cs = check_cuda(c, "mpode_backward");
    if (cs != MPODE_OK) return cs;
    dev_err |= fwd_err;
    if (dev_err != 0u) return fail(c, MPODE_ERR_CUDA, "a device-side wait timed out (code " + std::to_string(dev_err) + ")");
    return rs;
}

mpode_status mpode_forward_host(mpode_ctx* c, void* cuda_stream, const float* theta_host, const float* y0_host,
                                const float* tgrid_host, int n_steps, const mpode_tableau* tab,
                                const signed char* probe_host, void* traj_dev, float* yT_host, void* io_dev, void* ws,
                                size_t ws_bytes) {
    if (!c || !theta_host || !y0_host || !yT_host || !io_dev) return MPODE_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    size_t p = c->v->param_count(), r = 255;
    size_t theta_b = (p * 4 + r) & ~r, st_b = ((size_t)c->B * c->D * 4 + r) & ~r;
    float* theta_dev = (float*)io_dev;
    float* sin_dev = (float*)((char*)io_dev + theta_b);
    float* sout_dev = (float*)((char*)io_dev + theta_b + st_b);
    signed char* probe_dev = (signed char*)((char*)io_dev + theta_b + 2 * st_b);
    cudaMemcpyAsync(theta_dev, theta_host, p * 4, cudaMemcpyHostToDevice, st);
    cudaMemcpyAsync(sin_dev, y0_host, (size_t)c->B * c->d * 4, cudaMemcpyHostToDevice, st);
    if (probe_host) cudaMemcpyAsync(probe_dev, probe_host, (size_t)c->B * c->d, cudaMemcpyHostToDevice, st);
    mpode_status s = mpode_forward(c, st, theta_dev, sin_dev, tgrid_host, n_steps, tab, probe_host ? probe_dev : nullptr,
                                   traj_dev, sout_dev, ws, ws_bytes);
    if (s != MPODE_OK) return s;
    cudaMemcpyAsync(yT_host, sout_dev, (size_t)c->B * c->D * 4, cudaMemcpyDeviceToHost, st);
    unsigned dev_err = 0;
    cudaMemcpyAsync(&dev_err, (unsigned*)at(ws, c->lay.scal) + 2, 4, cudaMemcpyDeviceToHost, st);
    cudaStreamSynchronize(st);
    mpode_status cs = check_cuda(c, "mpode_forward_host");
    if (cs != MPODE_OK) return cs;
    if (dev_err != 0u) {
        c->have_forward = false;
        return fail(c, MPODE_ERR_CUDA, "a device-side wait timed out (code " + std::to_string(dev_err) + ")");
    }
    return MPODE_OK;
}

mpode_status mpode_backward_host(mpode_ctx* c, void* cuda_stream, const float* dL_dyT_host, float* dL_dy0_host,
                                 float* dL_dtheta_host, mpode_scale_log* log, void* io_dev, void* ws, size_t ws_bytes) {
    if (!c || !dL_dyT_host || !dL_dy0_host || !dL_dtheta_host || !io_dev) return MPODE_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    size_t p = c->v->param_count(), r = 255;
    size_t theta_b = (p * 4 + r) & ~r, st_b = ((size_t)c->B * c->D * 4 + r) & ~r;
    size_t probe_b = ((size_t)c->B * c->d + r) & ~r;
    float* sin_dev = (float*)((char*)io_dev + theta_b);
    float* sout_dev = (float*)((char*)io_dev + theta_b + st_b);
    float* g_dev = (float*)((char*)io_dev + theta_b + 2 * st_b + probe_b);
    cudaMemcpyAsync(sin_dev, dL_dyT_host, (size_t)c->B * c->D * 4, cudaMemcpyHostToDevice, st);
    mpode_status s = mpode_backward(c, st, sin_dev, sout_dev, g_dev, 0, log, ws, ws_bytes);
    if (s != MPODE_OK && s != MPODE_WARN_NONFINITE_GRAD) return s;
    cudaMemcpyAsync(dL_dy0_host, sout_dev, (size_t)c->B * c->D * 4, cudaMemcpyDeviceToHost, st);
    cudaMemcpyAsync(dL_dtheta_host, g_dev, p * 4, cudaMemcpyDeviceToHost, st);
    cudaStreamSynchronize(st);
    mpode_status cs = check_cuda(c, "mpode_backward_host");
    return cs != MPODE_OK ? cs : s;
}

// ---------------------------------------------------------------------------------------------------------------
// Backward pass on a workspace that is part of the library image (see mpode.h): for callers that cannot allocate.
// In host code `g_static_workspace` is only a handle for the runtime, never a device address: the address a kernel can
// use comes from cudaGetSymbolAddress, looked up once per device with that device current.
static __device__ __align__(256) unsigned char g_static_workspace[MPODE_STATIC_WORKSPACE_BYTES];

namespace {
void* g_static_ws_ptr[kMaxDevices] = {nullptr};
std::mutex g_static_ws_mu;

mpode_status static_workspace_address(mpode_ctx* c, int dev, void** out) {
    std::lock_guard<std::mutex> lock(g_static_ws_mu);
    if (g_static_ws_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_workspace);
        if (e != cudaSuccess || ptr == nullptr)
            return fail(c, MPODE_ERR_CUDA, std::string("cudaGetSymbolAddress(static workspace): ") + cudaGetErrorString(e));
        g_static_ws_ptr[dev] = ptr;
    }
    *out = g_static_ws_ptr[dev];
    return MPODE_OK;
}
}  // namespace

mpode_status mpode_backward_static_workspace(mpode_ctx* c, void* cuda_stream, const float* dL_dyT_dev, float* dL_dy0_dev,
                                             float* dL_dtheta_dev, int accumulate_dtheta, mpode_scale_log* log) {
    if (!c) return MPODE_ERR_INVALID_ARG;
    if (c->lay.total > (size_t)MPODE_STATIC_WORKSPACE_BYTES)
        return fail(c, MPODE_ERR_WORKSPACE_TOO_SMALL,
                    "this context needs " + std::to_string(c->lay.total) + " bytes of workspace, the static workspace holds " +
                        std::to_string((size_t)MPODE_STATIC_WORKSPACE_BYTES));
    // everything mpode_backward would refuse is refused here first, so that an invalid call queues nothing on the stream
    if (!c->have_forward) return fail(c, MPODE_ERR_BAD_STATE, "mpode_backward needs a preceding mpode_forward");
    if (!dL_dyT_dev || !dL_dy0_dev || !dL_dtheta_dev) return fail(c, MPODE_ERR_INVALID_ARG, "null pointer argument");
    if (((uintptr_t)dL_dy0_dev & 15) || ((uintptr_t)dL_dtheta_dev & 15) || ((uintptr_t)dL_dyT_dev & 15))
        return fail(c, MPODE_ERR_INVALID_ARG, "misaligned device pointer");
    if (log && (log->n_steps < c->n_steps || !log->exp_used || !log->attempts || !log->doubled))
        return fail(c, MPODE_ERR_INVALID_ARG, "scale log arrays too small");
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return fail(c, MPODE_ERR_CUDA, "mpode_backward_static_workspace: no current CUDA device");
    cudaPointerAttributes pa{};
    if (cudaPointerGetAttributes(&pa, dL_dyT_dev) != cudaSuccess || pa.type != cudaMemoryTypeDevice || pa.device != dev) {
        cudaGetLastError();
        return fail(c, MPODE_ERR_INVALID_ARG, "dL_dyT_dev is not memory of the current device: the static workspace of another device would be used");
    }
    void* ws = nullptr;
    mpode_status s = static_workspace_address(c, dev, &ws);
    if (s != MPODE_OK) return s;
    // the array keeps the previous call's contents: the scalar words (non-finite flag, norm, device error word) must
    // start at zero; every other slice is written by the backward pass before it is read
    cudaMemsetAsync((char*)ws + c->lay.scal, 0, 256, (cudaStream_t)cuda_stream);
    c->allow_side = false;      // no second stream here: creating one may allocate
    s = mpode_backward(c, cuda_stream, dL_dyT_dev, dL_dy0_dev, dL_dtheta_dev, accumulate_dtheta, log, ws, c->lay.total);
    c->allow_side = true;
    return s;
}

}  // extern "C"
