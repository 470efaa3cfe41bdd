/*
 * mpode.h - C ABI of the mixed-precision neural-ODE time-stepping library (one NVIDIA B200, sm_100a).
 *
 * The library implements the forward pass of Alg. 1 ("Mixed Precision Forward Pass") and the backward pass
 * of Alg. 2 ("Mixed Precision Backward Pass with Dynamic Adjoint Scaling") of "Mixed Precision Training of
 * Neural ODEs" for explicit Runge-Kutta increment functions (Sec. 3) and a small set of built-in velocity
 * networks f(t, y; theta).
 *
 * Conventions
 *   - extern "C", plain pointers and sizes.  No exception crosses the boundary; every call returns a status.
 *   - "_dev" pointers are CUDA device pointers, "_host" pointers are host pointers.  The caller owns every
 *     device buffer (state, trajectory, gradients, workspace) and the stream; the library owns only the
 *     host-side context, which remembers the pointers given to mpode_forward for the following mpode_backward.
 *   - Batched row-major layout: a state is [B, D] (D = d, or d + 1 for the CNF velocity whose last column is
 *     the log-density l), the stored trajectory is [(N + 1), B, d] in the low format.
 *   - "low" is the 16-bit format of Sec. 2 (float16 or bfloat16; float32 makes every Q16 the identity),
 *     "high" is float32.  All rounding is round-to-nearest-even.
 *   - The device never traps: numerical failures are reported as status codes.
 *   - Dense velocities in the 16-bit formats run as persistent kernels with one thread block per SM whose blocks hand tiles
 *     to each other through counters in the workspace.  They expect the GPU to themselves for the duration of a call: if
 *     other work keeps some SMs occupied for seconds, a block's bounded wait (2 s) gives up and the call returns
 *     MPODE_ERR_CUDA with "a device-side wait timed out" instead of hanging.  mpode_backward may use a second, internal
 *     stream for part of its work; everything is joined to `cuda_stream` before the call returns.
 *   - These kernels move 32-byte pieces of trajectory rows: with a trajectory pointer that is only 16-byte aligned the
 *     library silently takes its layer-by-layer path.
 */
#ifndef MPODE_H_
#define MPODE_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mpode_ctx mpode_ctx; /* opaque, host side */

typedef enum {
    MPODE_OK = 0,
    MPODE_ERR_INVALID_ARG = 1,
    MPODE_ERR_UNSUPPORTED = 2,
    MPODE_ERR_WORKSPACE_TOO_SMALL = 3,
    MPODE_ERR_CUDA = 4,
    MPODE_ERR_BAD_STATE = 5,        /* mpode_backward without a preceding mpode_forward */
    MPODE_ERR_NONFINITE_INPUT = 6,  /* NaN/Inf in dL/dy_T when the scale is initialised (Alg. 2, scale initialisation) */
    MPODE_ERR_SCALE_FAILED = 7,     /* Alg. 2, failure branch: no finite VJP within k_max attempts */
    MPODE_WARN_NONFINITE_GRAD = 8   /* NONE_SAFE scaling: overflow seen, gradients returned as +Inf (Sec. 5) */
} mpode_status;

typedef enum { MPODE_F32 = 0, MPODE_BF16 = 1, MPODE_F16 = 2 } mpode_dtype;

/* Sec. 5: the three backward variants (unscaled, unscaled-safe, dynamic adjoint scaling). */
typedef enum { MPODE_SCALE_NONE = 0, MPODE_SCALE_NONE_SAFE = 1, MPODE_SCALE_DYNAMIC = 2 } mpode_scaling;

typedef enum { MPODE_ACT_NONE = 0, MPODE_ACT_TANH = 1, MPODE_ACT_SOFTPLUS = 2, MPODE_ACT_RELU = 3 } mpode_act;

typedef enum {
    MPODE_VEL_MLP = 0,       /* f = W_L act(... act(W_1 [y; t] + b_1) ...) + b_L ; one bias-free layer = linear ODE */
    MPODE_VEL_CONV3X3_2 = 1, /* f = conv3x3(act(conv3x3([y; t]) + b1)) + b2 on an NHWC image, stride 1, zero pad 1 (the stand-in for
                                the convolutional ODE blocks of Sec. 6.3 uses act = ReLU) */
    MPODE_VEL_CNF_MLP = 2,   /* joint CNF state [z; l] (Sec. 6.1): z' = MLP([z; t]), l' = -eps^T (dz'/dz) eps */
    MPODE_VEL_PARABOLIC_CONV = 4, /* the parabolic convolutional layer of Sec. 6.3, Eq. (NODE_STL10): f = -W(t)^T N(relu(W(t) y + b(t))) on
                                an NHWC image with C channels, W a 3x3 convolution (stride 1, zero pad 1) and W^T its transpose with
                                the same weights, N the instance normalisation (per image and channel over the pixels, biased
                                variance, eps 1e-5, no affine part; instance_norm = 0 leaves it out), weights piecewise constant in
                                time: step i of an n-step solve uses piece i * n_intervals / n (integer division) */
    MPODE_VEL_SCALAR_POLY = 3, /* the scalar test problem of Example 1 (Sec. 3): f = -(theta_1 t^2 + theta_2 t + theta_3) y, d = 1,
                                 theta = (theta_1, theta_2, theta_3); every arithmetic operation of f and of its
                                 vector-Jacobian product is rounded to the low format; batch <= 1024 */
    MPODE_VEL_CNF_HYPER = 5   /* the two-dimensional flows of Sec. 6.1 with the trace written out: joint state [z; l],
                                 z' = (1/w) sum_j U_j(t) tanh(W_j(t) . z + b_j(t)), l' = -(1/w) sum_j (U_j . W_j)(1 - tanh^2(.)); the w weight
                                 sets come from t through three fully connected layers of hidden width h with tanh between them
                                 (the paper fixes the formula of z' and the width; the rest is this library's reading).  d <= 8 */
} mpode_vel_kind;

/*
 * Velocity description.  Parameter vector theta (fp32, flat):
 *   MLP / CNF_MLP : for layer l = 0..n_layers-1: W_l [widths[l+1], widths[l] (+1 time column when l == 0 and
 *                   append_time)] row-major, then b_l [widths[l+1]] when has_bias.  widths has n_layers + 1
 *                   entries, widths[0] == widths[n_layers] == d.  The activation follows every layer but the last.
 *   CONV3X3_2     : W1 [C][3][3][C+1] (last input channel = time), b1 [C], W2 [C][3][3][C], b2 [C]; d = H*W*C.
 *   PARABOLIC_CONV: for each of the n_intervals pieces W_i [C][3][3][C], then b_i [C]; d = H*W*C.
 *   SCALAR_POLY   : theta_1, theta_2, theta_3.
 *   CNF_HYPER     : n_layers = 1, widths = {h, w}: A1 [h][1], c1 [h], A2 [h][h], c2 [h], A3 [m][h], c3 [m] with m = w (2 d + 1); the
 *                   hypernetwork's output is ordered W [w][d], b [w], U [w][d].
 */
typedef struct {
    mpode_vel_kind kind;
    int d;              /* stored state width per sample */
    int n_layers;       /* MLP kinds */
    const int* widths;  /* MLP kinds: n_layers + 1 entries (copied by mpode_create) */
    mpode_act act;      /* MLP kinds: between the layers; CONV3X3_2: between the two convolutions */
    int append_time;    /* MLP kinds: time is appended to the first layer's input */
    int has_bias;       /* MLP kinds */
    int H, W, C;        /* CONV3X3_2, PARABOLIC_CONV */
    int n_intervals;    /* PARABOLIC_CONV: number of pieces of the piecewise-constant weights (>= 1) */
    int instance_norm;  /* PARABOLIC_CONV: 1 = with N, 0 = without */
} mpode_velocity_desc;

/* Explicit Runge-Kutta tableau (Sec. 3): Phi = sum_j b_j k_j, k_j = f(t_i + c_j h, y_i + h sum_{l<j} a[j*s+l] k_l). */
typedef struct {
    int stages;      /* 1..4 */
    const double* a; /* stages*stages, strictly lower triangular, row-major */
    const double* b; /* stages */
    const double* c; /* stages */
} mpode_tableau;

const mpode_tableau* mpode_tableau_euler(void); /* forward Euler, named in Sec. 3 */
const mpode_tableau* mpode_tableau_rk4(void);   /* classic 4th-order Runge-Kutta, Sec. 5 */

/*
 * Precision / scaling policy.
 *   low                     : format of Q16 (Sec. 2).
 *   scaling                 : backward variant (Sec. 5).
 *   k_max                   : maximum VJP attempts per step (Alg. 2, "maximum number of attempts"); <= 0 means 10.
 *   growth_rule             : 0 = double S when the scaled adjoint is small, S*||a||_inf <= 1/(2 u_L) (text below
 *                             Eq. (12)); 1 = the growth test as printed in Alg. 2, ||a||_inf <= 1/(2 u_L).
 *   round_increment         : 0 = y += sum_j (h b_j) k_j in fp32 from the 16-bit k_j; 1 = Phi rounded to 16 bits
 *                             before y += h Phi (Alg. 1 as printed).
 *   init_scale_exp_override : test hook.  MPODE_NO_OVERRIDE = off; otherwise the initial exponent of S (dynamic)
 *                             or a constant exponent (none / none_safe).
 *   time_gradient           : 1 = the backward pass also forms the derivative with respect to the time grid (the dt and dh
 *                             entries of Eq. (vjp) and the two t' updates of Alg. 2), returned by mpode_backward_ex; costs
 *                             some workspace and a full recompute of the last stage.  Dense velocities (MPODE_VEL_MLP,
 *                             MPODE_VEL_SCALAR_POLY) only; mpode_create returns MPODE_ERR_UNSUPPORTED for the others.
 */
#define MPODE_NO_OVERRIDE (-2147483647 - 1)
typedef struct {
    mpode_dtype low;
    mpode_scaling scaling;
    int k_max;
    int growth_rule;
    int round_increment;
    int init_scale_exp_override;
    int time_gradient;
} mpode_policy;

/* Per-step record of Alg. 2's scale decisions (host arrays of n_steps entries, caller-owned; index = step i). */
typedef struct {
    int n_steps;
    int* exp_used;            /* log2 S_i of the accepted attempt */
    int* attempts;            /* k of the accepted attempt (1 = no retry) */
    unsigned char* doubled;   /* 1 if S was doubled after step i (Alg. 2, growth branch) */
    int first_failed_step;    /* -1, or the step at which MPODE_ERR_SCALE_FAILED was raised */
} mpode_scale_log;

/* Counters of the last forward/backward pair, for benchmarks and for checking which kernels a configuration runs on. */
typedef struct {
    long long kernel_launches;     /* kernels of this library launched by the last call */
    long long retries;             /* halvings in the last mpode_backward */
    long long host_syncs;          /* times the last call waited for its stream to drain */
    long long tc_contractions;     /* layer-by-layer contractions that ran on the tensor-core kernels */
    long long simt_contractions;   /* layer-by-layer contractions that ran on the CUDA-core kernel (float32 mode, odd shapes) */
    long long fused_launches;      /* launches of the fused Runge-Kutta kernel (whole steps on the tensor cores) */
    long long whole_solve_launches;/* launches of the whole-solve kernels for very small networks */
    long long step_waits;          /* dynamic scaling: waits for the decision of a step, taken on the device, while the recompute of the
                                      next step is already queued (the stream keeps work) */
} mpode_stats;

/*
 * Create a context for (velocity, batch, policy).  max_steps bounds n_steps of later calls.
 * Returns INVALID_ARG for inconsistent sizes, UNSUPPORTED for shapes outside the built-in kernels' range.
 */
mpode_status mpode_create(mpode_ctx** out, const mpode_velocity_desc* vel, int batch, int max_steps,
                          const mpode_policy* policy);
void mpode_destroy(mpode_ctx* ctx);

size_t mpode_param_count(const mpode_ctx* ctx);                        /* p, number of fp32 parameters */
size_t mpode_state_width(const mpode_ctx* ctx);                        /* D */
size_t mpode_workspace_bytes(const mpode_ctx* ctx);                    /* device scratch the caller must provide */
size_t mpode_trajectory_bytes(const mpode_ctx* ctx, int n_steps);      /* (n_steps+1)*B*d low-format elements */

/*
 * Alg. 1.  theta_dev fp32[p]; y0_dev fp32[B, d]; tgrid_host fp32[n_steps+1], strictly increasing;
 * probe_dev int8 +-1 [B, d] for CNF_MLP (one Rademacher probe per sample, fixed over the solve), else NULL;
 * traj_dev out: low[(n_steps+1), B, d] = {Q16(y_i)}; yT_dev out: fp32[B, D] = y_N (for CNF_MLP column d holds l_N,
 * started at 0).  Asynchronous on `cuda_stream` (a cudaStream_t); workspace_dev must stay untouched until the
 * matching mpode_backward has returned.  256-byte alignment is required of workspace_dev, 16-byte of the others.
 * Because the call does not wait for the device, a device-side wait that timed out during it is reported by the next
 * call on this context that synchronises (mpode_backward, mpode_forward_host), as MPODE_ERR_CUDA.
 */
mpode_status mpode_forward(mpode_ctx* ctx, void* cuda_stream, const float* theta_dev, const float* y0_dev,
                           const float* tgrid_host, int n_steps, const mpode_tableau* tableau,
                           const signed char* probe_dev, void* traj_dev, float* yT_dev, void* workspace_dev,
                           size_t workspace_bytes);

/*
 * Alg. 2 (outputs dL/dx and dL/dtheta; mpode_backward_ex below also returns the time-grid gradient dL/dt).
 * dL_dyT_dev fp32[B, D] (terminal cost gradient; for CNF_MLP column d is dL/dl_N);
 * dL_dy0_dev out fp32[B, D]; dL_dtheta_dev fp32[p], overwritten, or accumulated into when accumulate_dtheta != 0;
 * log may be NULL.  Uses theta, trajectory, grid, tableau and probe of the last mpode_forward on this context.
 * Returns after its status is known.  With dynamic scaling the scale S, the accept / halve / double decisions and the log stay
 * on the device: a pass in which no attempt overflows waits for the stream to drain once, at its end (mpode_stats.host_syncs).
 * Per step the host waits for the device's decision (mpode_stats.step_waits, read from mapped host memory) with the recompute of
 * the next step already queued, so that an overflowing attempt wastes that recompute at most; after an overflow the host reads
 * the state and queues the failed step again.
 * On MPODE_ERR_SCALE_FAILED the outputs are unspecified and log->first_failed_step is set.
 */
mpode_status mpode_backward(mpode_ctx* ctx, void* cuda_stream, const float* dL_dyT_dev, float* dL_dy0_dev,
                            float* dL_dtheta_dev, int accumulate_dtheta, mpode_scale_log* log,
                            void* workspace_dev, size_t workspace_bytes);

/*
 * Alg. 2 with all three of its outputs and with a running cost (Sec. 3: the discrete objective sum_i w_i R(t_i, y_i) + C(y_N)).
 * Everything mpode_backward takes means the same here; in addition
 *   dL_dtraj_dev : NULL, or fp32 [n_steps][B, D]: the partial derivatives w_i dR/dy_i of the objective with respect to the states
 *                  y_0 .. y_{N-1} (that of y_N is part of dL_dyT_dev).  Slice i is added to the adjoint right after the update
 *                  of step i (Alg. 2, adjoint update), before the growth test.
 *   dL_dt_host   : NULL, or a HOST array of n_steps + 1 floats that receives dL/dt, the derivative with respect to the grid
 *                  points: per step the vector-Jacobian product's stage-time cotangents give dt = sum_j dtau_j and
 *                  dh = sum_j (c_j dtau_j + sum_{l<j} a_jl <psi_j, k_l>), then t'_i += (h_i / S_i)(dt - dh) - Phi^T a_{i+1} and
 *                  t'_{i+1} += (h_i / S_i) dh + Phi^T a_{i+1} in fp32 (Alg. 2, the two t' lines; signs as for the adjoint
 *                  update).  Q16(dt) and Q16(dh) join the finiteness test.  Needs a context created with
 *                  policy.time_gradient = 1 (MPODE_ERR_INVALID_ARG otherwise).
 * mpode_backward is this call with both set to NULL.
 */
mpode_status mpode_backward_ex(mpode_ctx* ctx, void* cuda_stream, const float* dL_dyT_dev, const float* dL_dtraj_dev,
                               float* dL_dy0_dev, float* dL_dtheta_dev, int accumulate_dtheta, float* dL_dt_host,
                               mpode_scale_log* log, void* workspace_dev, size_t workspace_bytes);

/*
 * Host-buffer variants of the two calls above (same algorithms, Alg. 1 / Alg. 2): inputs and outputs are HOST
 * pointers (pinned memory recommended); the library stages them through `io_dev`, a caller-provided device
 * buffer of at least mpode_io_bytes(ctx) bytes, copies the results back and synchronises the stream before
 * returning.  traj_dev and workspace_dev remain device buffers.
 */
size_t mpode_io_bytes(const mpode_ctx* ctx);
mpode_status mpode_forward_host(mpode_ctx* ctx, void* cuda_stream, const float* theta_host, const float* y0_host,
                                const float* tgrid_host, int n_steps, const mpode_tableau* tableau,
                                const signed char* probe_host, void* traj_dev, float* yT_host, void* io_dev,
                                void* workspace_dev, size_t workspace_bytes);
mpode_status mpode_backward_host(mpode_ctx* ctx, void* cuda_stream, const float* dL_dyT_host, float* dL_dy0_host,
                                 float* dL_dtheta_host, mpode_scale_log* log, void* io_dev, void* workspace_dev,
                                 size_t workspace_bytes);

/*
 * mpode_backward for callers that must not allocate device memory (the paper has no counterpart of this call).
 * Some hosts of this library cannot call cudaMalloc at the point where they need a gradient: code that runs inside
 * another framework's step with that framework's allocator locked, real-time loops that may not take the driver's
 * allocation lock, and processes whose memory budget was fixed at start-up.  For them the scratch memory of the
 * backward pass (the workspace every other call takes from the caller) lives in an array that is part of the
 * library image: MPODE_STATIC_WORKSPACE_BYTES bytes of device memory on every GPU that loads the library, held until
 * the process exits.  Inputs and outputs are still the caller's: dL_dyT_dev, dL_dy0_dev, dL_dtheta_dev and log mean
 * what they mean for mpode_backward, and the trajectory, parameters and time grid are those of the last
 * mpode_forward on this context (which keeps using the caller's workspace).
 *   - Returns MPODE_ERR_WORKSPACE_TOO_SMALL, with a message in mpode_last_error, when
 *     mpode_workspace_bytes(ctx) > MPODE_STATIC_WORKSPACE_BYTES; nothing is launched then.
 *   - The first call on a device looks up the array's device address (no allocation, but a runtime query): make that
 *     first call before any stream capture begins.
 *   - The CUDA runtime may load a kernel's code the first time that kernel is launched in a process, and that can allocate.
 *     A caller with a no-allocation region therefore runs one forward / backward pair of each configuration once, as a
 *     warm-up, before entering that region; from then on the call launches only kernels that are already resident.
 *   - The context, its buffers and the array must live on the current device: a dL_dyT_dev that belongs to another device
 *     is refused with MPODE_ERR_INVALID_ARG.  Arguments are checked before anything is queued on the stream.
 *   - All calls, from all contexts and streams, share the one array, and it keeps what the last call left in it; the
 *     call clears the words that must start at zero itself.  Two calls that overlap on the GPU race on it: serialise
 *     them.
 * No device memory is allocated or freed by this call or by anything it uses.
 */
#define MPODE_STATIC_WORKSPACE_BYTES (32u * 1024u * 1024u)
mpode_status mpode_backward_static_workspace(mpode_ctx* ctx, void* cuda_stream, const float* dL_dyT_dev,
                                             float* dL_dy0_dev, float* dL_dtheta_dev, int accumulate_dtheta,
                                             mpode_scale_log* log);

void mpode_get_stats(const mpode_ctx* ctx, mpode_stats* out);

/*
 * Test hook for the bounded device-side waits (the paper has no counterpart).  Every wait of the tensor-core kernels on a
 * counter or barrier gives up after a time limit, records a code in the workspace and lets the kernel wind down; the call
 * that next synchronises returns MPODE_ERR_CUDA ("a device-side wait timed out").  wait_limit_ns > 0 replaces the default
 * limit of 2 s for later calls on this context (0 restores it); starve_forward != 0 makes the second phase of the fused
 * forward program wait for a tile count one higher than is ever published, so that the limit is reached by construction.
 * Nothing faults or hangs: the context and the device stay usable.
 */
void mpode_debug_waits(mpode_ctx* ctx, unsigned long long wait_limit_ns, int starve_forward);

/*
 * Measurement hook (the paper has no counterpart).  While enabled, each velocity-layer contraction launch is
 * bracketed by CUDA events on the caller's stream.  mpode_collect_profile synchronises the device and returns, per
 * class (arrays of 4: 0 = forward layers, including the fused forward and recompute launches; 1 = input-gradient
 * layers; 2 = weight-gradient layers; 3 = fused backward launches, which hold input- and weight-gradient phases
 * together), the summed device time in milliseconds, the number of launches and the algorithmic FLOPs (2 M N K per
 * contraction), then clears the records.
 */
void mpode_set_profiling(mpode_ctx* ctx, int enabled);
mpode_status mpode_collect_profile(mpode_ctx* ctx, double* ms, long long* launches, double* flops);
const char* mpode_status_string(mpode_status s);
const char* mpode_last_error(const mpode_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* MPODE_H_ */
