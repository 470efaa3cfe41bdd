"""More pins of the CPU oracle (no GPU needed): the tableaux other than Euler / RK4, the convolution, the literal
readings (rounded increment, printed growth test), a 16-bit running state, the increment's Jacobian against a hand-written
forward-mode tangent, and the time-grid gradient / running-cost terms of Alg. 2.

Each test ties the oracle to something it does not compute itself: an order of convergence, a direct six-loop sum,
exact rational arithmetic rounded by numpy's own float16, a consequence of the printed rule, the appendix's ordering
of the accumulator against the naive scheme, finite differences, an analytic solution.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import BY_NAME, Policy, make_velocity, odeint_backward, odeint_forward, precision_bits, quantize
from oracle.odeint import _stages
from paper_2510_23498_b200 import inputs

EXACT = Policy(low="f64")
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ observed order of every named tableau

@pytest.mark.parametrize("solver,order", [("midpoint", 2), ("heun", 2), ("kutta3", 3), ("rk38", 4)])
def test_named_tableaux_converge_with_their_order(solver, order):
    # a wrong coefficient anywhere in a table lowers the observed order (the adjoint tests cannot see that: they
    # are consistent with whatever map the table defines)
    wl = inputs.linear_ode(batch=6, n_steps=10, d=8, solver="rk4")
    Q, lam, A = wl.extra["Q"], wl.extra["lam"], wl.extra["A"]
    vel = make_velocity(wl.vel)
    y0 = wl.y0.astype(np.float64)
    exact = y0 @ ((Q * np.exp(-lam)[None, :]) @ Q.T).T
    errs = []
    for N in (40, 80, 160):
        _, yN = odeint_forward(vel, A.ravel(), y0, np.linspace(0, 1, N + 1), BY_NAME[solver], EXACT)
        errs.append(np.linalg.norm(yN - exact))
    r1, r2 = np.log2(errs[0] / errs[1]), np.log2(errs[1] / errs[2])
    assert abs(r1 - order) < 0.3 and abs(r2 - order) < 0.2, (solver, r1, r2)


@pytest.mark.parametrize("solver", ["euler", "midpoint", "heun", "kutta3", "rk4", "rk38"])
def test_tableau_consistency_conditions(solver):
    tab = BY_NAME[solver]
    assert abs(tab.b.sum() - 1.0) < 1e-15                                     # order 1
    assert np.allclose(tab.a.sum(axis=1), tab.c, atol=1e-15)                   # row sums = nodes
    if tab.stages > 1:
        assert abs(tab.b @ tab.c - 0.5) < 1e-15                                # order 2


# ------------------------------------------------------------------ convolution against a direct six-loop sum

def test_conv_velocity_matches_direct_loops_with_zero_padded_time_channel():
    rng = np.random.default_rng(3)
    B, H, W, C = 2, 3, 4, 2
    vel = make_velocity(dict(kind="conv", H=H, W=W, C=C, d=H * W * C))
    th = rng.standard_normal(vel.p)
    W1, b1, W2, b2 = vel.unpack(th)
    Y = rng.standard_normal((B, H * W * C))
    tau = 0.37
    k, cache = vel.forward(tau, Y, th, EXACT.q)
    y = Y.reshape(B, H, W, C)

    def conv(x_of, cin, Wt, bias):          # x_of(b, yy, xx, ci): the input, zero outside the image
        out = np.zeros((B, H, W, Wt.shape[0]))
        for b in range(B):
            for yy in range(H):
                for xx in range(W):
                    for co in range(Wt.shape[0]):
                        acc = bias[co]
                        for r in range(3):
                            for s in range(3):
                                for ci in range(cin):
                                    acc += Wt[co, r, s, ci] * x_of(b, yy + r - 1, xx + s - 1, ci)
                        out[b, yy, xx, co] = acc
        return out

    def x1(b, yy, xx, ci):
        if not (0 <= yy < H and 0 <= xx < W):
            return 0.0                      # padding: the time channel is zero there too
        return tau if ci == C else y[b, yy, xx, ci]
    h1 = np.maximum(conv(x1, C + 1, W1, b1), 0.0)

    def x2(b, yy, xx, ci):
        return h1[b, yy, xx, ci] if (0 <= yy < H and 0 <= xx < W) else 0.0
    ref = conv(x2, C, W2, b2)
    assert np.allclose(cache["H1"], h1, rtol=1e-13, atol=1e-13)
    assert np.allclose(k.reshape(B, H, W, C), ref, rtol=1e-12, atol=1e-13)
    # a corner pixel sees only four taps of the time channel: its pre-activation differs from an interior one's by exactly
    # the five missing time weights when the data channels are zero
    k0, c0 = vel.forward(tau, np.zeros_like(Y), th, EXACT.q)
    pre_corner = b1 + tau * W1[:, 1:, 1:, C].sum(axis=(1, 2))
    assert np.allclose(c0["H1"][0, 0, 0], np.maximum(pre_corner, 0.0), atol=1e-14)


# ------------------------------------------------------------------ literal readings

def _f16(x):
    """Round an exact rational to float16 with numpy's own conversion (independent of the oracle's quantiser)."""
    return Fraction(float(np.float16(np.float64(float(x)))))


def _f32(x):
    return Fraction(float(np.float32(np.float64(float(x)))))


@pytest.mark.parametrize("round_increment", [0, 1])
def test_increment_rounding_matches_exact_rational_arithmetic(round_increment):
    # one Heun step of y' = theta y in float16, every operation written out with exact fractions and numpy's rounding
    theta, y0, t0, t1 = 0.7431640625 + 2.0 ** -13, 1.23456789, 0.0, 0.30000001192092896
    vel = make_velocity(dict(kind="linear", d=1, widths=[1, 1], act="none"))
    pol = Policy(low="f16", round_increment=round_increment)
    traj, y = odeint_forward(vel, np.array([theta]), np.array([[y0]]), np.array([t0, t1], dtype=np.float32), BY_NAME["heun"], pol)
    th16, y32 = _f16(Fraction(theta)), _f32(Fraction(y0))
    ybar = _f16(y32)
    h = _f32(_f32(Fraction(t1)) - _f32(Fraction(t0)))
    k1 = _f16(th16 * ybar)
    Y2 = _f16(ybar + _f32(h * 1) * k1)
    k2 = _f16(th16 * Y2)
    if round_increment:      # Alg. 1 as printed: dy is a low-precision result, then y + h Q32(dy)
        phi = _f16(_f32(Fraction(1, 2)) * k1 + _f32(Fraction(1, 2)) * k2)
        y1 = _f32(y32 + h * phi)
    else:                    # stage derivatives are low precision, their combination is accumulated in high precision
        y1 = _f32(y32 + _f32(h * Fraction(1, 2)) * k1 + _f32(h * Fraction(1, 2)) * k2)
    assert Fraction(float(traj[0, 0, 0])) == ybar
    assert Fraction(float(y[0, 0])) == y1
    assert Fraction(float(traj[1, 0, 0])) == _f16(y1)


def test_increment_rounding_changes_the_result():
    wl = inputs.toy_mlp(batch=16, n_steps=8, hidden=8, low="bf16", scaling="none")
    vel = make_velocity(wl.vel)
    ya = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, BY_NAME["rk4"], Policy(low="bf16"))[1]
    yb = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, BY_NAME["rk4"], Policy(low="bf16", round_increment=1))[1]
    ye = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, BY_NAME["rk4"], EXACT)[1]
    assert not np.array_equal(ya, yb)
    # the extra rounding of Phi costs accuracy, it cannot gain any
    assert np.linalg.norm(ya - ye) <= 1.5 * np.linalg.norm(yb - ye)


def test_growth_rules_consequences():
    # small terminal cotangents: ||a|| stays far below 1/(2 u_L).  The printed test of Alg. 2 (unscaled norm) is then true
    # after every clean step, so S doubles every step until an overflow forces a halving; the scaled test keeps
    # S ||a|| inside (1/(2 u_L), 1/u_L] instead.
    wl = inputs.toy_mlp(batch=24, n_steps=12, hidden=8, low="f16", scaling="dynamic")
    vel = make_velocity(wl.vel)
    tab = BY_NAME["rk4"]
    traj, yN = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, tab, Policy(low="f16", scaling="dynamic"))
    aN = 1e-3 * wl.loss(yN)[1]
    p = precision_bits("f16")
    a1, g1, log1 = odeint_backward(vel, wl.theta, traj, wl.tgrid, tab, Policy(low="f16", scaling="dynamic", growth_rule=1, k_max=40), aN)
    a0, g0, log0 = odeint_backward(vel, wl.theta, traj, wl.tgrid, tab, Policy(low="f16", scaling="dynamic", growth_rule=0), aN)
    N = wl.n_steps
    assert np.max(np.abs(a1)) < 2.0 ** (p - 1)
    for i in range(N):
        assert log1.doubled[i] == (1 if log1.attempts[i] == 1 else 0)          # printed rule: always true here when k = 1
    assert sum(k - 1 for k in log1.attempts) >= 1                               # ... so S eventually overflows and is halved back
    assert max(log1.exp_used) > max(log0.exp_used)
    # scaled rule: the exponent follows the norm of the adjoint, few changes, no overflow
    assert all(k == 1 for k in log0.attempts)
    for i in range(N - 1):
        assert log0.exp_used[i] - log0.exp_used[i + 1] == log0.doubled[i + 1]
    m0 = np.max(np.abs(a0))
    e_next = log0.exp_used[0] + log0.doubled[0]
    assert 2.0 ** (p - 1) < m0 * 2.0 ** e_next <= 2.0 ** (p + 1)
    # both give the gradient to float16 accuracy
    assert np.linalg.norm(g1 - g0) <= 5e-3 * np.linalg.norm(g0)


# ------------------------------------------------------------------ a 16-bit running state (no high-precision accumulator)

def _angle_table():
    rows = {}
    for line in open(os.path.join(GOLDEN, "adjoint_angle_linearized.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            rows[k] = float(v)
    return rows


@pytest.mark.parametrize("low,name", [("bf16", "bfloat16"), ("f16", "float16")])
def test_low_precision_accumulator_is_an_order_of_magnitude_worse(low, name):
    # Sec. 4 (the u_H / h term with u_H = u_L) and the appendix's adjoint-direction table: forward Euler at half the
    # stability limit, 1000 steps, on a linear system y' = -K^T K y whose matrix is symmetric negative semi-definite with
    # a kernel (like the appendix's linearised block) and exactly representable in both 16-bit formats, so that rounding
    # the weights changes nothing and only the accumulator differs: the scheme with a float32 running state against the
    # naive one that keeps state, adjoint and gradient in the low format
    rng = np.random.default_rng(5)
    d, m, N = 24, 12, 1000
    K = rng.integers(-1, 2, size=(m, d)).astype(np.float64)
    A = -(K.T @ K) / 16
    assert np.array_equal(quantize(A, "bf16"), A)
    vel = make_velocity(dict(kind="linear", d=d, widths=[d, d], act="none"))
    h = 0.5 * 2.0 / np.max(np.abs(np.linalg.eigvalsh(A)))
    t = h * np.arange(N + 1)
    y0 = rng.standard_normal((4, d))
    tab = BY_NAME["euler"]

    def grad(pol, tt):
        traj, yN = odeint_forward(vel, A.ravel(), y0, tt, tab, pol)
        a0, _, _ = odeint_backward(vel, A.ravel(), traj, tt, tab, pol, yN)
        return a0.ravel(), yN

    ref, yN = grad(EXACT, t)
    assert 0.5 < np.linalg.norm(yN) / np.linalg.norm(y0) < 0.9      # the kernel's share of y0 survives (appendix: about 0.69)
    t32 = t.astype(np.float32)

    def angle(v):
        c = v @ ref / (np.linalg.norm(v) * np.linalg.norm(ref))
        return float(np.arccos(min(1.0, c)))

    mixed = angle(grad(Policy(low=low, high="f32"), t32)[0])
    naive = angle(grad(Policy(low=low, high=low), t32)[0])
    tab_ = _angle_table()
    assert naive >= 10.0 * mixed, (low, mixed, naive)                                  # "one to two orders of magnitude"
    assert tab_["mixed_" + name] / 10 < mixed < tab_["mixed_" + name] * 10             # same order as the printed value
    assert naive < tab_["naive_" + name] * 10
    assert mixed < 2.0 ** -precision_bits(low)                                          # O(u_L), the theorem of Sec. 4


# ------------------------------------------------------------------ increment Jacobian against a hand-written tangent

def _mlp_tangent(vel, theta, tau, Y, dY, dtheta, dtau):
    """Forward-mode derivative of the tanh MLP velocity, written directly from the chain rule."""
    layers = vel.unpack(theta)
    dlayers = vel.unpack(dtheta)
    X, dX = Y, dY
    for l, ((W, b), (dW, db)) in enumerate(zip(layers, dlayers)):
        n_in = vel.widths[l]
        Z = X @ W[:, :n_in].T + b
        dZ = dX @ W[:, :n_in].T + X @ dW[:, :n_in].T + db
        if l == 0:
            Z = Z + tau * W[:, n_in]
            dZ = dZ + dtau * W[:, n_in] + tau * dW[:, n_in]
        if l < vel.L - 1:
            X = np.tanh(Z)
            dX = (1.0 - X * X) * dZ
        else:
            X, dX = Z, dZ
    return X, dX


@pytest.mark.parametrize("solver", ["rk4", "kutta3", "rk38"])
def test_increment_vjp_is_the_transpose_of_a_hand_written_tangent(solver):
    # <d(h Phi), w> from a forward-mode tangent through the stage recursion equals <(u, dtheta, dt), VJP(w)> to roundoff
    rng = np.random.default_rng(17)
    vel = make_velocity(dict(kind="mlp", d=3, widths=[3, 5, 4, 3], act="tanh", append_time=True, bias=True))
    theta = 0.6 * rng.standard_normal(vel.p)
    tab = BY_NAME[solver]
    s = tab.stages
    y = rng.standard_normal((4, 3))
    t0, t1 = 0.2, 0.55
    h = t1 - t0
    u, dth = rng.standard_normal(y.shape), rng.standard_normal(vel.p)
    dt0, dt1 = 0.7, -0.4                      # tangent of the two grid points
    dhh = dt1 - dt0
    w = rng.standard_normal(y.shape)
    ks, dks = [], []
    for j in range(s):
        Yj = y + h * sum(tab.a[j, l] * ks[l] for l in range(j))
        dYj = u + dhh * sum(tab.a[j, l] * ks[l] for l in range(j)) + h * sum(tab.a[j, l] * dks[l] for l in range(j))
        k, dk = _mlp_tangent(vel, theta, t0 + tab.c[j] * h, Yj, dYj, dth, dt0 + tab.c[j] * dhh)
        ks.append(k)
        dks.append(dk)
    phi = sum(tab.b[j] * ks[j] for j in range(s))
    dstep = u + dhh * phi + h * sum(tab.b[j] * dks[j] for j in range(s))      # tangent of y + h Phi
    lhs = float(np.sum(dstep * w))
    a0, g, _, tp = odeint_backward(vel, theta, np.stack([y, y]), np.array([t0, t1]), tab, EXACT, w, want_dt=True)
    rhs = float(np.sum(a0 * u) + g @ dth + tp[0] * dt0 + tp[1] * dt1)
    assert abs(lhs - rhs) <= 1e-12 * max(1.0, abs(lhs)), (lhs, rhs)


# ------------------------------------------------------------------ time-grid gradient and running cost (Alg. 2, t' lines)

def _tiny(kind):
    rng = np.random.default_rng(7)
    if kind == "mlp_tanh":
        desc = dict(kind="mlp", d=3, widths=[3, 5, 3], act="tanh", append_time=True, bias=True)
    elif kind == "linear":
        desc = dict(kind="linear", d=4, widths=[4, 4], act="none", append_time=False, bias=False)
    elif kind == "conv":
        desc = dict(kind="conv", H=4, W=3, C=2, d=24)
    elif kind == "cnf":
        desc = dict(kind="cnf", d=4, widths=[4, 6, 5, 4], act="softplus", append_time=True, bias=True)
    elif kind == "scalar_poly":
        desc = dict(kind="scalar_poly")
    vel = make_velocity(desc)
    theta = rng.standard_normal(vel.p) * 0.5
    y0 = rng.standard_normal((3, vel.d))
    aux = rng.choice([-1.0, 1.0], size=(3, vel.d)) if kind == "cnf" else None
    return vel, theta, y0, aux


@pytest.mark.parametrize("kind", ["mlp_tanh", "linear", "conv", "cnf", "scalar_poly"])
@pytest.mark.parametrize("solver", ["euler", "rk4", "kutta3"])
def test_time_grid_gradient_matches_central_differences(kind, solver):
    vel, theta, y0, aux = _tiny(kind)
    tab = BY_NAME[solver]
    t = np.array([0.0, 0.13, 0.3, 0.41, 0.7])
    rng = np.random.default_rng(23)
    w = rng.uniform(0.5, 1.5, size=(y0.shape[0], vel.D))
    wr = rng.uniform(0.2, 0.8, size=(len(t) - 1, y0.shape[0], vel.d))          # running cost sum_i <wr_i, y_i^2> / 2, i < N

    def loss(tt, th=theta, x=y0):
        traj, yN = odeint_forward(vel, th, x, tt, tab, EXACT, aux)
        return 0.5 * np.sum(w * yN * yN) + 0.5 * np.sum(wr * traj[:-1] ** 2), traj, yN

    L, traj, yN = loss(t)
    cot = np.zeros((len(t) - 1, y0.shape[0], vel.D))
    cot[:, :, :vel.d] = wr * traj[:-1]
    a0, g, _, tp = odeint_backward(vel, theta, traj, t, tab, EXACT, w * yN, aux, running_cot=cot, want_dt=True)
    eps = 1e-6
    for i in range(len(t)):
        e = np.zeros_like(t); e[i] = eps
        fd = (loss(t + e)[0] - loss(t - e)[0]) / (2 * eps)
        assert abs(fd - tp[i]) <= 3e-7 * max(1.0, abs(fd)), (kind, solver, i, fd, tp[i])
    # the running cost also reaches dL/dy0 and dL/dtheta
    dy, dth = rng.standard_normal(y0.shape), rng.standard_normal(theta.shape)
    fd = (loss(t, theta + eps * dth, y0 + eps * dy)[0] - loss(t, theta - eps * dth, y0 - eps * dy)[0]) / (2 * eps)
    an = np.sum(a0[:, :vel.d] * dy) + g @ dth
    assert abs(fd - an) <= 3e-7 * max(1.0, abs(fd))
    # a velocity without explicit time dependence only sees differences of grid points: shifting the grid changes nothing
    if kind == "linear":
        assert abs(tp.sum()) <= 1e-12 * np.abs(tp).max()


def test_time_grid_gradient_of_the_scalar_example_is_the_analytic_end_point_derivative():
    # Example 1: y(T) = x exp(-int_0^T lambda), L = y(T)^2 / 2, so dL/dT = -lambda(T) y(T)^2, dL/dt_0 = +lambda(0) y(T)^2 and the
    # interior grid points do not matter (up to the discretisation error of RK4)
    vel = make_velocity(dict(kind="scalar_poly"))
    th = np.array([0.8, -1.1, 0.3])
    T, N, x = 1.3, 200, 1.7
    t = np.linspace(0.0, T, N + 1)
    traj, y = odeint_forward(vel, th, np.array([[x]]), t, BY_NAME["rk4"], EXACT)
    _, _, _, tp = odeint_backward(vel, th, traj, t, BY_NAME["rk4"], EXACT, y.copy(), want_dt=True)
    lamT, lam0 = th[0] * T * T + th[1] * T + th[2], th[2]
    yT = x * np.exp(-(th[0] / 3 * T ** 3 + th[1] / 2 * T ** 2 + th[2] * T))
    assert abs(tp[-1] + lamT * yT * yT) <= 1e-6 * abs(lamT * yT * yT)
    assert abs(tp[0] - lam0 * yT * yT) <= 1e-6 * abs(lam0 * yT * yT)
    assert np.max(np.abs(tp[1:-1])) <= 1e-7 * abs(tp[-1])


@pytest.mark.parametrize("low,scaling", [("bf16", "none"), ("f16", "dynamic"), ("f32", "none")])
def test_time_grid_gradient_in_mixed_precision_stays_at_the_low_precision_level(low, scaling):
    # the entries of dL/dt are differences of nearly equal terms (Phi_{i-1}^T a_i - Phi_i^T a_{i+1}), so their error is a
    # moderate multiple of the unit roundoff of the low format, the same multiple in every format
    tol = 32 * 2.0 ** -precision_bits(low)
    wl = inputs.toy_mlp(batch=32, n_steps=6, hidden=16, low=low, scaling=scaling)
    vel = make_velocity(wl.vel)
    tab = BY_NAME["rk4"]
    tr_e, y_e = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, tab, EXACT)
    _, _, _, tp_e = odeint_backward(vel, wl.theta, tr_e, wl.tgrid, tab, EXACT, wl.loss(y_e)[1], want_dt=True)
    pol = Policy(low=low, scaling=scaling)
    tr, y = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, tab, pol)
    a, g, log, tp = odeint_backward(vel, wl.theta, tr, wl.tgrid, tab, pol, wl.loss(y)[1], want_dt=True)
    assert np.linalg.norm(tp - tp_e) <= tol * np.linalg.norm(tp_e)
    # asking for dL/dt does not change the other outputs
    a2, g2, log2 = odeint_backward(vel, wl.theta, tr, wl.tgrid, tab, pol, wl.loss(y)[1])
    assert np.array_equal(a, a2) and np.array_equal(g, g2) and log.exp_used == log2.exp_used


# ------------------------------------------------------------------ the parabolic convolutional layer (Sec. 6.3, Eq. (NODE_STL10))

def _parabolic(norm=True, n_intervals=2, n_steps=4, seed=9):
    rng = np.random.default_rng(seed)
    H, W, C = 4, 3, 3
    vel = make_velocity(dict(kind="parabolic", H=H, W=W, C=C, n_intervals=n_intervals, n_steps=n_steps, norm=norm, d=H * W * C))
    theta = 0.5 * rng.standard_normal(vel.p)
    y0 = rng.standard_normal((2, vel.d))
    return vel, theta, y0


def test_parabolic_layer_pieces_against_their_definitions():
    vel, theta, y0 = _parabolic()
    H, W, C = vel.H, vel.W, vel.C
    Wt, b = vel.unpack(theta, 0)
    vel.set_step(0)
    k, cache = vel.forward(0.0, y0, theta, EXACT.q)
    # instance normalisation: every (image, channel) plane of Z has zero mean and variance var / (var + eps)
    S, Z = cache["S"], cache["Z"]
    for bi in range(2):
        for c in range(C):
            plane = S[bi, :, :, c]
            mu = sum(plane.ravel()) / (H * W)
            var = sum((v - mu) ** 2 for v in plane.ravel()) / (H * W)
            assert np.allclose(Z[bi, :, :, c], (plane - mu) / np.sqrt(var + 1e-5), rtol=1e-12, atol=1e-13)
    # the transposed convolution is the adjoint of the convolution (itself pinned by the six-loop test) with the SAME weights:
    # scatter definition out[p + tap, ci] += Z[p, co] W[co, tap, ci]
    out = np.zeros((2, H, W, C))
    for bi in range(2):
        for yy in range(H):
            for xx in range(W):
                for co in range(C):
                    for r in range(3):
                        for s_ in range(3):
                            y2, x2 = yy + r - 1, xx + s_ - 1
                            if 0 <= y2 < H and 0 <= x2 < W:
                                out[bi, y2, x2, :] += Z[bi, yy, xx, co] * Wt[co, r, s_, :]
    assert np.allclose(k.reshape(2, H, W, C), -out, rtol=1e-12, atol=1e-13)
    # piecewise-constant weights: steps 0, 1 use the first set, steps 2, 3 the second
    vel.set_step(1); k1 = vel.forward(0.0, y0, theta, EXACT.q)[0]
    vel.set_step(2); k2 = vel.forward(0.0, y0, theta, EXACT.q)[0]
    assert np.array_equal(k1, k) and not np.allclose(k2, k)


def test_parabolic_layer_without_normalisation_has_a_symmetric_negative_semidefinite_jacobian():
    # J = -W^T diag(relu') W (appendix: the structure behind the step-size study)
    vel, theta, y0 = _parabolic(norm=False)
    vel.set_step(0)
    rng = np.random.default_rng(2)
    _, cache = vel.forward(0.0, y0, theta, EXACT.q)
    u, v = rng.standard_normal(y0.shape), rng.standard_normal(y0.shape)
    Ju = vel.vjp(cache, u, theta, EXACT.q)[0]          # J^T u
    Jv = vel.vjp(cache, v, theta, EXACT.q)[0]
    assert abs(np.sum(Ju * v) - np.sum(u * Jv)) <= 1e-12 * abs(np.sum(Ju * v))      # <J^T u, v> = <u, J^T v>
    assert np.sum(Jv * v) <= 0.0 and np.sum(Ju * u) <= 0.0
    eps = 1e-6                                          # and J^T = J is the Jacobian of the forward map
    fd = (vel.forward(0.0, y0 + eps * v, theta, EXACT.q)[0] - vel.forward(0.0, y0 - eps * v, theta, EXACT.q)[0]) / (2 * eps)
    assert np.allclose(fd, Jv, rtol=1e-6, atol=1e-8)


@pytest.mark.parametrize("norm", [True, False])
@pytest.mark.parametrize("solver", ["euler", "rk4"])
def test_parabolic_layer_discrete_adjoint_matches_central_differences(norm, solver):
    vel, theta, y0 = _parabolic(norm=norm)
    tab = BY_NAME[solver]
    t = np.linspace(0.0, 0.6, 5)
    rng = np.random.default_rng(4)
    w = rng.uniform(0.5, 1.5, size=y0.shape)

    def loss_grad(th, x):
        traj, yN = odeint_forward(vel, th, x, t, tab, EXACT)
        a0, g, _ = odeint_backward(vel, th, traj, t, tab, EXACT, w * yN)
        return 0.5 * np.sum(w * yN * yN), a0, g

    L, a0, g = loss_grad(theta, y0)
    per = vel.per
    assert np.any(g[:per] != 0) and np.any(g[per:] != 0)           # both weight sets receive a gradient, each from its own steps
    eps = 1e-6
    for trial in range(4):
        dth, dy = rng.standard_normal(theta.shape), rng.standard_normal(y0.shape)
        fd = (loss_grad(theta + eps * dth, y0 + eps * dy)[0] - loss_grad(theta - eps * dth, y0 - eps * dy)[0]) / (2 * eps)
        an = np.sum(a0 * dy) + g @ dth
        assert abs(fd - an) <= 5e-7 * max(1.0, abs(fd)), (norm, solver, fd, an)


# ------------------------------------------------------------------ the two-dimensional flows with the exact trace (Sec. 6.1)

def _hyper(batch=6, hidden=8, w=16, seed=5):
    vel = make_velocity(dict(kind="cnf_hyper", d=2, hidden=hidden, w=w))
    rng = np.random.default_rng(seed)
    return vel, 0.5 * rng.standard_normal(vel.p), rng.standard_normal((batch, 2)), rng


def test_hypernetwork_velocity_is_the_printed_formula_and_its_trace_is_the_jacobian_trace():
    vel, theta, z, _ = _hyper()
    tau = 0.37
    k, _ = vel.forward(tau, z, theta, EXACT.q)
    # the weight sets: three fully connected layers from t, written out unit by unit
    P = vel.unpack(theta)
    h1 = [np.tanh(P["A1"][i, 0] * tau + P["c1"][i]) for i in range(vel.h)]
    h2 = [np.tanh(sum(P["A2"][i, j] * h1[j] for j in range(vel.h)) + P["c2"][i]) for i in range(vel.h)]
    o = [sum(P["A3"][i, j] * h2[j] for j in range(vel.h)) + P["c3"][i] for i in range(vel.m)]
    w, d = vel.w, vel.d
    Wj = lambda j: np.array(o[j * d:(j + 1) * d]); bj = lambda j: o[w * d + j]; Uj = lambda j: np.array(o[w * d + w + j * d:w * d + w + (j + 1) * d])

    def v_of(zz):        # v = (1/w) sum_j U_j tanh(W_j . z + b_j)
        return sum(Uj(j) * np.tanh(Wj(j) @ zz + bj(j)) for j in range(w)) / w
    for b in range(z.shape[0]):
        assert np.allclose(k[b, :2], v_of(z[b]), rtol=1e-12, atol=1e-14)
        J, e = np.zeros((2, 2)), 1e-6
        for i in range(2):
            dz = np.zeros(2); dz[i] = e
            J[:, i] = (v_of(z[b] + dz) - v_of(z[b] - dz)) / (2 * e)
        assert abs(k[b, 2] + np.trace(J)) <= 1e-8 * max(1.0, abs(np.trace(J)))     # l' = -tr(dv/dz), no estimate


def test_hypernetwork_flow_discrete_adjoint_matches_central_differences_and_the_dot_product_test():
    vel, theta, z, rng = _hyper(batch=5)
    t = np.array([0.0, 0.2, 0.45, 0.7, 1.0])
    tab = BY_NAME["rk4"]
    wgt = rng.uniform(0.5, 1.5, size=(5, 3))

    def loss_grad(th, x):
        traj, yN = odeint_forward(vel, th, x, t, tab, EXACT)
        a0, g, _ = odeint_backward(vel, th, traj, t, tab, EXACT, wgt * yN)
        return 0.5 * np.sum(wgt * yN * yN), a0, g, yN

    L, a0, g, yN = loss_grad(theta, z)
    assert np.allclose(a0[:, 2], (wgt * yN)[:, 2])          # l enters no velocity: its adjoint stays the terminal cotangent
    eps = 1e-6
    for trial in range(4):
        dth, dz = rng.standard_normal(theta.shape), rng.standard_normal(z.shape)
        fd = (loss_grad(theta + eps * dth, z + eps * dz)[0] - loss_grad(theta - eps * dth, z - eps * dz)[0]) / (2 * eps)
        an = np.sum(a0[:, :2] * dz) + g @ dth
        assert abs(fd - an) <= 2e-7 * max(1.0, abs(an)), (trial, fd, an)
    # <J u, kappa> = <u, J^T kappa> for one velocity evaluation: tangent by differences, cotangent by the VJP
    k0, cache = vel.forward(0.3, z, theta, EXACT.q)
    kap, u = rng.standard_normal(k0.shape), rng.standard_normal(z.shape)
    Ju = (vel.forward(0.3, z + eps * u, theta, EXACT.q)[0] - vel.forward(0.3, z - eps * u, theta, EXACT.q)[0]) / (2 * eps)
    psi = vel.vjp(cache, kap, theta, EXACT.q)[0]
    assert abs(np.sum(Ju * kap) - np.sum(u * psi)) <= 1e-7 * max(1.0, abs(np.sum(u * psi)))


def test_hypernetwork_flow_mixed_precision_stays_close_to_the_exact_discrete_gradient():
    wl = inputs.hyper_cnf(batch=48, n_steps=6, hidden=8, w=16)
    vel = make_velocity(wl.vel)
    y0 = wl.y0.astype(np.float64)
    tab = BY_NAME["rk4"]
    out = {}
    for name, pol in (("exact", EXACT), ("f16", Policy(low="f16", scaling="dynamic")), ("bf16", Policy(low="bf16", scaling="none"))):
        traj, yN = odeint_forward(vel, wl.theta, y0, wl.tgrid, tab, pol)
        _, dy = wl.loss(yN)
        a0, g, _ = odeint_backward(vel, wl.theta, traj, wl.tgrid, tab, pol, dy)
        out[name] = (yN, a0, g)
    for name, tol in (("f16", 5e-3), ("bf16", 4e-2)):
        for k in range(3):
            e = np.linalg.norm(out[name][k] - out["exact"][k]) / np.linalg.norm(out["exact"][k])
            assert e <= tol, (name, k, e)
