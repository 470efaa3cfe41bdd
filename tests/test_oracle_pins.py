"""Pins that tie the CPU oracle to what the paper and the mathematics fix (no GPU needed).

Closed forms for the linear ODE (the paper's own unit-test problem, Sec. 5), observed convergence order,
finite differences / dot-product tests for every velocity and tableau, the trace estimator against a
brute-force Jacobian, scale arithmetic against exact rational arithmetic, scaling neutrality, forced-overflow
bookkeeping, and the printed Table 1 of Example 1.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import (BY_NAME, EULER, RK4, Policy, initial_scale_exponent, make_velocity, odeint_backward,
                    odeint_forward, precision_bits, quantize)
from paper_2510_23498_b200 import inputs

EXACT = Policy(low="f64")
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _stab(z, name):
    return 1 + z if name == "euler" else 1 + z + z ** 2 / 2 + z ** 3 / 6 + z ** 4 / 24


def _dstab(z, name):
    return np.ones_like(z) if name == "euler" else 1 + z + z ** 2 / 2 + z ** 3 / 6


# ------------------------------------------------------------------ linear ODE: exact discrete closed forms

@pytest.mark.parametrize("solver", ["euler", "rk4"])
def test_linear_ode_discrete_closed_form_state_and_gradients(solver):
    wl = inputs.linear_ode(batch=16, n_steps=50, d=12, solver=solver)
    Q, lam, A = wl.extra["Q"], wl.extra["lam"], wl.extra["A"]
    vel = make_velocity(wl.vel)
    tab = BY_NAME[solver]
    N, B = wl.n_steps, wl.batch
    t = np.linspace(0.0, 1.0, N + 1)
    h = 1.0 / N
    y0 = wl.y0.astype(np.float64)
    traj, yN = odeint_forward(vel, A.ravel(), y0, t, tab, EXACT)
    mu = -lam
    gmu = _stab(h * mu, solver) ** N
    M = (Q * gmu[None, :]) @ Q.T
    assert np.allclose(yN, y0 @ M.T, rtol=1e-11, atol=1e-13)
    assert np.array_equal(traj[-1], yN)
    # gradients of L = mean_b 0.5 ||y_N||^2
    _, aN = wl.loss(yN)
    a0, g, _ = odeint_backward(vel, A.ravel(), traj, t, tab, EXACT, aN)
    assert np.allclose(a0, aN @ M, rtol=1e-10, atol=1e-14)
    dg = N * _stab(h * mu, solver) ** (N - 1) * _dstab(h * mu, solver) * h
    Gam = np.empty((len(mu), len(mu)))
    for i in range(len(mu)):
        for j in range(len(mu)):
            Gam[i, j] = dg[i] if i == j else (gmu[i] - gmu[j]) / (mu[i] - mu[j])
    C = aN.T @ y0                                    # sum_b a_b y0_b^T
    G = Q @ (Gam * (Q.T @ C @ Q)) @ Q.T
    assert np.allclose(g.reshape(A.shape), G, rtol=1e-8, atol=1e-12)


@pytest.mark.parametrize("solver,order", [("euler", 1), ("rk4", 4)])
def test_convergence_order_to_matrix_exponential(solver, order):
    wl = inputs.linear_ode(batch=8, n_steps=10, d=10, solver=solver)
    Q, lam, A = wl.extra["Q"], wl.extra["lam"], wl.extra["A"]
    vel = make_velocity(wl.vel)
    y0 = wl.y0.astype(np.float64)
    exact = y0 @ ((Q * np.exp(-lam)[None, :]) @ Q.T).T
    errs = []
    for N in (40, 80, 160):
        _, yN = odeint_forward(vel, A.ravel(), y0, np.linspace(0, 1, N + 1), BY_NAME[solver], EXACT)
        errs.append(np.linalg.norm(yN - exact))
    r1, r2 = errs[0] / errs[1], errs[1] / errs[2]
    assert abs(np.log2(r1) - order) < 0.25 and abs(np.log2(r2) - order) < 0.15


# ------------------------------------------------------------------ finite differences for every velocity / tableau

def _tiny(kind):
    rng = np.random.default_rng(7)
    if kind == "mlp_tanh":
        desc = dict(kind="mlp", d=3, widths=[3, 5, 3], act="tanh", append_time=True, bias=True)
    elif kind == "mlp_softplus":
        desc = dict(kind="mlp", d=3, widths=[3, 6, 4, 3], act="softplus", append_time=True, bias=True)
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
    B = 3
    y0 = rng.standard_normal((B, vel.d))
    aux = rng.choice([-1.0, 1.0], size=(B, vel.d)) if kind == "cnf" else None
    return vel, theta, y0, aux


def _loss_and_grad(vel, theta, y0, t, tab, aux, w):
    traj, yN = odeint_forward(vel, theta, y0, t, tab, EXACT, aux)
    L = 0.5 * np.sum(w * yN * yN)
    a0, g, _ = odeint_backward(vel, theta, traj, t, tab, EXACT, w * yN, aux)
    return L, a0, g


@pytest.mark.parametrize("kind", ["mlp_tanh", "mlp_softplus", "linear", "conv", "cnf", "scalar_poly"])
@pytest.mark.parametrize("solver", ["euler", "rk4", "midpoint", "heun", "kutta3", "rk38"])
def test_discrete_adjoint_matches_central_differences(kind, solver):
    vel, theta, y0, aux = _tiny(kind)
    tab = BY_NAME[solver]
    t = np.array([0.0, 0.13, 0.3, 0.41, 0.7])          # non-uniform grid
    rng = np.random.default_rng(11)
    w = rng.uniform(0.5, 1.5, size=(y0.shape[0], vel.D))
    L, a0, g = _loss_and_grad(vel, theta, y0, t, tab, aux, w)
    eps = 1e-6
    for trial in range(4):
        dth = rng.standard_normal(theta.shape)
        dy = rng.standard_normal(y0.shape)
        Lp = _loss_and_grad(vel, theta + eps * dth, y0 + eps * dy, t, tab, aux, w)[0]
        Lm = _loss_and_grad(vel, theta - eps * dth, y0 - eps * dy, t, tab, aux, w)[0]
        fd = (Lp - Lm) / (2 * eps)
        an = np.sum(a0[:, :vel.d] * dy) + np.sum(g * dth)
        assert abs(fd - an) <= 2e-7 * max(1.0, abs(fd)), (kind, solver, fd, an)


@pytest.mark.parametrize("kind", ["mlp_tanh", "conv", "cnf"])
def test_dot_product_identity_of_velocity_vjp(kind):
    # <J u, w> = <u, J^T w>, J u from central differences of the velocity itself
    vel, theta, y0, aux = _tiny(kind)
    q = EXACT.q
    rng = np.random.default_rng(5)
    u = rng.standard_normal(y0.shape)
    w = rng.standard_normal((y0.shape[0], vel.D))
    k0, cache = vel.forward(0.3, y0, theta, q, aux)
    eps = 1e-6
    Ju = (vel.forward(0.3, y0 + eps * u, theta, q, aux)[0] - vel.forward(0.3, y0 - eps * u, theta, q, aux)[0]) / (2 * eps)
    psi = vel.vjp(cache, w, theta, q)[0]
    assert abs(np.sum(Ju * w) - np.sum(u * psi)) <= 1e-8 * max(1.0, abs(np.sum(u * psi)))


def test_flipped_adjoint_sign_fails_finite_differences():
    # the printed "a - (h/S) da" (Alg. 2, adjoint update) cannot be the adjoint of y + h Phi: with the sign flipped the
    # first-order change of the loss is wrong already for y' = -y
    vel = make_velocity(dict(kind="linear", d=1, widths=[1, 1], act="none"))
    th = np.array([-1.0])
    t = np.linspace(0, 1, 5)
    traj, yN = odeint_forward(vel, th, np.array([[2.0]]), t, EULER, EXACT)
    a0, _, _ = odeint_backward(vel, th, traj, t, EULER, EXACT, np.ones((1, 1)))
    assert np.isclose(a0[0, 0], (1 - 0.25) ** 4)             # d y_N / d y_0 = (1 + h A)^N, "+" sign
    assert not np.isclose(a0[0, 0], (1 + 0.25) ** 4)


# ------------------------------------------------------------------ CNF: trace estimate

def test_cnf_trace_estimate_is_probe_quadratic_form_and_averages_to_trace():
    vel, theta, y0, _ = _tiny("cnf")
    d = vel.d
    q = EXACT.q
    z = y0[:1]
    eps_fd = 1e-6
    J = np.empty((d, d))
    for n in range(d):
        e = np.zeros((1, d)); e[0, n] = eps_fd
        kp = vel.forward(0.2, z + e, theta, q, np.ones((1, d)))[0][0, :d]
        km = vel.forward(0.2, z - e, theta, q, np.ones((1, d)))[0][0, :d]
        J[:, n] = (kp - km) / (2 * eps_fd)
    est = []
    for signs in itertools.product([-1.0, 1.0], repeat=d):
        p = np.array(signs)[None, :]
        k = vel.forward(0.2, z, theta, q, p)[0]
        assert abs(k[0, d] + p[0] @ J @ p[0]) < 1e-7             # k_l = -eps^T J eps
        est.append(k[0, d])
    assert abs(np.mean(est) + np.trace(J)) < 1e-7                # mean over all probes = -tr J


# ------------------------------------------------------------------ scale arithmetic (Alg. 2, initial scale)

@pytest.mark.parametrize("low", ["f16", "bf16", "f32"])
def test_initial_scale_is_floor_of_minus_log2_exactly(low):
    p = precision_bits(low)
    rng = np.random.default_rng(3)
    ms = list(np.exp(rng.uniform(-40, 30, 300))) + [2.0 ** k for k in range(-30, 20)]
    ms += [np.nextafter(2.0 ** k, np.inf) for k in range(-10, 10)] + [np.nextafter(2.0 ** k, 0) for k in range(-10, 10)]
    for m in ms:
        e = initial_scale_exponent(float(m), low)
        x = Fraction(2) ** p / Fraction(float(m))            # 1 / (u_L m), exact
        assert Fraction(2) ** e <= x < Fraction(2) ** (e + 1)  # e = floor(log2 x)
        sm = Fraction(float(m)) * Fraction(2) ** e
        assert Fraction(2) ** (p - 1) < sm <= Fraction(2) ** p  # ||S a|| in (1/(2 u_L), 1/u_L]
    assert initial_scale_exponent(0.0, low) == 0


# ------------------------------------------------------------------ scaling neutrality, retries, failure

def _small_mlp(low, scaling, B=24, N=6, **kw):
    wl = inputs.toy_mlp(batch=B, n_steps=N, hidden=8, low=low, scaling=scaling)
    vel = make_velocity(wl.vel)
    pol = Policy(low=low, scaling=scaling, **kw)
    return wl, vel, pol


@pytest.mark.parametrize("low", ["bf16", "f32"])
def test_power_of_two_scale_is_gradient_neutral_without_overflow(low):
    wl, vel, pol = _small_mlp(low, "none")
    traj, yN = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, RK4, pol)
    _, aN = wl.loss(yN)
    base = odeint_backward(vel, wl.theta, traj, wl.tgrid, RK4, pol, aN)
    for e in (-4, 3, 12):
        pe = Policy(low=low, scaling="none", init_scale_exp_override=e)
        a, g, _ = odeint_backward(vel, wl.theta, traj, wl.tgrid, RK4, pe, aN)
        assert np.array_equal(a, base[0]) and np.array_equal(g, base[1])


def test_dynamic_scaling_log_bookkeeping_under_forced_overflow():
    wl, vel, pol = _small_mlp("f16", "dynamic", k_max=40, init_scale_exp_override=30)
    traj, yN = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, RK4, pol)
    _, aN = wl.loss(yN)
    a, g, log = odeint_backward(vel, wl.theta, traj, wl.tgrid, RK4, pol, aN)
    N = wl.n_steps
    assert log.attempts[N - 1] > 1                               # 2^30 a overflows float16
    assert log.exp_used[N - 1] == 30 - (log.attempts[N - 1] - 1)   # one halving per retry
    for i in range(N - 2, -1, -1):
        start = log.exp_used[i + 1] + log.doubled[i + 1]
        assert log.exp_used[i] == start - (log.attempts[i] - 1)
        assert not (log.doubled[i] and log.attempts[i] > 1)        # growth only when no retry was needed
    # same gradients (to float16 accuracy) as the run that starts from the natural scale
    pol2 = Policy(low="f16", scaling="dynamic")
    a2, g2, log2 = odeint_backward(vel, wl.theta, traj, wl.tgrid, RK4, pol2, aN)
    assert np.linalg.norm(g - g2) <= 5e-3 * np.linalg.norm(g2)
    assert np.linalg.norm(a - a2) <= 5e-3 * np.linalg.norm(a2)
    assert all(np.isfinite(g)) and np.all(np.isfinite(a))
    p = precision_bits("f16")
    m = np.max(np.abs(aN))
    assert 2.0 ** (p - 1) < m * 2.0 ** initial_scale_exponent(m, "f16") <= 2.0 ** p


def test_dynamic_scaling_reports_failure_after_k_max():
    wl, vel, pol = _small_mlp("f16", "dynamic", k_max=1, init_scale_exp_override=40)
    traj, yN = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, RK4, pol)
    _, aN = wl.loss(yN)
    with pytest.raises(RuntimeError, match="failed at step %d" % (wl.n_steps - 1)):
        odeint_backward(vel, wl.theta, traj, wl.tgrid, RK4, pol, aN)


def test_none_safe_returns_infinite_gradients_on_overflow():
    wl, vel, pol = _small_mlp("f16", "none_safe", init_scale_exp_override=30)
    traj, yN = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, RK4, pol)
    _, aN = wl.loss(yN)
    a, g, log = odeint_backward(vel, wl.theta, traj, wl.tgrid, RK4, pol, aN)
    assert log.overflowed and np.all(np.isinf(g)) and np.all(np.isinf(a))
    pol_ok = Policy(low="f16", scaling="none_safe")
    a, g, log = odeint_backward(vel, wl.theta, traj, wl.tgrid, RK4, pol_ok, aN)
    assert not log.overflowed and np.all(np.isfinite(g))


def test_dynamic_scaling_rescues_underflowing_float16_adjoint():
    # terminal gradients of size 1e-7 are far below float16's normal range (2^-14)
    wl, vel, _ = _small_mlp("f16", "none")
    exact_traj, exact_yN = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, RK4, EXACT)
    aN = 1e-7 * np.random.default_rng(0).standard_normal(exact_yN.shape)
    _, g_ref, _ = odeint_backward(vel, wl.theta, exact_traj, wl.tgrid, RK4, EXACT, aN)
    errs = {}
    for sc in ("none", "dynamic"):
        pol = Policy(low="f16", scaling=sc)
        traj, _ = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, RK4, pol)
        _, g, _ = odeint_backward(vel, wl.theta, traj, wl.tgrid, RK4, pol, aN)
        errs[sc] = np.linalg.norm(g - g_ref) / np.linalg.norm(g_ref)
    assert errs["dynamic"] < 5e-3 and errs["none"] > 0.05


# ------------------------------------------------------------------ Example 1 / Table 1

def _example1(low, scaling):
    vel = make_velocity(dict(kind="scalar_poly"))
    T, N = 2.65, 400
    th = np.array([8.0, -11.0, 2.0 ** -16])
    x = 65504.0 / 180.0
    t = np.linspace(0, T, N + 1)
    pol = Policy(low=low, scaling=scaling)
    if low != "f64":
        t = t.astype(np.float32)
    traj, y = odeint_forward(vel, th, np.array([[x]]), t, RK4, pol)
    a, g, log = odeint_backward(vel, th, traj, t, RK4, pol, y.copy())
    yT = x * np.exp(-(th[0] / 3 * T ** 3 + th[1] / 2 * T ** 2 + th[2] * T))       # analytic solution
    ref = np.array([yT, yT * yT / x, -yT * yT * T ** 3 / 3, -yT * yT * T ** 2 / 2, -yT * yT * T])
    got = np.array([y[0, 0], a[0, 0], g[0], g[1], g[2]])
    return np.abs(got - ref) / np.abs(ref), log


def _table1():
    rows = {}
    for line in open(os.path.join(GOLDEN, "example1_relative_errors.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        rows[(f[0], f[1])] = np.array([float(v) for v in f[2:]])
    return rows


def test_example1_matches_table1_in_magnitude_and_outcome():
    tab = _table1()
    re64, _ = _example1("f64", "none")
    # float32 row is dominated by the RK4 discretisation error, which the exact mode isolates
    assert 0.3 * tab[("float32", "none")][0] < re64[0] < 1.5 * tab[("float32", "none")][0]
    assert np.allclose(re64[1:] / re64[0], 2.0, rtol=0.15)          # L = y^2/2 doubles the relative error
    for name, low in (("float32", "f32"), ("bfloat16", "bf16")):
        rn, _ = _example1(low, "none")
        rd, _ = _example1(low, "dynamic")
        assert np.all(rn <= 1.5 * tab[(name, "none")]) and np.all(rd <= 1.5 * tab[(name, "dynamic")])
        assert np.all(rn >= tab[(name, "none")] / 30)                # same order of magnitude (wide stage sums help)
        assert np.allclose(rn, rd, rtol=0.05, atol=1e-6)             # scaling does not matter at fp32 range
    r16n, _ = _example1("f16", "none")
    r16d, log = _example1("f16", "dynamic")
    assert r16n[0] <= tab[("float16", "none")][0] and np.all(r16n[1:] > 0.1)   # gradient lost without scaling
    assert np.all(r16d <= 1.5 * tab[("float16", "dynamic")]) and np.all(r16d[1:] <= 10 * r16d[0])
    assert sum(log.doubled) >= 10 and sum(k - 1 for k in log.attempts) >= 10      # both directions exercised


# ------------------------------------------------------------------ theory: error does not grow with N (Thm. 1)

def test_mixed_precision_error_is_flat_in_number_of_steps():
    wl, vel, pol = _small_mlp("bf16", "none", B=32)
    errs_y, errs_g = [], []
    for N in (8, 32, 128, 512):
        t = np.linspace(0, 1, N + 1)
        tr_e, y_e = odeint_forward(vel, wl.theta, wl.y0, t, RK4, EXACT)
        _, g_e, _ = odeint_backward(vel, wl.theta, tr_e, t, RK4, EXACT, y_e)
        tr, y = odeint_forward(vel, wl.theta, wl.y0, t.astype(np.float32), RK4, pol)
        _, g, _ = odeint_backward(vel, wl.theta, tr, t.astype(np.float32), RK4, pol, y)
        errs_y.append(np.linalg.norm(y - y_e) / np.linalg.norm(y_e))
        errs_g.append(np.linalg.norm(g - g_e) / np.linalg.norm(g_e))
    u = 2.0 ** -8
    assert max(errs_y) < 4 * u and max(errs_g) < 8 * u               # O(u_L), no growth with N
    assert max(errs_y) / min(errs_y) < 4 and max(errs_g) / min(errs_g) < 4
