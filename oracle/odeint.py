"""Mixed-precision forward pass (Alg. 1) and backward pass with dynamic adjoint scaling (Alg. 2), on the CPU.

TEST INFRASTRUCTURE ONLY.  This is the slow, plain statement of the method the
CUDA path is checked against; only the tests, the smoke check and the
benchmark's CPU-baseline leg may call it.  It shares no code with the CUDA path.

The method is a finite-precision algorithm, so the oracle follows its steps in
the paper's order in fp64 and applies the quantisers at fixed points:

  Q16 (low):  theta (Alg. 1, Alg. 2: weights in low precision), the stored states (Alg. 1), every stage input and
              stage time handed to the velocity, each velocity tensor (see velocity.py), the seed
              Q16(S a) (Eq. (vjp)), the stage cotangents kappa_j and psi_j.
  Q32 (high): the running state y (Alg. 1) and the accumulators a, g (Alg. 2, high-precision updates),
              rounded once per update when `high="f32"`.

Two modes: exact (`low="f64"`: no rounding anywhere; the fp64 discrete RK map and its exact
discrete adjoint) and emulate (`low` in f16 / bf16 / f32).

Readings where the paper is silent or inconsistent (all configurable where two readings exist):
  * Adjoint sign: the adjoint update of Alg. 2 prints "a - (h/S) da" beside "g + (h/S) dg" from the same VJP.  The exact
    adjoint of y_{i+1} = y_i + h Phi(y_i) is a_i = a_{i+1} + h J^T a_{i+1}; this code uses "+" for both
    (pinned by finite differences in the tests).
  * Growth test (Alg. 2's last branch vs. the text below Eq. (12)): `growth_rule=0` doubles when the *scaled*
    adjoint is small, S ||a|| <= 1/(2 u_L); `growth_rule=1` is the literal ||a|| <= 1/(2 u_L).  Parity unpinned
    by the paper.
  * Increment: default sums h b_j k_j wide from the 16-bit k_j; `round_increment=1` rounds Phi to 16 bits first
    (Alg. 1 as printed).
  * Overflow test (Alg. 2, "all finite"): any non-finite value among the 16-bit tensors of the attempt (seed, kappa_j,
    the velocity's cotangents, psi_j) or in Q16(dg).
  * Time quantities: grid given in fp32; h_i, tau_j and the products h a_jl, h b_j, h / S are formed in fp64 and
    rounded to fp32 once (emulate mode only).
  * k_max is not given in the paper: default 10 (parity unpinned).  ||a|| = 0 gives S = 1; exponents are clamped to
    [-100, 100].
  * Time-grid gradient (the two t' updates of Alg. 2, the dt and dh entries of Eq. (vjp)): per stage the velocity returns the
    cotangent of its stage time, d tau_j = kappa_j^T df/dtau; then dt = sum_j d tau_j and
    dh = sum_j (c_j d tau_j + sum_{l<j} a_jl <psi_j, k_l>), sums and inner products formed wide from the 16-bit tensors
    (roundings of stage inputs and stage times are differentiated as the identity); Phi^T a uses Phi = sum_j b_j k_j formed
    wide and the adjoint before its update.  dt and dh join the finiteness test as Q16(dt), Q16(dh), like dg.  The
    signs follow the "+" reading of the adjoint update.  Parity unpinned by the paper beyond Alg. 2's two lines.
  * Running cost: the caller supplies w_i dR/dy_i (i < N) as `running_cot`; it is added to the adjoint after the update of
    step i (Alg. 2, adjoint update), before the growth test.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

from .quantize import precision_bits, quantize
from .tableau import Tableau

EXP_MIN, EXP_MAX = -100, 100


class Rounding:
    """Q16 as a callable, plus the contraction `mm` in the accumulation precision of the policy."""

    def __init__(self, low: str, acc: str = "f64"):
        self.low, self.acc = low, acc

    def __call__(self, x):
        return quantize(x, self.low)

    def mm(self, a, b):
        if self.acc == "f32":
            return (np.asarray(a, dtype=np.float32) @ np.asarray(b, dtype=np.float32)).astype(np.float64)
        return a @ b


@dataclass
class Policy:
    low: str = "bf16"            # "f64" (exact) | "f32" | "bf16" | "f16"
    high: str = "f32"            # "f64" | "f32": precision of y, a, g (ignored in exact mode)
    scaling: str = "none"        # "none" | "none_safe" | "dynamic"
    k_max: int = 10
    growth_rule: int = 0
    round_increment: int = 0
    init_scale_exp_override: Optional[int] = None   # test hook: initial (dynamic) or constant (none) exponent
    acc: str = "f64"             # "f64" | "f32": precision in which the velocity's contractions are accumulated.
                                 # Sec. 2 describes tensor units as accumulating in single precision ("block FMA");
                                 # "f32" emulates that with float32 library matmuls and is used to measure how
                                 # sensitive a result is to the accumulation order, not as the reference.

    @property
    def exact(self) -> bool:
        return self.low == "f64"

    @property
    def q(self):
        return Rounding(self.low, self.acc)

    def Q32(self, x):
        return x if self.exact else quantize(x, self.high)

    def f32(self, x: float) -> float:
        """Host scalars (step sizes, stage times, coefficients): one rounding to fp32."""
        return float(x) if self.exact else float(np.float32(x))


@dataclass
class ScaleLog:
    exp_used: List[int] = field(default_factory=list)   # per step i = N-1 .. 0, stored at index i
    attempts: List[int] = field(default_factory=list)
    doubled: List[int] = field(default_factory=list)
    first_failed_step: int = -1
    margin: float = np.inf        # smallest relative distance of a thresholded quantity from its threshold
    overflowed: bool = False      # none_safe: a non-finite value was seen


def initial_scale_exponent(m: float, low: str) -> int:
    """S_N = 2^floor(-log2(u_L ||a||)) (Alg. 2, scale initialisation) in integer arithmetic.
    With u_L = 2^-p and m = f 2^E, f in [0.5, 1): floor(p - log2 m) = p - ceil(log2 m),
    ceil(log2 m) = E if f > 0.5 and E - 1 if f = 0.5."""
    if m == 0.0:
        return 0
    f, E = np.frexp(m)
    c = int(E) if f > 0.5 else int(E) - 1
    return int(min(max(precision_bits(low) - c, EXP_MIN), EXP_MAX))


def _stage_time(pol: Policy, t_i: float, c_j: float, h: float) -> float:
    return pol.f32(float(t_i) + c_j * float(h))


def _stages(vel, th16, ybar, t_i, h, tab: Tableau, pol: Policy, aux, keep_cache: bool):
    """Evaluate the stages k_j = f(tau_j, Y_j) of one step from the stored low-precision state `ybar`."""
    d = vel.d
    ks, caches = [], []
    for j in range(tab.stages):
        tau16 = float(pol.q(_stage_time(pol, t_i, tab.c[j], h)))
        if j == 0:
            Y = ybar
        else:
            acc = ybar.copy()
            for l in range(j):
                if tab.a[j, l] != 0.0:
                    acc = acc + pol.f32(h * tab.a[j, l]) * ks[l][:, :d]
            Y = pol.q(acc)
        k, cache = vel.forward(tau16, Y, th16, pol.q, aux)
        ks.append(k)
        caches.append(cache if keep_cache else None)
    return ks, caches


def odeint_forward(vel, theta, y0, tgrid, tab: Tableau, pol: Policy, aux=None):
    """Alg. 1.  Returns (traj [N+1, B, d] holding Q16(y_i) as fp64, y_N [B, D] wide)."""
    theta = np.asarray(theta, dtype=np.float64)
    tgrid = np.asarray(tgrid, dtype=np.float64)
    N = tgrid.shape[0] - 1
    d, D = vel.d, vel.D
    B = y0.shape[0]
    th16 = pol.q(theta)
    y = np.zeros((B, D))
    y[:, :d] = pol.Q32(np.asarray(y0, dtype=np.float64))
    traj = np.empty((N + 1, B, d))
    traj[0] = pol.q(y[:, :d])
    for i in range(N):
        h = pol.f32(tgrid[i + 1] - tgrid[i])
        if hasattr(vel, "set_step"):
            vel.set_step(i)             # velocities whose parameters are piecewise constant in time (Sec. 6.3)
        ks, _ = _stages(vel, th16, traj[i], tgrid[i], h, tab, pol, aux, False)
        if pol.round_increment:
            phi = sum(pol.f32(tab.b[j]) * ks[j] for j in range(tab.stages))
            y = pol.Q32(y + h * pol.q(phi))
        else:
            inc = sum(pol.f32(h * tab.b[j]) * ks[j] for j in range(tab.stages))
            y = pol.Q32(y + inc)
        traj[i + 1] = pol.q(y[:, :d])
    return traj, y


def _rel_dist(x: float, thr: float) -> float:
    return abs(x - thr) / thr if thr > 0 else np.inf


def odeint_backward(vel, theta, traj, tgrid, tab: Tableau, pol: Policy, dL_dyT, aux=None, g0=None, running_cot=None,
                    want_dt: bool = False, tprime0=None):
    """Alg. 2.  Returns (dL/dy0 [B, D], dL/dtheta [p], ScaleLog), plus dL/dt [N+1] as a fourth value when `want_dt`.
    `running_cot` [N, B, D] holds the partial derivatives w_i dR/dy_i of a running cost for i < N (the terminal one is part
    of dL_dyT); `tprime0` the partial derivative of the loss with respect to the grid (default zero).  Raises RuntimeError
    when dynamic scaling exhausts k_max attempts (Alg. 2, failure branch)."""
    theta = np.asarray(theta, dtype=np.float64)
    tgrid = np.asarray(tgrid, dtype=np.float64)
    N = tgrid.shape[0] - 1
    d, D = vel.d, vel.D
    s = tab.stages
    pbits = precision_bits(pol.low)
    a = pol.Q32(np.asarray(dL_dyT, dtype=np.float64)).copy()
    g = np.zeros(vel.p) if g0 is None else pol.Q32(np.asarray(g0, dtype=np.float64)).copy()
    tprime = np.zeros(N + 1) if tprime0 is None else pol.Q32(np.asarray(tprime0, dtype=np.float64)).copy()
    log = ScaleLog(exp_used=[0] * N, attempts=[0] * N, doubled=[0] * N)
    dynamic = pol.scaling == "dynamic"
    checked = pol.scaling in ("dynamic", "none_safe")

    e = 0
    if dynamic:
        m = float(np.max(np.abs(a))) if a.size else 0.0
        if not np.isfinite(m):
            raise ValueError("non-finite dL/dy_T")
        e = initial_scale_exponent(m, pol.low)
        if m > 0:
            f, _ = np.frexp(m)
            log.margin = min(log.margin, _rel_dist(f, 0.5), _rel_dist(f, 1.0))
    if pol.init_scale_exp_override is not None:
        # test hook: start (dynamic) or stay (none / none_safe) at a given exponent
        e = int(pol.init_scale_exp_override)
    th16 = pol.q(theta)

    for i in range(N - 1, -1, -1):
        h = pol.f32(tgrid[i + 1] - tgrid[i])
        if hasattr(vel, "set_step"):
            vel.set_step(i)
        ks, caches = _stages(vel, th16, traj[i], tgrid[i], h, tab, pol, aux, True)  # Alg. 2: recompute
        accepted = False
        k_try = 0
        while k_try < (pol.k_max if dynamic else 1):
            k_try += 1
            v = pol.q(np.ldexp(a, e))                                              # Q16(S_i a), Eq. (vjp)
            lows = [v]
            psis = [None] * s
            da = np.zeros((a.shape[0], D))
            dg = np.zeros(vel.p)
            dt = 0.0
            dh = 0.0
            for j in range(s - 1, -1, -1):
                acc = pol.f32(tab.b[j]) * v
                for l in range(j + 1, s):
                    if tab.a[l, j] != 0.0:
                        acc[:, :d] = acc[:, :d] + pol.f32(h * tab.a[l, j]) * psis[l]
                kappa = pol.q(acc)
                psi, dth, vl, dtau = vel.vjp(caches[j], kappa, th16, pol.q, want_dt)
                psis[j] = psi
                da[:, :d] += psi
                dg += dth
                if want_dt:       # tau_j = t_i + c_j h and Y_j = ybar + h sum_l a_jl k_l both depend on the grid
                    dt += dtau
                    dh += pol.f32(tab.c[j]) * dtau
                    for l in range(j):
                        if tab.a[j, l] != 0.0:
                            dh += pol.f32(tab.a[j, l]) * float(np.sum(psi * ks[l][:, :d]))
                lows.append(kappa)
                lows += vl
            bad = False
            if checked:
                bad = any(not np.all(np.isfinite(x)) for x in lows) or not np.all(np.isfinite(pol.q(dg)))
                if want_dt:
                    bad = bad or not np.all(np.isfinite(pol.q(np.array([dt, dh]))))
            if dynamic and bad:
                e = max(e - 1, EXP_MIN)                                            # Alg. 2: halve, retry
                continue
            if bad:
                log.overflowed = True
            accepted = True
            break
        if not accepted:
            log.first_failed_step = i
            log.attempts[i] = k_try
            raise RuntimeError("dynamic adjoint scaling failed at step %d" % i)
        coef = pol.f32(h * 2.0 ** (-e))
        if want_dt:                                                                # Alg. 2: the two t' updates
            if pol.round_increment:
                phi = pol.q(sum(pol.f32(tab.b[j]) * ks[j] for j in range(s)))
            else:
                phi = sum(pol.f32(tab.b[j]) * ks[j] for j in range(s))
            phi_a = float(pol.Q32(np.sum(phi * a)))                                # Phi^T a_{i+1}, the adjoint before its update
            tprime[i] = pol.Q32(tprime[i] + pol.Q32(coef * (dt - dh)) - phi_a)
            tprime[i + 1] = pol.Q32(tprime[i + 1] + pol.Q32(coef * dh) + phi_a)
        a = pol.Q32(a + coef * da)                                                 # Alg. 2 adjoint update (sign: see header)
        if running_cot is not None:
            a = pol.Q32(a + pol.Q32(np.asarray(running_cot[i], dtype=np.float64)))  # w_i dR/dy_i
        g = pol.Q32(g + coef * dg)                                                 # Alg. 2 gradient update
        log.exp_used[i] = e
        log.attempts[i] = k_try
        if dynamic and k_try == 1:                                                 # Alg. 2: growth
            m = float(np.max(np.abs(a)))
            scaled = m * 2.0 ** e if pol.growth_rule == 0 else m
            thr = 2.0 ** (pbits - 1)
            if np.isfinite(scaled) and scaled > 0:
                log.margin = min(log.margin, _rel_dist(scaled, thr))
            if scaled <= thr and e < EXP_MAX:
                e += 1
                log.doubled[i] = 1
    if pol.scaling == "none_safe" and log.overflowed:
        a = np.full_like(a, np.inf)
        g = np.full_like(g, np.inf)
        tprime = np.full_like(tprime, np.inf)
    if want_dt:
        return a, g, log, tprime
    return a, g, log
