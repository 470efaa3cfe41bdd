"""Seeded synthetic inputs for the five benchmark workloads.

This module serves both the CPU oracle's tests and the CUDA path's tests and
benchmark.  It holds none of the method's arithmetic: it only draws numbers
(a counter-based SplitMix64 stream, Box-Muller normals), shapes them like the
paper's workloads (Sec. 6: toy CNF-sized MLP, the linear ODE of its unit
tests, an MLP block, a conv block standing in for the STL-10 parabolic CNN,
a CNF with a trace estimate) and defines the caller-side loss heads that
turn a terminal state into dL/dy_T.  Everything is numpy; nothing here
touches CUDA or the oracle.

Seed 25 is the paper's fixed seed (Sec. 6.3).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, Optional, Tuple

import numpy as np

SEED = 25
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def splitmix64(key: int, n: int) -> np.ndarray:
    """n 64-bit words of the SplitMix64 stream started at `key` (counter based)."""
    with np.errstate(over="ignore"):
        ctr = np.arange(1, n + 1, dtype=np.uint64)
        return _mix(np.uint64(key & 0xFFFFFFFFFFFFFFFF) + ctr * _GOLDEN)


def stream_key(seed: int, config: int, tensor: int) -> int:
    """One independent stream per (seed, config index, tensor index)."""
    with np.errstate(over="ignore"):
        k = _mix(np.array([seed * 1000003 + config * 1009 + tensor + 1], dtype=np.uint64) * _GOLDEN)
    return int(k[0])


def uniform(key: int, n: int) -> np.ndarray:
    """n doubles in (0, 1)."""
    return ((splitmix64(key, n) >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(key: int, shape, scale: float = 1.0) -> np.ndarray:
    """Standard normals (Box-Muller in fp64) times `scale`, as fp64."""
    n = int(np.prod(shape))
    m = (n + 1) // 2
    u = uniform(key, 2 * m)
    r = np.sqrt(-2.0 * np.log(u[:m]))
    ang = 2.0 * np.pi * u[m:]
    z = np.concatenate([r * np.cos(ang), r * np.sin(ang)])[:n]
    return (z * scale).reshape(shape)


def rademacher(key: int, shape) -> np.ndarray:
    """+-1 as int8."""
    n = int(np.prod(shape))
    bits = (splitmix64(key, n) >> np.uint64(63)).astype(np.int8)
    return (2 * bits - 1).reshape(shape)


# ----------------------------------------------------------------------------
# workload description
# ----------------------------------------------------------------------------

@dataclass
class Workload:
    """One synthetic workload: what the caller hands to odeint forward/backward.

    vel        : dict describing the velocity (kind, sizes, activation)
    theta      : flat fp32 parameter vector in the library's documented layout
    y0         : fp32 [B, d]
    tgrid      : fp32 [N+1]
    solver     : "euler" | "rk4"
    low        : "f32" | "bf16" | "f16"
    scaling    : "none" | "none_safe" | "dynamic"
    k_max      : Alg. 2's maximum number of attempts per step
    probe      : int8 [B, d] Rademacher probe (CNF only)
    loss       : callable yT(float64 [B, D]) -> (loss value, dL/dyT float64 [B, D])
    extra      : generator by-products tests use (e.g. the eigen-decomposition of A)
    """
    name: str
    vel: Dict
    theta: np.ndarray
    y0: np.ndarray
    tgrid: np.ndarray
    solver: str
    low: str
    scaling: str
    loss: Callable[[np.ndarray], Tuple[float, np.ndarray]]
    probe: Optional[np.ndarray] = None
    extra: Dict = field(default_factory=dict)
    k_max: int = 10            # attempts per step that dynamic scaling may take (Alg. 2's k_max) when this workload is benchmarked

    @property
    def batch(self) -> int:
        return int(self.y0.shape[0])

    @property
    def n_steps(self) -> int:
        return int(self.tgrid.shape[0] - 1)


def mlp_param_count(widths, append_time: bool, bias: bool = True) -> int:
    p = 0
    for l in range(len(widths) - 1):
        fan_in = widths[l] + (1 if (append_time and l == 0) else 0)
        p += widths[l + 1] * fan_in + (widths[l + 1] if bias else 0)
    return p


def mlp_theta(cfg: int, widths, append_time: bool, bias: bool = True, first_tensor: int = 0) -> np.ndarray:
    """Layer l: W_l [out, in(+1 if time appended to the first layer)] row-major
    ~ N(0, 1/fan_in), then b_l [out] = 0.  Returned flat, fp32."""
    parts = []
    for l in range(len(widths) - 1):
        fan_in = widths[l] + (1 if (append_time and l == 0) else 0)
        W = normal(stream_key(SEED, cfg, first_tensor + l), (widths[l + 1], fan_in), 1.0 / np.sqrt(fan_in))
        parts.append(W.ravel())
        if bias:
            parts.append(np.zeros(widths[l + 1]))
    return np.concatenate(parts).astype(np.float32)


def _linspace01(n_steps: int) -> np.ndarray:
    return np.linspace(0.0, 1.0, n_steps + 1).astype(np.float32)


# ----------------------------------------------------------------------------
# caller-side loss heads (not part of the RK loop): terminal state -> dL/dy_T
# ----------------------------------------------------------------------------

def _loss_half_sq_to(target: np.ndarray):
    def f(yT):
        r = yT - target
        B = yT.shape[0]
        return 0.5 * float(np.sum(r * r)) / B, r / B
    return f


def _loss_mse_to(target: np.ndarray):
    def f(yT):
        r = yT - target
        return float(np.mean(r * r)), 2.0 * r / r.size
    return f


def _loss_gap_linear_ce(Wh: np.ndarray, bh: np.ndarray, labels: np.ndarray, H: int, W: int, C: int):
    def f(yT):
        B = yT.shape[0]
        feat = yT.reshape(B, H * W, C).mean(axis=1)
        logits = feat @ Wh.T + bh
        logits = logits - logits.max(axis=1, keepdims=True)
        lse = np.log(np.exp(logits).sum(axis=1, keepdims=True))
        logp = logits - lse
        loss = -float(np.mean(logp[np.arange(B), labels]))
        dlog = np.exp(logp)
        dlog[np.arange(B), labels] -= 1.0
        dfeat = (dlog / B) @ Wh
        dy = np.repeat(dfeat[:, None, :] / (H * W), H * W, axis=1).reshape(B, H * W * C)
        return loss, dy
    return f


def _loss_nll_standard_normal(d: int):
    def f(yT):
        B = yT.shape[0]
        z, ell = yT[:, :d], yT[:, d]
        loss = float(np.mean(0.5 * np.sum(z * z, axis=1) + 0.5 * d * np.log(2.0 * np.pi) + ell))
        dy = np.concatenate([z / B, np.full((B, 1), 1.0 / B)], axis=1)
        return loss, dy
    return f


# ----------------------------------------------------------------------------
# the five configurations
# ----------------------------------------------------------------------------

def toy_mlp(batch: int = 512, n_steps: int = 10, hidden: int = 32, low: str = "f16",
            scaling: str = "dynamic") -> Workload:
    """d=2, f = W2 tanh(W1 [y;t] + b1) + b2, RK4, loss 0.5||y(1) - R y0||^2 (mean over batch)."""
    cfg, d = 1, 2
    widths = [d, hidden, d]
    theta = mlp_theta(cfg, widths, True)
    y0 = normal(stream_key(SEED, cfg, 10), (batch, d)).astype(np.float32)
    R = np.array([[0.0, -1.0], [1.0, 0.0]])
    target = y0.astype(np.float64) @ R.T
    vel = dict(kind="mlp", d=d, widths=widths, act="tanh", append_time=True, bias=True)
    return Workload("c1_toy_mlp", vel, theta, y0, _linspace01(n_steps), "rk4", low, scaling,
                    _loss_half_sq_to(target))


def linear_ode(batch: int = 1024, n_steps: int = 100, d: int = 64, solver: str = "rk4",
               low: str = "bf16", scaling: str = "none") -> Workload:
    """y' = A y, A = -Q diag(lam) Q^T, lam log-uniform in [0.1, 10]; loss mean_b 0.5||y_b(1)||^2."""
    cfg = 2
    G = normal(stream_key(SEED, cfg, 0), (d, d))
    Q, Rm = np.linalg.qr(G)
    Q = Q * np.sign(np.diag(Rm))[None, :]
    lam = 10.0 ** (2.0 * uniform(stream_key(SEED, cfg, 1), d) - 1.0)
    A = -(Q * lam[None, :]) @ Q.T
    y0 = normal(stream_key(SEED, cfg, 10), (batch, d)).astype(np.float32)
    vel = dict(kind="linear", d=d, widths=[d, d], act="none", append_time=False, bias=False)
    return Workload("c2_linear_%s" % solver, vel, A.astype(np.float32).ravel(), y0, _linspace01(n_steps),
                    solver, low, scaling, _loss_half_sq_to(np.zeros((batch, d))),
                    extra=dict(Q=Q, lam=lam, A=A))


def mlp_block(batch: int = 8192, n_steps: int = 64, d: int = 256, hidden: int = 1024,
              low: str = "bf16", scaling: str = "none") -> Workload:
    """d -> hidden -> hidden -> d softplus MLP with time appended to the input; MSE to a N(0,1) target."""
    cfg = 3
    widths = [d, hidden, hidden, d]
    theta = mlp_theta(cfg, widths, True)
    y0 = normal(stream_key(SEED, cfg, 10), (batch, d)).astype(np.float32)
    target = normal(stream_key(SEED, cfg, 11), (batch, d)).astype(np.float32).astype(np.float64)
    vel = dict(kind="mlp", d=d, widths=widths, act="softplus", append_time=True, bias=True)
    return Workload("c3_mlp_block", vel, theta, y0, _linspace01(n_steps), "rk4", low, scaling,
                    _loss_mse_to(target), extra=dict(target=target))


def conv_block(batch: int = 256, n_steps: int = 8, H: int = 32, W: int = 32, C: int = 64,
               low: str = "f16", scaling: str = "dynamic", act: str = "relu", solver: str = "rk4") -> Workload:
    """NHWC state; f = conv3x3(C+1 -> C, time channel appended) -> ReLU -> conv3x3(C -> C), He init,
    zero biases; head = global average pool + linear(C -> 10) + cross-entropy on uniform labels.
    Parameter layout: W1 [C][3][3][C+1], b1 [C], W2 [C][3][3][C], b2 [C]."""
    cfg = 4
    W1 = normal(stream_key(SEED, cfg, 0), (C, 3, 3, C + 1), np.sqrt(2.0 / (9 * (C + 1))))
    W2 = normal(stream_key(SEED, cfg, 1), (C, 3, 3, C), np.sqrt(2.0 / (9 * C)))
    theta = np.concatenate([W1.ravel(), np.zeros(C), W2.ravel(), np.zeros(C)]).astype(np.float32)
    y0 = normal(stream_key(SEED, cfg, 10), (batch, H * W * C)).astype(np.float32)
    Wh = normal(stream_key(SEED, cfg, 2), (10, C), 1.0 / np.sqrt(C))
    labels = np.minimum((uniform(stream_key(SEED, cfg, 3), batch) * 10).astype(np.int64), 9)
    vel = dict(kind="conv", d=H * W * C, H=H, W=W, C=C, act=act, append_time=True)
    return Workload("c4_conv_block", vel, theta, y0, _linspace01(n_steps), solver, low, scaling,
                    _loss_gap_linear_ce(Wh, np.zeros(10), labels, H, W, C),
                    extra=dict(labels=labels, Wh=Wh),
                    # the pooled loss gives every pixel of an image the same cotangent: the weight gradient of the first step adds
                    # up coherently over all pixels and overflows until S_N has been halved about fifteen times at full size
                    k_max=40)


def parabolic_block(batch: int = 4, n_steps: int = 4, H: int = 32, W: int = 32, C: int = 128, n_intervals: int = 4,
                    low: str = "bf16", scaling: str = "none", norm: bool = True, solver: str = "rk4") -> Workload:
    """The parabolic convolutional ODE block of the paper's image classifier (Sec. 6.3): y' = -W(t)^T N(relu(W(t) y + b(t))), a 3x3
    convolution with C channels and its transpose with the same weights, instance normalisation, weights piecewise constant on
    `n_intervals` pieces of the step range (the paper: four RK4 steps, one set of weights per step, C = 128 / 256 / 512).  He
    initialisation, small random biases, N(0, 1) state, mean-squared error to a N(0, 1) target.
    Parameter layout: for each piece W_i [C][3][3][C] then b_i [C]."""
    cfg = 6
    parts = []
    for i in range(n_intervals):
        parts.append(normal(stream_key(SEED, cfg, 2 * i), (C, 3, 3, C), np.sqrt(2.0 / (9 * C))).ravel())
        parts.append(normal(stream_key(SEED, cfg, 2 * i + 1), (C,), 0.1))
    theta = np.concatenate(parts).astype(np.float32)
    y0 = normal(stream_key(SEED, cfg, 100), (batch, H * W * C)).astype(np.float32)
    target = normal(stream_key(SEED, cfg, 101), (batch, H * W * C)).astype(np.float32).astype(np.float64)
    vel = dict(kind="parabolic", d=H * W * C, H=H, W=W, C=C, n_intervals=n_intervals, n_steps=n_steps, norm=norm, act="relu")
    return Workload("parabolic_conv_block", vel, theta, y0, _linspace01(n_steps), solver, low, scaling, _loss_mse_to(target),
                    extra=dict(target=target))


def cnf_mlp(batch: int = 2048, n_steps: int = 8, d: int = 784, hidden: int = 2048,
            low: str = "bf16", scaling: str = "none") -> Workload:
    """Joint state [z; l]; z' = MLP(d+1 -> hidden -> hidden -> d, softplus)([z;t]), l' = -eps^T (dv/dz) eps
    with one Rademacher probe per sample; NLL under a standard normal base density."""
    cfg = 5
    widths = [d, hidden, hidden, d]
    theta = mlp_theta(cfg, widths, True)
    x0 = normal(stream_key(SEED, cfg, 10), (batch, d)).astype(np.float32)
    probe = rademacher(stream_key(SEED, cfg, 11), (batch, d))
    vel = dict(kind="cnf", d=d, widths=widths, act="softplus", append_time=True, bias=True)
    return Workload("c5_cnf_mlp", vel, theta, x0, _linspace01(n_steps), "rk4", low, scaling,
                    _loss_nll_standard_normal(d), probe=probe)


def hyper_cnf(batch: int = 1024, n_steps: int = 128, d: int = 2, hidden: int = 32, w: int = 128,
              low: str = "f16", scaling: str = "dynamic") -> Workload:
    """The two-dimensional flows of Sec. 6.1: joint state [z; l], z' = (1/w) sum_j U_j(t) tanh(W_j(t) . z + b_j(t)) with the w weight
    sets produced from t by three fully connected layers of width `hidden`, l' = -tr(dv/dz) written out exactly; batch 1024, RK4
    with 128 steps as in the paper; NLL under a standard normal base density.  The paper's 2-D point sets are not available:
    z_0 is a seeded two-ring mixture of the same scale.  Parameter layout: A1 [h][1], c1 [h], A2 [h][h], c2 [h], A3 [m][h], c3 [m],
    m = w (2 d + 1)."""
    cfg = 6
    m = w * (2 * d + 1)
    A1 = normal(stream_key(SEED, cfg, 0), (hidden, 1), 1.0)
    A2 = normal(stream_key(SEED, cfg, 1), (hidden, hidden), 1.0 / np.sqrt(hidden))
    A3 = normal(stream_key(SEED, cfg, 2), (m, hidden), 1.0 / np.sqrt(hidden))
    theta = np.concatenate([A1.ravel(), np.zeros(hidden), A2.ravel(), np.zeros(hidden), A3.ravel(), np.zeros(m)]).astype(np.float32)
    ang = uniform(stream_key(SEED, cfg, 10), batch) * 2.0 * np.pi
    rad = 1.0 + (uniform(stream_key(SEED, cfg, 11), batch) > 0.5) * 1.5 + 0.1 * normal(stream_key(SEED, cfg, 12), (batch,))
    x0 = np.zeros((batch, d))
    x0[:, 0], x0[:, 1 % d] = rad * np.cos(ang), rad * np.sin(ang)
    vel = dict(kind="cnf_hyper", d=d, hidden=hidden, w=w)
    return Workload("n4_hyper_cnf", vel, theta, x0.astype(np.float32), _linspace01(n_steps), "rk4", low, scaling,
                    _loss_nll_standard_normal(d))


def scalar_example(batch: int = 1, n_steps: int = 400, low: str = "f16", scaling: str = "dynamic") -> Workload:
    """The worked example of the paper (Example 1, Sec. 3): y' = -(theta_1 t^2 + theta_2 t + theta_3) y on [0, 2.65] with
    theta = (8, -11, 2^-16), x = 65504 / 180, classic RK4 with 400 equidistant steps, loss 0.5 y_N^2.  The adjoint
    y_N^2 / y_i falls far below the float16 range and climbs back, which is what dynamic adjoint scaling is for.
    Rows beyond the first repeat the example from slightly smaller initial values."""
    theta = np.array([8.0, -11.0, 2.0 ** -16], dtype=np.float32)
    x = 65504.0 / 180.0
    y0 = (x * (1.0 - 0.01 * np.arange(batch))).reshape(batch, 1).astype(np.float32)
    tgrid = np.linspace(0.0, 2.65, n_steps + 1).astype(np.float32)

    def loss(yT):
        return 0.5 * float(np.sum(yT * yT)), yT.copy()
    vel = dict(kind="scalar_poly", d=1)
    return Workload("example1_scalar", vel, theta, y0, tgrid, "rk4", low, scaling, loss)


FULL_CONFIGS = {
    "c1": toy_mlp,
    "c2": linear_ode,
    "c3": mlp_block,
    "c4": conv_block,
    "c5": cnf_mlp,
    # beyond the five configurations: the third ODE block of the paper's image classifier (Sec. 6.3: 512 channels at 32 x 32 pixels,
    # batch 16, four RK4 steps with one set of weights per step)
    "n2": lambda **kw: parabolic_block(**{**dict(batch=16, n_steps=4, H=32, W=32, C=512, n_intervals=4), **kw}),
    # the two-dimensional flows of Sec. 6.1 with the exact trace (hypernetwork velocity, batch 1024, 128 RK4 steps)
    "n4": hyper_cnf,
}
