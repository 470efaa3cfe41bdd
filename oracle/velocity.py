"""Velocity networks f(t, y; theta) and their vector-Jacobian products, in fp64 with emulated rounding.

TEST INFRASTRUCTURE ONLY (CPU oracle); shares no code with the CUDA path.

The paper evaluates the velocity and its VJP "in low precision" (Sec. 3,
Eq. (vjp)): operands are 16-bit, products are accumulated wide (the block-FMA
model of Sec. 2) and each tensor an operator produces is rounded once with
Q16.  `q` below is that rounding (the identity in exact mode).  Every
function takes already-rounded parameters `th16 = Q16(theta)` (Alg. 1 and Alg. 2 cast
the weights once per pass) and the already-rounded stage time `tau16`.

Rounding points inside a velocity (the paper does not list them; this list is
this implementation's reading, parity unpinned by the paper): each layer output after bias and activation
(one rounding; the pre-activation is not rounded separately); in the VJP each
cotangent after the activation-derivative product; the input cotangent psi.
Activation derivatives are evaluated from the rounded stored layer output H:
tanh' = 1 - H^2, softplus' = 1 - exp(-H), relu' = [H > 0].

Parameter layouts (flat fp32 vector theta):
  mlp / linear / cnf : for each layer l: W_l [out, in (+1 for the time column of the first layer)]
                       row-major, then b_l [out] if the network has biases.
  conv               : W1 [C][3][3][C+1], b1 [C], W2 [C][3][3][C], b2 [C].
  parabolic          : per time piece W_i [C][3][3][C], b_i [C].
  scalar_poly        : theta_1, theta_2, theta_3 of Example 1.
  cnf_hyper          : A1 [h][1], c1 [h], A2 [h][h], c2 [h], A3 [m][h], c3 [m] with m = w (2 d + 1); the hypernetwork output is
                       ordered W [w][d], b [w], U [w][d].
"""
from __future__ import annotations

from typing import Callable, Dict, List, Tuple

import numpy as np

Q = Callable[[np.ndarray], np.ndarray]


def _mm(q, a, b):
    """Contraction in the policy's accumulation precision (fp64 unless the rounding object says otherwise)."""
    mm = getattr(q, "mm", None)
    return mm(a, b) if mm is not None else a @ b


def _softplus(x):
    return np.maximum(x, 0.0) + np.log1p(np.exp(-np.abs(x)))


def act_forward(name: str, z):
    if name == "none":
        return z
    if name == "tanh":
        return np.tanh(z)
    if name == "softplus":
        return _softplus(z)
    if name == "relu":
        return np.maximum(z, 0.0)
    raise ValueError(name)


def act_deriv_from_output(name: str, H):
    """sigma'(z) written in terms of the layer output H = sigma(z)."""
    if name == "none":
        return np.ones_like(H)
    if name == "tanh":
        return 1.0 - H * H
    if name == "softplus":
        return -np.expm1(-H)
    if name == "relu":
        return (H > 0.0).astype(np.float64)
    raise ValueError(name)


class MLPVelocity:
    """f(t, y) = W_L act(... act(W_1 [y; t] + b_1) ...) + b_L.  `linear` is the one-layer, bias-free case."""

    def __init__(self, d: int, widths: List[int], act: str, append_time: bool, bias: bool = True):
        assert widths[0] == d and widths[-1] == d
        self.d = d
        self.D = d
        self.widths = list(widths)
        self.act = act
        self.append_time = append_time
        self.bias = bias
        self.L = len(widths) - 1
        self.slices = []
        off = 0
        for l in range(self.L):
            fan_in = widths[l] + (1 if (append_time and l == 0) else 0)
            w = (off, off + widths[l + 1] * fan_in, (widths[l + 1], fan_in))
            off = w[1]
            b = None
            if bias:
                b = (off, off + widths[l + 1])
                off = b[1]
            self.slices.append((w, b))
        self.p = off

    def unpack(self, th):
        out = []
        for (w, b) in self.slices:
            W = th[w[0]:w[1]].reshape(w[2])
            bb = th[b[0]:b[1]] if b is not None else None
            out.append((W, bb))
        return out

    def forward(self, tau16: float, Y, th16, q: Q, aux=None):
        layers = self.unpack(th16)
        X = Y
        Xs = [X]
        for l, (W, b) in enumerate(layers):
            n_in = self.widths[l]
            Z = _mm(q, X, W[:, :n_in].T)
            if b is not None:
                Z = Z + b
            if self.append_time and l == 0:
                Z = Z + tau16 * W[:, n_in]
            X = q(act_forward(self.act, Z)) if l < self.L - 1 else q(Z)
            Xs.append(X)
        return X, dict(Xs=Xs, tau16=tau16)

    def vjp(self, cache, kappa, th16, q: Q, want_dtau: bool = False):
        layers = self.unpack(th16)
        Xs = cache["Xs"]
        dth = np.zeros(self.p)
        lows = []
        dZ = kappa
        psi = None
        dtau = 0.0
        for l in range(self.L - 1, -1, -1):
            W, _ = layers[l]
            (w, b) = self.slices[l]
            n_in = self.widths[l]
            dW = np.zeros(w[2])
            dW[:, :n_in] = _mm(q, dZ.T, Xs[l])
            colsum = dZ.sum(axis=0)
            if self.append_time and l == 0:
                dW[:, n_in] = cache["tau16"] * colsum
                dtau = float(colsum @ W[:, n_in])          # z_1 = ... + tau w_t: the stage time enters through the time column
            dth[w[0]:w[1]] = dW.ravel()
            if b is not None:
                dth[b[0]:b[1]] = colsum
            dX = _mm(q, dZ, W[:, :n_in])
            if l > 0:
                dZ = q(act_deriv_from_output(self.act, Xs[l]) * dX)
                lows.append(dZ)
            else:
                psi = q(dX)
                lows.append(psi)
        return psi, dth, lows, dtau


class CNFVelocity(MLPVelocity):
    """Joint dynamics of a continuous normalising flow (Sec. 6.1): y = [z; l],
    z' = v(t, z), l' = -tr(dv/dz), the trace replaced by the one-probe estimate eps^T (dv/dz) eps
    carried as a forward-mode tangent through the same weights.

    Per layer l < L:  z_l = W_l x_{l-1} + b_l,  H_l = q(softplus(z_l)),
                      U_l = q(W_l g_{l-1})  (g_0 = eps, state columns only),
                      G_l = q(s(H_l) * U_l),  s(H) = softplus'(z) from the rounded output H.
    Last layer:       k_z = q(W_L H_{L-1} + b_L), U_L = q(W_L G_{L-1}), k_l = q(-sum_n eps_n U_L,n).
    """

    def __init__(self, d, widths, act, append_time, bias=True):
        super().__init__(d, widths, act, append_time, bias)
        self.D = d + 1

    def forward(self, tau16, Y, th16, q: Q, aux=None):
        eps = np.asarray(aux, dtype=np.float64)
        layers = self.unpack(th16)
        X, G = Y, eps
        Xs, Gs, Us = [X], [G], [None]
        for l, (W, b) in enumerate(layers):
            n_in = self.widths[l]
            Z = _mm(q, X, W[:, :n_in].T)
            if b is not None:
                Z = Z + b
            if self.append_time and l == 0:
                Z = Z + tau16 * W[:, n_in]
            U = q(_mm(q, G, W[:, :n_in].T))
            if l < self.L - 1:
                X = q(act_forward(self.act, Z))
                G = q(act_deriv_from_output(self.act, X) * U)
            else:
                X = q(Z)
                G = None
            Xs.append(X)
            Gs.append(G)
            Us.append(U)
        k_l = q(-np.sum(eps * Us[-1], axis=1, keepdims=True))
        k = np.concatenate([Xs[-1], k_l], axis=1)
        return k, dict(Xs=Xs, Gs=Gs, Us=Us, tau16=tau16, eps=eps)

    def vjp(self, cache, kappa, th16, q: Q, want_dtau: bool = False):
        assert self.act == "softplus"
        layers = self.unpack(th16)
        Xs, Gs, Us, eps = cache["Xs"], cache["Gs"], cache["Us"], cache["eps"]
        d = self.d
        dth = np.zeros(self.p)
        lows = []
        zeta = kappa[:, :d]                     # cotangent of the primal pre-activation
        ubar = q(-kappa[:, d:d + 1] * eps)      # cotangent of the tangent output U_L
        lows.append(ubar)
        psi = None
        dtau = 0.0
        for l in range(self.L - 1, -1, -1):
            W, _ = layers[l]
            (w, b) = self.slices[l]
            n_in = self.widths[l]
            dW = np.zeros(w[2])
            dW[:, :n_in] = _mm(q, zeta.T, Xs[l]) + _mm(q, ubar.T, Gs[l])
            colsum = zeta.sum(axis=0)
            if self.append_time and l == 0:
                dW[:, n_in] = cache["tau16"] * colsum
                dtau = float(colsum @ W[:, n_in])          # the tangent rows do not see the time column
            dth[w[0]:w[1]] = dW.ravel()
            if b is not None:
                dth[b[0]:b[1]] = colsum
            hbar = _mm(q, zeta, W[:, :n_in])
            if l > 0:
                gbar = _mm(q, ubar, W[:, :n_in])
                s = act_deriv_from_output(self.act, Xs[l])
                ubar = q(s * gbar)
                zeta = q(s * hbar + s * (1.0 - s) * Us[l] * gbar)
                lows += [ubar, zeta]
            else:
                psi = q(hbar)
                lows.append(psi)
        return psi, dth, lows, dtau


class HyperCNFVelocity:
    """The two-dimensional flows of Sec. 6.1: y = [z; l], z' = v(t, z) = (1/w) sum_j U_j(t) tanh(W_j(t) . z + b_j(t)) with the w
    weight sets (W_j, b_j, U_j) produced from t by three fully connected layers of hidden width h, and l' = -tr(dv/dz) with
    the trace written out, tr = (1/w) sum_j (U_j . W_j) (1 - tanh^2(W_j . z + b_j)), in place of a stochastic estimate.

    The paper gives the formula of v and says that the weights come from three fully connected layers of hidden width 32;
    everything else is this implementation's reading (parity unpinned by the paper): tanh between the three layers, none
    after the last; rounding points: the two hidden layers and the output of the hypernetwork, the products c_j = q(U_j . W_j),
    the units a_j = q(tanh(.)), the two outputs q(v) and q(-tr); in the VJP the unit cotangents, psi, and the batch-summed
    cotangents of the hypernetwork's output and hidden layers.  Sums are wide, one rounding per tensor.
    """

    def __init__(self, d: int, hidden: int, w: int):
        self.d, self.D, self.h, self.w = d, d + 1, hidden, w
        self.m = w * (2 * d + 1)
        h, m = hidden, self.m
        sizes = [("A1", (h, 1)), ("c1", (h,)), ("A2", (h, h)), ("c2", (h,)), ("A3", (m, h)), ("c3", (m,))]
        self.slices, off = {}, 0
        for name, shape in sizes:
            n = int(np.prod(shape))
            self.slices[name] = (off, off + n, shape)
            off += n
        self.p = off

    def unpack(self, th):
        return {k: th[a:b].reshape(shape) for k, (a, b, shape) in self.slices.items()}

    def _hyper(self, tau16, P, q):
        h1 = q(np.tanh(P["A1"][:, 0] * tau16 + P["c1"]))
        h2 = q(np.tanh(P["A2"] @ h1 + P["c2"]))
        o = q(P["A3"] @ h2 + P["c3"])
        w, d = self.w, self.d
        W, b, U = o[:w * d].reshape(w, d), o[w * d:w * d + w], o[w * d + w:].reshape(w, d)
        c = q(np.sum(U * W, axis=1))
        return h1, h2, W, b, U, c

    def forward(self, tau16, Y, th16, q: Q, aux=None):
        P = self.unpack(th16)
        h1, h2, W, b, U, c = self._hyper(tau16, P, q)
        A = q(np.tanh(Y @ W.T + b))                      # [B, w]
        v = q((A @ U) / self.w)
        k_l = q(-((1.0 - A * A) @ c) / self.w)[:, None]
        return np.concatenate([v, k_l], axis=1), dict(Y=Y, A=A, h1=h1, h2=h2, W=W, U=U, c=c, tau16=tau16)

    def vjp(self, cache, kappa, th16, q: Q, want_dtau: bool = False):
        P = self.unpack(th16)
        Y, A, h1, h2, W, U, c = (cache[k] for k in ("Y", "A", "h1", "h2", "W", "U", "c"))
        d, w = self.d, self.w
        kz, kl = kappa[:, :d], kappa[:, d]
        one_m = 1.0 - A * A
        abar = (kz @ U.T) / w + kl[:, None] * (2.0 / w) * c[None, :] * A      # tr enters with the sign of l' = -tr
        sbar = q(abar * one_m)
        psi = q(sbar @ W)
        cbar = -(kl @ one_m) / w
        Wbar = sbar.T @ Y + cbar[:, None] * U
        bbar = sbar.sum(axis=0)
        Ubar = (A.T @ kz) / w + cbar[:, None] * W
        obar = q(np.concatenate([Wbar.ravel(), bbar, Ubar.ravel()]))
        dth = np.zeros(self.p)

        def put(name, val):
            a, b_, _ = self.slices[name]
            dth[a:b_] = np.asarray(val).ravel()
        put("A3", np.outer(obar, h2)); put("c3", obar)
        h2bar = q((1.0 - h2 * h2) * (P["A3"].T @ obar))
        put("A2", np.outer(h2bar, h1)); put("c2", h2bar)
        h1bar = q((1.0 - h1 * h1) * (P["A2"].T @ h2bar))
        put("A1", h1bar * cache["tau16"]); put("c1", h1bar)
        return psi, dth, [sbar, psi, obar, h2bar, h1bar], 0.0


class ConvVelocity:
    """f(t, y) = conv3x3(act(conv3x3([y; t]) + b1)) + b2 on an NHWC image state, stride 1, zero padding 1, act = ReLU
    unless stated otherwise.  The time channel is appended to the input before padding (it is zero in the halo).
    Stand-in for the convolutional ODE blocks of Sec. 6.3."""

    def __init__(self, H: int, W: int, C: int, act: str = "relu"):
        self.H, self.W, self.C = H, W, C
        self.act = act
        self.d = H * W * C
        self.D = self.d
        n1 = C * 9 * (C + 1)
        n2 = C * 9 * C
        self.o_w1, self.o_b1, self.o_w2, self.o_b2 = 0, n1, n1 + C, n1 + C + n2
        self.p = n1 + C + n2 + C

    def unpack(self, th):
        C = self.C
        W1 = th[self.o_w1:self.o_b1].reshape(C, 3, 3, C + 1)
        b1 = th[self.o_b1:self.o_w2]
        W2 = th[self.o_w2:self.o_b2].reshape(C, 3, 3, C)
        b2 = th[self.o_b2:self.p]
        return W1, b1, W2, b2

    @staticmethod
    def _conv(X, Wt, q=None):
        B, H, W, Ci = X.shape
        Co = Wt.shape[0]
        Xp = np.zeros((B, H + 2, W + 2, Ci))
        Xp[:, 1:-1, 1:-1, :] = X
        out = np.zeros((B, H, W, Co))
        for r in range(3):
            for s in range(3):
                out += _mm(q, Xp[:, r:r + H, s:s + W, :], Wt[:, r, s, :].T)
        return out

    @staticmethod
    def _conv_transpose(dZ, Wt, q=None):
        B, H, W, Co = dZ.shape
        Ci = Wt.shape[3]
        dXp = np.zeros((B, H + 2, W + 2, Ci))
        for r in range(3):
            for s in range(3):
                dXp[:, r:r + H, s:s + W, :] += _mm(q, dZ, Wt[:, r, s, :])
        return dXp[:, 1:-1, 1:-1, :]

    @staticmethod
    def _wgrad(X, dZ, q=None):
        B, H, W, Ci = X.shape
        Co = dZ.shape[3]
        Xp = np.zeros((B, H + 2, W + 2, Ci))
        Xp[:, 1:-1, 1:-1, :] = X
        dW = np.zeros((Co, 3, 3, Ci))
        dZf = dZ.reshape(-1, Co)
        for r in range(3):
            for s in range(3):
                dW[:, r, s, :] = _mm(q, dZf.T, Xp[:, r:r + H, s:s + W, :].reshape(-1, Ci))
        return dW

    def forward(self, tau16, Y, th16, q: Q, aux=None):
        W1, b1, W2, b2 = self.unpack(th16)
        B = Y.shape[0]
        X = np.empty((B, self.H, self.W, self.C + 1))
        X[..., :self.C] = Y.reshape(B, self.H, self.W, self.C)
        X[..., self.C] = tau16
        H1 = q(act_forward(self.act, self._conv(X, W1, q) + b1))
        k = q(self._conv(H1, W2, q) + b2)
        return k.reshape(B, self.d), dict(X=X, H1=H1)

    def vjp(self, cache, kappa, th16, q: Q, want_dtau: bool = False):
        W1, b1, W2, b2 = self.unpack(th16)
        X, H1 = cache["X"], cache["H1"]
        B = X.shape[0]
        dth = np.zeros(self.p)
        dZ2 = kappa.reshape(B, self.H, self.W, self.C)
        dth[self.o_w2:self.o_b2] = self._wgrad(H1, dZ2, q).ravel()
        dth[self.o_b2:self.p] = dZ2.sum(axis=(0, 1, 2))
        dZ1 = q(act_deriv_from_output(self.act, H1) * self._conv_transpose(dZ2, W2, q))
        dth[self.o_w1:self.o_b1] = self._wgrad(X, dZ1, q).ravel()
        dth[self.o_b1:self.o_w2] = dZ1.sum(axis=(0, 1, 2))
        dX = self._conv_transpose(dZ1, W1, q)
        psi = q(dX[..., :self.C]).reshape(B, self.d)
        dtau = float(dX[..., self.C].sum())       # cotangent of the appended time channel, summed over the pixels (all inside the image)
        return psi, dth, [dZ1, psi], dtau


class ParabolicConvVelocity:
    """The parabolic convolutional layer of Sec. 6.3, Eq. (NODE_STL10): y' = -W(t)^T N(relu(W(t) y + b(t))), W a 3x3 convolution with
    C input and C output channels (stride 1, zero padding 1, NHWC), W^T its transpose with the same weights, N the instance
    normalisation, weights and biases piecewise constant in time.

    Readings (the paper gives none of these details; parity unpinned by the paper): N has no affine part, normalises each
    (image, channel) plane over its H*W pixels with the biased variance and eps = 1e-5, its statistics are formed wide from the
    rounded activations; one rounding per operator output (S = Q16(relu(W y + b)), Z = Q16(N(S)), k = Q16(-W^T Z)) and per
    cotangent in the VJP; `n_intervals` equal pieces of the step range share one (W_i, b_i): step i uses piece
    i * n_intervals // n_steps.  theta: for each piece W_i [C][3][3][C] then b_i [C].
    """
    EPS = 1e-5

    def __init__(self, H: int, W: int, C: int, n_intervals: int, n_steps: int, norm: bool = True):
        self.H, self.W, self.C = H, W, C
        self.norm = norm            # False: y' = -W^T relu(W y + b), the un-normalised block of the appendix's stability study
        self.d = H * W * C
        self.D = self.d
        self.n_intervals, self.n_steps = n_intervals, n_steps
        self.per = C * 9 * C + C
        self.p = n_intervals * self.per
        self.step = 0

    def set_step(self, i: int):
        self.step = int(i)

    def _piece(self):
        return self.step * self.n_intervals // self.n_steps

    def unpack(self, th, piece):
        C = self.C
        o = piece * self.per
        return th[o:o + 9 * C * C].reshape(C, 3, 3, C), th[o + 9 * C * C:o + self.per]

    def forward(self, tau16, Y, th16, q: Q, aux=None):
        piece = self._piece()
        Wt, b = self.unpack(th16, piece)
        B = Y.shape[0]
        X = Y.reshape(B, self.H, self.W, self.C)
        S = q(np.maximum(ConvVelocity._conv(X, Wt, q) + b, 0.0))
        if self.norm:
            mu = S.mean(axis=(1, 2), keepdims=True)
            var = ((S - mu) ** 2).mean(axis=(1, 2), keepdims=True)
            r = 1.0 / np.sqrt(var + self.EPS)
            Z = q((S - mu) * r)
        else:
            r, Z = None, S
        k = q(-ConvVelocity._conv_transpose(Z, Wt, q))
        return k.reshape(B, self.d), dict(X=X, S=S, Z=Z, r=r, piece=piece)

    def vjp(self, cache, kappa, th16, q: Q, want_dtau: bool = False):
        X, S, Z, r, piece = cache["X"], cache["S"], cache["Z"], cache["r"], cache["piece"]
        Wt, b = self.unpack(th16, piece)
        B, C = X.shape[0], self.C
        kap = kappa.reshape(B, self.H, self.W, C)
        dth = np.zeros(self.p)
        o = piece * self.per
        dZ = q(-ConvVelocity._conv(kap, Wt, q))                                   # transpose of the transposed convolution
        dW_out = -ConvVelocity._wgrad(kap, Z, q)                                  # k = -W^T Z as a function of W
        # instance normalisation, per (image, channel): dS = r (dZ - mean(dZ) - Z mean(dZ Z)), Z taken as stored (rounded)
        if self.norm:
            m1 = dZ.mean(axis=(1, 2), keepdims=True)
            m2 = (dZ * Z).mean(axis=(1, 2), keepdims=True)
            dS = q(r * (dZ - m1 - Z * m2))
        else:
            dS = dZ
        dU = q((S > 0.0) * dS)
        dth[o:o + 9 * C * C] = (ConvVelocity._wgrad(X, dU, q) + dW_out).ravel()
        dth[o + 9 * C * C:o + self.per] = dU.sum(axis=(0, 1, 2))
        psi = q(ConvVelocity._conv_transpose(dU, Wt, q)).reshape(B, self.d)
        return psi, dth, [dZ, dS, dU, psi], 0.0


class ScalarPolyVelocity:
    """Example 1: y' = -(theta_1 t^2 + theta_2 t + theta_3) y, a scalar state.
    Every arithmetic operation is rounded (the backward of Sec. 5 runs all operations in low precision)."""

    d = 1
    D = 1
    p = 3

    def forward(self, tau16, Y, th16, q: Q, aux=None):
        t2 = q(tau16 * tau16)
        lam = q(q(q(th16[0] * t2) + q(th16[1] * tau16)) + th16[2])
        k = q(-lam * Y)
        return k, dict(Y=Y, lam=lam, t2=t2, tau16=tau16)

    def vjp(self, cache, kappa, th16, q: Q, want_dtau: bool = False):
        Y, lam, t2, tau16 = cache["Y"], cache["lam"], cache["t2"], cache["tau16"]
        psi = q(-lam * kappa)
        dlam = q(-Y * kappa)                     # cotangent of lambda, per sample
        d1 = q(dlam * t2)
        d2 = q(dlam * tau16)
        dth = np.array([d1.sum(), d2.sum(), dlam.sum()])
        if not want_dtau:
            return psi, dth, [psi, dlam, d1, d2], 0.0
        # lambda = theta_1 t^2 + theta_2 t + theta_3 with t^2 formed as one rounded product: d lambda / d tau, operation by operation
        dt2 = q(dlam * th16[0])
        dtau_s = q(q(dt2 * q(2.0 * tau16)) + q(dlam * th16[1]))
        return psi, dth, [psi, dlam, d1, d2, dt2, dtau_s], float(dtau_s.sum())


def make_velocity(desc: Dict):
    kind = desc["kind"]
    if kind in ("mlp", "linear"):
        return MLPVelocity(desc["d"], desc["widths"], desc.get("act", "none"),
                           desc.get("append_time", False), desc.get("bias", kind == "mlp"))
    if kind == "cnf":
        return CNFVelocity(desc["d"], desc["widths"], desc["act"], desc["append_time"], desc.get("bias", True))
    if kind == "conv":
        return ConvVelocity(desc["H"], desc["W"], desc["C"], desc.get("act", "relu"))
    if kind == "parabolic":
        return ParabolicConvVelocity(desc["H"], desc["W"], desc["C"], desc["n_intervals"], desc["n_steps"], desc.get("norm", True))
    if kind == "scalar_poly":
        return ScalarPolyVelocity()
    if kind == "cnf_hyper":
        return HyperCNFVelocity(desc["d"], desc["hidden"], desc["w"])
    raise ValueError(kind)
