"""ctypes binding of the C ABI in include/mpode.h: same names, argument marshalling only.

PyTorch is used for device memory and streams, nothing else: every step of Alg. 1 / Alg. 2 runs in the
library's kernels.  There is no CPU fallback: if the shared library is missing and cannot be built, importing
the entry points raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmpode.so")

# enums of mpode.h
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_BAD_STATE, ERR_NONFINITE_INPUT, \
    ERR_SCALE_FAILED, WARN_NONFINITE_GRAD = range(9)
DTYPES = {"f32": 0, "bf16": 1, "f16": 2}
SCALINGS = {"none": 0, "none_safe": 1, "dynamic": 2}
ACTS = {"none": 0, "tanh": 1, "softplus": 2, "relu": 3}
KINDS = {"mlp": 0, "linear": 0, "conv": 1, "cnf": 2, "scalar_poly": 3, "parabolic": 4, "cnf_hyper": 5}
NO_OVERRIDE = -2147483648

EXPORTS = [
    "mpode_tableau_euler", "mpode_tableau_rk4", "mpode_create", "mpode_destroy", "mpode_param_count",
    "mpode_state_width", "mpode_workspace_bytes", "mpode_trajectory_bytes", "mpode_forward", "mpode_backward",
    "mpode_io_bytes", "mpode_forward_host", "mpode_backward_host", "mpode_get_stats", "mpode_status_string",
    "mpode_last_error", "mpode_set_profiling", "mpode_collect_profile", "mpode_backward_static_workspace",
    "mpode_debug_waits", "mpode_backward_ex",
]
STATIC_WORKSPACE_BYTES = 32 * 1024 * 1024


class VelocityDesc(C.Structure):
    _fields_ = [("kind", C.c_int), ("d", C.c_int), ("n_layers", C.c_int), ("widths", C.POINTER(C.c_int)),
                ("act", C.c_int), ("append_time", C.c_int), ("has_bias", C.c_int),
                ("H", C.c_int), ("W", C.c_int), ("C", C.c_int), ("n_intervals", C.c_int), ("instance_norm", C.c_int)]


class Tableau(C.Structure):
    _fields_ = [("stages", C.c_int), ("a", C.POINTER(C.c_double)), ("b", C.POINTER(C.c_double)),
                ("c", C.POINTER(C.c_double))]


class Policy(C.Structure):
    _fields_ = [("low", C.c_int), ("scaling", C.c_int), ("k_max", C.c_int), ("growth_rule", C.c_int),
                ("round_increment", C.c_int), ("init_scale_exp_override", C.c_int), ("time_gradient", C.c_int)]


class ScaleLog(C.Structure):
    _fields_ = [("n_steps", C.c_int), ("exp_used", C.POINTER(C.c_int)), ("attempts", C.POINTER(C.c_int)),
                ("doubled", C.POINTER(C.c_ubyte)), ("first_failed_step", C.c_int)]


class Stats(C.Structure):
    _fields_ = [("kernel_launches", C.c_longlong), ("retries", C.c_longlong), ("host_syncs", C.c_longlong),
                ("tc_contractions", C.c_longlong), ("simt_contractions", C.c_longlong), ("fused_launches", C.c_longlong),
                ("whole_solve_launches", C.c_longlong), ("step_waits", C.c_longlong)]


_lib = None


def load_library(build_if_missing: bool = True) -> C.CDLL:
    """Load libmpode.so (building it with nvcc first if it is absent).  Raises if neither works."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        if not build_if_missing:
            raise RuntimeError("libmpode.so is missing; run `python -m paper_2510_23498_b200.build`")
        from . import build as _build
        _build.build()
    lib = C.CDLL(_LIB_PATH)
    vp, sz, i32 = C.c_void_p, C.c_size_t, C.c_int
    lib.mpode_tableau_euler.restype = C.POINTER(Tableau)
    lib.mpode_tableau_rk4.restype = C.POINTER(Tableau)
    lib.mpode_create.argtypes = [C.POINTER(vp), C.POINTER(VelocityDesc), i32, i32, C.POINTER(Policy)]
    lib.mpode_create.restype = i32
    lib.mpode_destroy.argtypes = [vp]
    lib.mpode_destroy.restype = None
    for name in ("mpode_param_count", "mpode_state_width", "mpode_workspace_bytes", "mpode_io_bytes"):
        getattr(lib, name).argtypes = [vp]
        getattr(lib, name).restype = sz
    lib.mpode_trajectory_bytes.argtypes = [vp, i32]
    lib.mpode_trajectory_bytes.restype = sz
    lib.mpode_forward.argtypes = [vp, vp, vp, vp, C.POINTER(C.c_float), i32, C.POINTER(Tableau), vp, vp, vp, vp, sz]
    lib.mpode_forward.restype = i32
    lib.mpode_backward.argtypes = [vp, vp, vp, vp, vp, i32, C.POINTER(ScaleLog), vp, sz]
    lib.mpode_backward.restype = i32
    lib.mpode_backward_ex.argtypes = [vp, vp, vp, vp, vp, vp, i32, C.POINTER(C.c_float), C.POINTER(ScaleLog), vp, sz]
    lib.mpode_backward_ex.restype = i32
    lib.mpode_backward_static_workspace.argtypes = [vp, vp, vp, vp, vp, i32, C.POINTER(ScaleLog)]
    lib.mpode_backward_static_workspace.restype = i32
    lib.mpode_forward_host.argtypes = [vp, vp, vp, vp, C.POINTER(C.c_float), i32, C.POINTER(Tableau), vp, vp, vp, vp,
                                       vp, sz]
    lib.mpode_forward_host.restype = i32
    lib.mpode_backward_host.argtypes = [vp, vp, vp, vp, vp, C.POINTER(ScaleLog), vp, vp, sz]
    lib.mpode_backward_host.restype = i32
    lib.mpode_get_stats.argtypes = [vp, C.POINTER(Stats)]
    lib.mpode_get_stats.restype = None
    lib.mpode_debug_waits.argtypes = [vp, C.c_ulonglong, i32]
    lib.mpode_debug_waits.restype = None
    lib.mpode_set_profiling.argtypes = [vp, i32]
    lib.mpode_set_profiling.restype = None
    lib.mpode_collect_profile.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_longlong), C.POINTER(C.c_double)]
    lib.mpode_collect_profile.restype = i32
    lib.mpode_status_string.argtypes = [i32]
    lib.mpode_status_string.restype = C.c_char_p
    lib.mpode_last_error.argtypes = [vp]
    lib.mpode_last_error.restype = C.c_char_p
    _lib = lib
    return lib


class MpodeError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("mpode status %d: %s" % (status, message))
        self.status = status


def make_tableau(a: Sequence[Sequence[float]], b: Sequence[float], c: Sequence[float]):
    """Build a Tableau struct; keeps the backing arrays alive on the returned object."""
    s = len(b)
    aa = (C.c_double * (s * s))(*[float(a[j][l]) for j in range(s) for l in range(s)])
    bb = (C.c_double * s)(*[float(x) for x in b])
    cc = (C.c_double * s)(*[float(x) for x in c])
    t = Tableau(s, C.cast(aa, C.POINTER(C.c_double)), C.cast(bb, C.POINTER(C.c_double)),
                C.cast(cc, C.POINTER(C.c_double)))
    t._keep = (aa, bb, cc)
    return t


NAMED_TABLEAUX = {
    "euler": ([[0.0]], [1.0], [0.0]),
    "midpoint": ([[0, 0], [0.5, 0]], [0.0, 1.0], [0.0, 0.5]),
    "heun": ([[0, 0], [1.0, 0]], [0.5, 0.5], [0.0, 1.0]),
    "kutta3": ([[0, 0, 0], [0.5, 0, 0], [-1.0, 2.0, 0]], [1 / 6, 2 / 3, 1 / 6], [0.0, 0.5, 1.0]),
    "rk4": ([[0, 0, 0, 0], [0.5, 0, 0, 0], [0, 0.5, 0, 0], [0, 0, 1.0, 0]], [1 / 6, 1 / 3, 1 / 3, 1 / 6],
            [0.0, 0.5, 0.5, 1.0]),
    "rk38": ([[0, 0, 0, 0], [1 / 3, 0, 0, 0], [-1 / 3, 1.0, 0, 0], [1.0, -1.0, 1.0, 0]],
             [1 / 8, 3 / 8, 3 / 8, 1 / 8], [0.0, 1 / 3, 2 / 3, 1.0]),
}


def _ptr(t) -> int:
    """Device (or pinned host) address of a torch tensor, or 0."""
    return 0 if t is None else int(t.data_ptr())


class Context:
    """Thin owner of one mpode_ctx plus the torch-allocated workspace and trajectory."""

    def __init__(self, vel: dict, batch: int, max_steps: int, low: str = "bf16", scaling: str = "none",
                 k_max: int = 10, growth_rule: int = 0, round_increment: int = 0,
                 init_scale_exp_override: Optional[int] = None, device: str = "cuda:0", time_gradient: bool = False):
        import torch
        self.torch = torch
        self.lib = load_library()
        self.device = torch.device(device)
        self.low = low
        kind = vel["kind"]
        widths = vel.get("widths")
        if kind == "cnf_hyper":
            widths = [int(vel["hidden"]), int(vel["w"])]
        self._widths = (C.c_int * len(widths))(*widths) if widths else None
        desc = VelocityDesc(KINDS[kind], int(vel["d"]), (len(widths) - 1) if widths else 0,
                            C.cast(self._widths, C.POINTER(C.c_int)) if widths else None,
                            ACTS[vel.get("act", "none")], int(bool(vel.get("append_time", False))),
                            int(bool(vel.get("bias", kind != "linear"))), int(vel.get("H", 0)), int(vel.get("W", 0)),
                            int(vel.get("C", 0)), int(vel.get("n_intervals", 0)), int(bool(vel.get("norm", True))))
        pol = Policy(DTYPES[low], SCALINGS[scaling], k_max, growth_rule, round_increment,
                     NO_OVERRIDE if init_scale_exp_override is None else int(init_scale_exp_override), 1 if time_gradient else 0)
        self.time_gradient = bool(time_gradient)
        h = C.c_void_p()
        st = self.lib.mpode_create(C.byref(h), C.byref(desc), batch, max_steps, C.byref(pol))
        if st != OK:
            raise MpodeError(st, self.lib.mpode_status_string(st).decode())
        self.h = h
        self.batch = batch
        self.max_steps = max_steps
        self.p = int(self.lib.mpode_param_count(h))
        self.D = int(self.lib.mpode_state_width(h))
        self.d = int(vel["d"])
        self.workspace_bytes = int(self.lib.mpode_workspace_bytes(h))
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=self.device)
        self.low_torch = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[low]
        self.traj = None
        self.io = None

    def close(self):
        if getattr(self, "h", None):
            self.lib.mpode_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int, allow=()):
        if st != OK and st not in allow:
            raise MpodeError(st, self.lib.mpode_last_error(self.h).decode() or self.lib.mpode_status_string(st).decode())
        return st

    def _stream(self) -> int:
        return int(self.torch.cuda.current_stream(self.device).cuda_stream)

    def _tableau(self, tab):
        if isinstance(tab, str):
            if tab == "euler":
                return self.lib.mpode_tableau_euler()
            if tab == "rk4":
                return self.lib.mpode_tableau_rk4()
            self._tab_keep = make_tableau(*NAMED_TABLEAUX[tab])
            return C.pointer(self._tab_keep)
        self._tab_keep = tab
        return C.pointer(tab)

    def forward(self, theta, y0, tgrid: np.ndarray, tab="rk4", probe=None, traj=None):
        """mpode_forward on device tensors.  Returns (traj [(N+1), B, d] low, yT [B, D] fp32).  `traj` may be a preallocated
        contiguous tensor of that shape (e.g. a view at an odd offset of a larger buffer)."""
        torch = self.torch
        n = int(len(tgrid) - 1)
        tg = np.ascontiguousarray(tgrid, dtype=np.float32)
        if traj is not None:
            assert tuple(traj.shape) == (n + 1, self.batch, self.d) and traj.dtype == self.low_torch and traj.is_contiguous()
            self.traj = traj
        elif self.traj is None or tuple(self.traj.shape) != (n + 1, self.batch, self.d) or self.traj.dtype != self.low_torch:
            self.traj = None                 # release the old buffer first: two trajectories must never be alive together
            self.traj = torch.empty((n + 1, self.batch, self.d), dtype=self.low_torch, device=self.device)
        yT = torch.empty((self.batch, self.D), dtype=torch.float32, device=self.device)
        self._keep = (theta, y0, probe, tg)
        st = self.lib.mpode_forward(self.h, self._stream(), _ptr(theta), _ptr(y0),
                                    tg.ctypes.data_as(C.POINTER(C.c_float)), n, self._tableau(tab), _ptr(probe),
                                    _ptr(self.traj), _ptr(yT), _ptr(self.workspace), self.workspace_bytes)
        self._check(st)
        return self.traj, yT

    def backward(self, dL_dyT, accumulate_into=None, want_log: bool = True, running_cot=None, want_dt: bool = False):
        """mpode_backward (mpode_backward_ex when a running-cost cotangent [N, B, D] or dL/dt is asked for).
        Returns (dL/dy0 [B, D], dL/dtheta [p], log dict or None, status); with want_dt the log dict carries "dL_dt"."""
        torch = self.torch
        n = self.traj.shape[0] - 1
        a0 = torch.empty((self.batch, self.D), dtype=torch.float32, device=self.device)
        g = accumulate_into if accumulate_into is not None else torch.empty(self.p, dtype=torch.float32, device=self.device)
        log = None
        if want_log:
            e = (C.c_int * n)()
            k = (C.c_int * n)()
            dbl = (C.c_ubyte * n)()
            log = ScaleLog(n, C.cast(e, C.POINTER(C.c_int)), C.cast(k, C.POINTER(C.c_int)),
                           C.cast(dbl, C.POINTER(C.c_ubyte)), -1)
        dt_arr = None
        if running_cot is not None or want_dt:
            dt_arr = np.zeros(n + 1, dtype=np.float32) if want_dt else None
            st = self.lib.mpode_backward_ex(self.h, self._stream(), _ptr(dL_dyT), _ptr(running_cot), _ptr(a0), _ptr(g),
                                            1 if accumulate_into is not None else 0,
                                            dt_arr.ctypes.data_as(C.POINTER(C.c_float)) if want_dt else None,
                                            C.byref(log) if log else None, _ptr(self.workspace), self.workspace_bytes)
        else:
            st = self.lib.mpode_backward(self.h, self._stream(), _ptr(dL_dyT), _ptr(a0), _ptr(g),
                                         1 if accumulate_into is not None else 0, C.byref(log) if log else None,
                                         _ptr(self.workspace), self.workspace_bytes)
        out_log = None
        if log is not None:
            out_log = dict(exp_used=list(e), attempts=list(k), doubled=[int(x) for x in dbl],
                           first_failed_step=int(log.first_failed_step))
        if dt_arr is not None:
            out_log = dict(out_log or {}, dL_dt=dt_arr)
        if st == ERR_SCALE_FAILED:
            return a0, g, out_log, st
        self._check(st, allow=(WARN_NONFINITE_GRAD,))
        return a0, g, out_log, st

    def backward_static_workspace(self, dL_dyT, out_a0=None, out_g=None, accumulate: bool = False, log_arrays=None):
        """mpode_backward_static_workspace: the backward pass on the library's own static device workspace (for callers
        that cannot allocate device memory).  With `out_a0` / `out_g` given (preallocated tensors) this wrapper allocates
        nothing either; `log_arrays` = (exp_used, attempts, doubled) ctypes arrays of n_steps entries receive the scale log.
        Returns (dL/dy0, dL/dtheta, status)."""
        torch = self.torch
        a0 = out_a0 if out_a0 is not None else torch.empty((self.batch, self.D), dtype=torch.float32, device=self.device)
        g = out_g if out_g is not None else torch.empty(self.p, dtype=torch.float32, device=self.device)
        log = None
        if log_arrays is not None:
            e, k, dbl = log_arrays
            log = ScaleLog(len(e), C.cast(e, C.POINTER(C.c_int)), C.cast(k, C.POINTER(C.c_int)), C.cast(dbl, C.POINTER(C.c_ubyte)), -1)
        st = self.lib.mpode_backward_static_workspace(self.h, self._stream(), _ptr(dL_dyT), _ptr(a0), _ptr(g),
                                                      1 if accumulate else 0, C.byref(log) if log is not None else None)
        self._check(st, allow=(WARN_NONFINITE_GRAD,))
        return a0, g, st

    # ---- host-buffer entry points (pinned torch tensors or numpy arrays as HOST pointers)
    def ensure_io(self):
        if self.io is None:
            nbytes = int(self.lib.mpode_io_bytes(self.h))
            self.io = self.torch.empty(nbytes + 256, dtype=self.torch.uint8, device=self.device)
        return self.io

    def forward_host(self, theta_h, y0_h, tgrid: np.ndarray, yT_h, tab="rk4", probe_h=None):
        torch = self.torch
        n = int(len(tgrid) - 1)
        tg = np.ascontiguousarray(tgrid, dtype=np.float32)
        if self.traj is None or self.traj.shape[0] != n + 1:
            self.traj = torch.empty((n + 1, self.batch, self.d), dtype=self.low_torch, device=self.device)
        self.ensure_io()
        self._keep = (theta_h, y0_h, probe_h, tg)
        st = self.lib.mpode_forward_host(self.h, self._stream(), _ptr(theta_h), _ptr(y0_h),
                                         tg.ctypes.data_as(C.POINTER(C.c_float)), n, self._tableau(tab),
                                         _ptr(probe_h), _ptr(self.traj), _ptr(yT_h), _ptr(self.io),
                                         _ptr(self.workspace), self.workspace_bytes)
        self._check(st)

    def backward_host(self, dL_dyT_h, dL_dy0_h, dL_dtheta_h):
        st = self.lib.mpode_backward_host(self.h, self._stream(), _ptr(dL_dyT_h), _ptr(dL_dy0_h), _ptr(dL_dtheta_h),
                                          None, _ptr(self.io), _ptr(self.workspace), self.workspace_bytes)
        return self._check(st, allow=(WARN_NONFINITE_GRAD,))

    def set_profiling(self, on: bool):
        self.lib.mpode_set_profiling(self.h, 1 if on else 0)

    def collect_profile(self) -> dict:
        ms = (C.c_double * 4)()
        n = (C.c_longlong * 4)()
        fl = (C.c_double * 4)()
        self._check(self.lib.mpode_collect_profile(self.h, ms, n, fl))
        names = ("forward", "dgrad", "wgrad", "fused_backward")
        return {names[k]: dict(ms=float(ms[k]), launches=int(n[k]), flops=float(fl[k])) for k in range(4)}

    def stats(self) -> dict:
        s = Stats()
        self.lib.mpode_get_stats(self.h, C.byref(s))
        return dict(kernel_launches=int(s.kernel_launches), retries=int(s.retries), host_syncs=int(s.host_syncs),
                    tc_contractions=int(s.tc_contractions), simt_contractions=int(s.simt_contractions),
                    fused_launches=int(s.fused_launches), whole_solve_launches=int(s.whole_solve_launches),
                    step_waits=int(s.step_waits))

    def debug_waits(self, wait_limit_ns: int = 0, starve_forward: bool = False):
        """Test hook of the bounded device-side waits (see mpode_debug_waits)."""
        self.lib.mpode_debug_waits(self.h, int(wait_limit_ns), 1 if starve_forward else 0)
