"""Shared helpers of the GPU parity tests: run one workload through the CPU oracle and through the C ABI."""
import numpy as np

from oracle import BY_NAME, Policy, make_velocity, odeint_backward, odeint_forward

TOL = {"f32": 1e-5, "bf16": 1e-2, "f16": 2e-3}     # relative L2 tolerances: fp32 mode vs the exact discrete solution, mixed modes vs the rounding-emulating oracle


def rel_l2(x, ref):
    x = np.asarray(x, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(x - ref) / den) if den > 0 else float(np.linalg.norm(x))


def run_oracle(wl, low=None, scaling=None, exact=False, want_dt=False, running_cot=None, **pol_kw):
    """Oracle forward + loss head + backward.  exact=True is the fp64 discrete solution (fp32-mode target)."""
    vel = make_velocity(wl.vel)
    pol = Policy(low="f64") if exact else Policy(low=low or wl.low, scaling=scaling or wl.scaling, **pol_kw)
    tab = BY_NAME[wl.solver]
    aux = None if wl.probe is None else wl.probe.astype(np.float64)
    traj, yT = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, tab, pol, aux)
    loss, dLdyT = wl.loss(yT)
    err = None
    tp = None
    try:
        out = odeint_backward(vel, wl.theta, traj, wl.tgrid, tab, pol, dLdyT, aux, running_cot=running_cot, want_dt=want_dt)
        a0, g, log = out[:3]
        tp = out[3] if want_dt else None
    except RuntimeError as ex:
        a0 = g = log = None
        err = str(ex)
    return dict(traj=traj, yT=yT, loss=loss, dLdyT=dLdyT, a0=a0, g=g, log=log, err=err, dL_dt=tp)


def run_gpu(wl, low=None, scaling=None, dLdyT=None, want_dt=False, running_cot=None, **pol_kw):
    """The same through mpode_forward / mpode_backward.  The loss head is caller-side numpy."""
    import torch
    from paper_2510_23498_b200 import binding
    low = low or wl.low
    ctx = binding.Context(wl.vel, wl.batch, wl.n_steps, low=low, scaling=scaling or wl.scaling, time_gradient=want_dt, **pol_kw)
    dev = ctx.device
    theta = torch.from_numpy(np.ascontiguousarray(wl.theta, dtype=np.float32)).to(dev)
    y0 = torch.from_numpy(np.ascontiguousarray(wl.y0, dtype=np.float32)).to(dev)
    probe = None if wl.probe is None else torch.from_numpy(np.ascontiguousarray(wl.probe)).to(dev)
    traj, yT = ctx.forward(theta, y0, wl.tgrid, wl.solver, probe)
    torch.cuda.synchronize()
    yT_h = yT.cpu().numpy().astype(np.float64)
    if dLdyT is None:
        loss, dLdyT = wl.loss(yT_h)
    else:
        loss = None
    dl = torch.from_numpy(np.ascontiguousarray(dLdyT, dtype=np.float32)).to(dev)
    cot = None if running_cot is None else torch.from_numpy(np.ascontiguousarray(running_cot, dtype=np.float32)).to(dev)
    a0, g, log, st = ctx.backward(dl, running_cot=cot, want_dt=want_dt)
    torch.cuda.synchronize()
    out = dict(dL_dt=(log or {}).get("dL_dt"), traj=traj.float().cpu().numpy(), yT=yT_h, loss=loss, dLdyT=dLdyT, a0=a0.cpu().numpy(),
               g=g.cpu().numpy(), log=log, status=st, stats=ctx.stats(), workspace_bytes=ctx.workspace_bytes)
    ctx.close()
    return out


def assert_parity(gpu, orc, tol, what=("yT", "traj", "a0", "g")):
    errs = {k: rel_l2(gpu[k], orc[k]) for k in what}
    bad = {k: v for k, v in errs.items() if not (v <= tol)}
    assert not bad, "relative L2 above %g: %s (all: %s)" % (tol, bad, errs)
    return errs


def assert_same_log(gpu_log, orc_log):
    assert gpu_log["exp_used"] == list(orc_log.exp_used), (gpu_log["exp_used"], orc_log.exp_used)
    assert gpu_log["attempts"] == list(orc_log.attempts), (gpu_log["attempts"], orc_log.attempts)
    assert gpu_log["doubled"] == list(orc_log.doubled), (gpu_log["doubled"], orc_log.doubled)
