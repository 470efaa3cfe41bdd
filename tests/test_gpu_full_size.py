"""Full-size configurations in the launch shapes the benchmark times, checked on sampled rows.

The oracle cannot run 8192 x 64 steps of the MLP block (or 256 images) in seconds, but samples are independent through
the forward loop and in the adjoint, and dL/dtheta is a sum over samples.  So the GPU runs the FULL batch, the oracle
runs a few sampled rows, and
  * y_N, the stored trajectory and dL/dy0 of those rows are compared directly;
  * dL/dtheta is compared by giving the GPU a terminal cotangent that is zero outside the sampled rows: rows with a zero
    adjoint contribute exactly nothing, so the full-batch gradient equals the oracle's gradient of the sampled rows.
"""
import numpy as np
import pytest

from oracle import BY_NAME, Policy, make_velocity, odeint_backward, odeint_forward
from paper_2510_23498_b200 import inputs
from _harness import TOL, rel_l2

pytestmark = pytest.mark.gpu


def _full_size_sampled(wl, rows, scale_log=False):
    import torch
    from paper_2510_23498_b200 import binding
    rows = np.asarray(rows)
    ctx = binding.Context(wl.vel, wl.batch, wl.n_steps, low=wl.low, scaling=wl.scaling)
    dev = ctx.device
    theta = torch.from_numpy(wl.theta).to(dev)
    y0 = torch.from_numpy(wl.y0).to(dev)
    probe = None if wl.probe is None else torch.from_numpy(wl.probe).to(dev)
    traj, yT = ctx.forward(theta, y0, wl.tgrid, wl.solver, probe)
    yT_h = yT.cpu().numpy().astype(np.float64)
    _, dl_full = wl.loss(yT_h)
    dl = np.zeros_like(dl_full)
    dl[rows] = dl_full[rows]                                   # cotangent only on the sampled rows
    a0, g, log, st = ctx.backward(torch.from_numpy(dl.astype(np.float32)).to(dev))
    assert st == 0
    torch.cuda.synchronize()
    gpu = dict(yT=yT_h[rows], traj=traj.float().cpu().numpy()[:, rows], a0=a0.cpu().numpy()[rows], g=g.cpu().numpy(), log=log,
               a0_rest=np.delete(a0.cpu().numpy(), rows, axis=0), stats=ctx.stats())
    ctx.close()
    # oracle on the sampled rows only, with the same cotangent
    vel, pol, tab = make_velocity(wl.vel), Policy(low=wl.low, scaling=wl.scaling), BY_NAME[wl.solver]
    aux = None if wl.probe is None else wl.probe[rows].astype(np.float64)
    otraj, oyT = odeint_forward(vel, wl.theta, wl.y0[rows], wl.tgrid, tab, pol, aux)
    oa0, og, olog = odeint_backward(vel, wl.theta, otraj, wl.tgrid, tab, pol, dl_full[rows].astype(np.float32).astype(np.float64), aux)
    tol = TOL[wl.low]
    errs = dict(yT=rel_l2(gpu["yT"], oyT), traj=rel_l2(gpu["traj"], otraj), a0=rel_l2(gpu["a0"], oa0), g=rel_l2(gpu["g"], og))
    assert all(v <= tol for v in errs.values()), errs
    assert not np.any(gpu["a0_rest"]), "rows without a cotangent must keep a zero adjoint"
    # the full-size configurations in the 16-bit formats run on the tensor cores only
    assert gpu["stats"]["simt_contractions"] == 0, gpu["stats"]
    return gpu, olog, errs


def test_c3_mlp_block_full_size_sampled_rows():
    wl = inputs.mlp_block()                                     # 8192 x 256, 64 RK4 steps, bf16: the benchmark's configuration
    _full_size_sampled(wl, [0, 127, 128, 4095, 5000, 8191])


def test_c5_cnf_full_size_sampled_rows():
    wl = inputs.cnf_mlp()                                       # 2048 x 784, 8 RK4 steps, bf16
    _full_size_sampled(wl, [0, 1, 1023, 2047])


def test_c4_conv_block_full_size_sampled_rows_and_scale_log():
    wl = inputs.conv_block()                                    # 256 images of 32 x 32 x 64, 8 RK4 steps, fp16, dynamic scaling
    import torch
    from paper_2510_23498_b200 import binding
    rows = np.array([0, 255])
    ctx = binding.Context(wl.vel, wl.batch, wl.n_steps, low=wl.low, scaling=wl.scaling)
    dev = ctx.device
    theta = torch.from_numpy(wl.theta).to(dev)
    traj, yT = ctx.forward(theta, torch.from_numpy(wl.y0).to(dev), wl.tgrid, wl.solver)
    yT_h = yT.cpu().numpy().astype(np.float64)
    _, dl_full = wl.loss(yT_h)
    dl = np.zeros_like(dl_full)
    dl[rows] = dl_full[rows]
    a0, g, log, st = ctx.backward(torch.from_numpy(dl.astype(np.float32)).to(dev))
    assert st == 0
    g_gpu, a_gpu = g.cpu().numpy(), a0.cpu().numpy()[rows]
    traj_gpu = traj.float().cpu().numpy()[:, rows]
    assert ctx.stats()["simt_contractions"] == 0 and ctx.stats()["tc_contractions"] > 0, ctx.stats()
    ctx.close()
    vel, pol, tab = make_velocity(wl.vel), Policy(low=wl.low, scaling=wl.scaling), BY_NAME[wl.solver]
    otraj, oyT = odeint_forward(vel, wl.theta, wl.y0[rows], wl.tgrid, tab, pol)
    oa0, og, olog = odeint_backward(vel, wl.theta, otraj, wl.tgrid, tab, pol, dl_full[rows].astype(np.float32).astype(np.float64))
    tol = TOL[wl.low]
    assert rel_l2(yT_h[rows], oyT) <= tol and rel_l2(traj_gpu, otraj) <= tol and rel_l2(g_gpu, og) <= tol
    # The input gradient through ReLU is kink-sensitive (see KINK_FACTOR in test_gpu_parity): an accumulation-order difference
    # flips the 0/1 derivative of a few units per layer, and over 8 steps x 4 stages those flips add up.  It is bounded by the
    # same multiple of the oracle's own sensitivity to the accumulation precision (float32 against float64 sums).
    pol32 = Policy(low=wl.low, scaling=wl.scaling, acc="f32")
    na0, _, _ = odeint_backward(vel, wl.theta, otraj, wl.tgrid, tab, pol32, dl_full[rows].astype(np.float32).astype(np.float64))
    err_a0, noise = rel_l2(a_gpu, oa0), rel_l2(na0, oa0)
    print("relu-kink case c4 full size (rows 0, 255): dL/dy0 rel. L2 GPU vs oracle %.3e, oracle f32-vs-f64 accumulation %.3e, tolerance %.1e"
          % (err_a0, noise, tol))
    from test_gpu_parity import KINK_FACTOR
    assert err_a0 <= max(tol, KINK_FACTOR * noise)
    # the adjoint of the other rows is zero, so the norm that drives the scale is that of the sampled rows: same decisions
    assert olog.margin > 1e-4
    assert log["exp_used"] == list(olog.exp_used) and log["attempts"] == list(olog.attempts) and log["doubled"] == list(olog.doubled)


# ------------------------------------------------------------------ full batch, dense cotangent: every slice of the batch-reduction counts

def _dense(wl, what=("yT", "traj", "a0", "g"), a0_minus_seed=False):
    """Both sides on the whole batch with the loss head's own (dense) terminal cotangent: every one of the batch rows that a
    weight-gradient slice sums is non-zero, so a dropped, doubled or mis-addressed slice shows in dL/dtheta."""
    from _harness import assert_parity, run_gpu, run_oracle
    orc, gpu = run_oracle(wl), run_gpu(wl)
    assert gpu["status"] == 0 and gpu["stats"]["simt_contractions"] == 0, gpu["stats"]
    if a0_minus_seed:
        gpu["a0"], orc["a0"] = gpu["a0"] - gpu["dLdyT"], orc["a0"] - orc["dLdyT"]
    errs = assert_parity(gpu, orc, TOL[wl.low], what=what)
    print("dense full-batch %s B=%d N=%d: %s" % (wl.name, wl.batch, wl.n_steps, {k: "%.2e" % v for k, v in errs.items()}))
    return gpu, orc


def test_c3_mlp_block_full_batch_dense_cotangent_two_steps():
    gpu, _ = _dense(inputs.mlp_block(n_steps=2))                # 8192 x 256, the benchmark's launch shapes, 2 RK4 steps
    assert gpu["stats"]["fused_launches"] > 0 and gpu["stats"]["tc_contractions"] == 0


def test_c5_cnf_full_batch_dense_cotangent_one_step():
    _dense(inputs.cnf_mlp(n_steps=1))                           # 2048 x 784 (+ log-density), 1 RK4 step


def test_c4_conv_block_sixteen_images_dense_cotangent_one_step():
    # 16 images of 32 x 32 x 64, one RK4 step; forward Euler as well, where dL/dy0 minus the seed isolates the convolutions
    from _harness import assert_same_log
    from test_gpu_parity import KINK_FACTOR
    wl = inputs.conv_block(batch=16, n_steps=1)
    gpu, orc = _dense(wl, what=("yT", "traj", "g"))
    assert_same_log(gpu["log"], orc["log"])
    from _harness import run_oracle
    noise = rel_l2(run_oracle(wl, acc="f32")["a0"], orc["a0"])
    err = rel_l2(gpu["a0"], orc["a0"])
    print("relu-kink case c4 16 images, 1 RK4 step: dL/dy0 rel. L2 GPU vs oracle %.3e, oracle f32-vs-f64 accumulation %.3e" % (err, noise))
    assert err <= max(TOL[wl.low], KINK_FACTOR * noise)
    _dense(inputs.conv_block(batch=16, n_steps=1, solver="euler"), a0_minus_seed=True)
