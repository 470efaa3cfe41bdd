"""GPU parity of the remaining outputs of Alg. 2: the time-grid gradient dL/dt (the dt, dh entries of Eq. (vjp) and the two t'
updates) and the running-cost cotangents w_i dR/dy_i of the adjoint update, through mpode_backward_ex.

Tolerances are those of the other parity tests (relative L2: 1e-5 in float32 mode against the exact fp64 discrete adjoint,
1e-2 bfloat16 / 2e-3 float16 against the rounding-emulating oracle); the scale log must be identical.
"""
import numpy as np
import pytest

from paper_2510_23498_b200 import inputs
from _harness import TOL, assert_parity, assert_same_log, rel_l2, run_gpu, run_oracle

pytestmark = pytest.mark.gpu


def _running_cot(wl, D, seed=3, scale=None):
    """A synthetic running cost sum_{i<N} <c_i, y_i> with seeded weights of the size of the terminal cotangent."""
    rng = np.random.default_rng(seed)
    s = scale if scale is not None else 1.0 / (wl.batch * D)
    return (s * rng.standard_normal((wl.n_steps, wl.batch, D))).astype(np.float32)


def _check(wl, low, scaling, cot=True, exact=False, **kw):
    D = wl.vel["d"] + (1 if wl.vel["kind"] == "cnf" else 0)
    rc = _running_cot(wl, D) if cot else None
    if exact:
        orc = run_oracle(wl, exact=True, want_dt=True, running_cot=rc)
        gpu = run_gpu(wl, "f32", "none", want_dt=True, running_cot=rc, **kw)
        tol = TOL["f32"]
    else:
        orc = run_oracle(wl, low, scaling, want_dt=True, running_cot=rc, **kw)
        gpu = run_gpu(wl, low, scaling, want_dt=True, running_cot=rc, **kw)
        tol = TOL[low]
    errs = assert_parity(gpu, orc, tol)
    errs["dL_dt"] = rel_l2(gpu["dL_dt"], orc["dL_dt"])
    assert errs["dL_dt"] <= tol, errs
    if not exact and scaling == "dynamic":
        assert orc["log"].margin > 1e-4
        assert_same_log(gpu["log"], orc["log"])
    return gpu, orc, errs


@pytest.mark.parametrize("low,scaling", [("f16", "dynamic"), ("bf16", "none")])
def test_toy_mlp_whole_solve_kernel_time_gradient_and_running_cost(low, scaling):
    gpu, _, _ = _check(inputs.toy_mlp(batch=100, n_steps=6, hidden=20), low, scaling)
    assert gpu["stats"]["whole_solve_launches"] == 2


def test_toy_mlp_float32_mode_against_the_exact_discrete_adjoint():
    wl = inputs.toy_mlp(batch=64, n_steps=5, hidden=16)
    wl.solver = "rk38"
    wl.tgrid = np.array([0.0, 0.1, 0.35, 0.5, 0.8, 1.0], dtype=np.float32)
    _check(wl, "f32", "none", exact=True)


@pytest.mark.parametrize("batch,d,hidden,n_steps", [(200, 256, 1024, 2), (130, 72, 200, 3)])
def test_mlp_block_fused_path_time_gradient_and_running_cost(batch, d, hidden, n_steps):
    wl = inputs.mlp_block(batch=batch, n_steps=n_steps, d=d, hidden=hidden)
    gpu, _, _ = _check(wl, "bf16", "none")
    assert gpu["stats"]["fused_launches"] > 0 and gpu["stats"]["simt_contractions"] == 0


def test_mlp_block_layer_by_layer_paths_time_gradient():
    wl = inputs.mlp_block(batch=96, n_steps=3, d=64, hidden=160)
    _check(wl, "f16", "dynamic")                       # fused kernels, finiteness test extended by Q16(dt), Q16(dh)
    wl.solver = "kutta3"
    wl.tgrid = np.array([0.0, 0.2, 0.55, 1.0], dtype=np.float32)
    _check(wl, "f32", "none", exact=True)              # CUDA-core float32 path, another tableau, non-uniform grid


def test_scalar_example_time_gradient_matches_oracle_and_the_analytic_end_point_derivative():
    wl = inputs.scalar_example(batch=3)
    orc = run_oracle(wl, "f16", "dynamic", want_dt=True)
    gpu = run_gpu(wl, "f16", "dynamic", dLdyT=orc["dLdyT"], want_dt=True)
    assert orc["log"].margin > 1e-4
    assert_same_log(gpu["log"], orc["log"])
    assert_parity(gpu, orc, TOL["f16"], what=("yT", "traj", "a0", "g"))
    assert rel_l2(gpu["dL_dt"], orc["dL_dt"]) <= TOL["f16"]
    # float32 mode: dL/dT = -lambda(T) y_N^2 summed over the samples (Example 1 with L = sum y_N^2 / 2), up to RK4's error
    g32 = run_gpu(wl, "f32", "none", want_dt=True)
    th, T = wl.theta.astype(np.float64), 2.65
    lamT = th[0] * T * T + th[1] * T + th[2]
    ref = -lamT * float(np.sum(g32["yT"] ** 2))
    assert abs(g32["dL_dt"][-1] - ref) <= 2e-3 * abs(ref)


def test_running_cost_on_the_convolution_and_cnf_paths():
    # the adjoint update's w_i dR/dy_i term; these velocities have no time-grid gradient
    for wl in (inputs.conv_block(batch=2, n_steps=2, H=8, W=8, C=16, act="softplus"), inputs.cnf_mlp(batch=24, n_steps=2, d=16, hidden=32)):
        D = wl.vel["d"] + (1 if wl.vel["kind"] == "cnf" else 0)
        rc = _running_cot(wl, D)
        orc = run_oracle(wl, running_cot=rc)
        gpu = run_gpu(wl, running_cot=rc)
        assert_parity(gpu, orc, TOL[wl.low])
        base = run_gpu(wl)
        assert not np.array_equal(base["a0"], gpu["a0"])
        if wl.scaling == "dynamic":
            assert_same_log(gpu["log"], orc["log"])


def test_time_gradient_is_refused_where_it_is_not_built_and_leaves_the_other_outputs_alone():
    import torch
    from paper_2510_23498_b200 import binding
    with pytest.raises(binding.MpodeError) as ei:
        binding.Context(inputs.conv_block(batch=2, n_steps=1, H=8, W=8, C=16).vel, 2, 1, low="f16", time_gradient=True)
    assert ei.value.status == binding.ERR_UNSUPPORTED
    wl = inputs.mlp_block(batch=80, n_steps=2, d=32, hidden=96)
    ctx = binding.Context(wl.vel, wl.batch, wl.n_steps, low="bf16")
    theta, y0 = torch.from_numpy(wl.theta).cuda(), torch.from_numpy(wl.y0).cuda()
    _, yT = ctx.forward(theta, y0, wl.tgrid, wl.solver)
    with pytest.raises(binding.MpodeError) as ei:                      # context without policy.time_gradient
        ctx.backward(torch.ones_like(yT), want_dt=True)
    assert ei.value.status == binding.ERR_INVALID_ARG
    ctx.close()
    plain, with_dt = run_gpu(wl), run_gpu(wl, want_dt=True)
    assert np.array_equal(plain["g"], with_dt["g"]) and np.array_equal(plain["a0"], with_dt["a0"])
