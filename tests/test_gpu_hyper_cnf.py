"""GPU parity of the two-dimensional flows of Sec. 6.1 with the exact trace (MPODE_VEL_CNF_HYPER) through the C ABI.

Tolerances are those of the other parity tests: relative L2 at most 1e-5 in float32 mode against the exact fp64 discrete
solution and its exact discrete adjoint, 1e-2 (bfloat16) / 2e-3 (float16) against the rounding-emulating oracle, scale log
identical under dynamic scaling.
"""
import numpy as np
import pytest

from paper_2510_23498_b200 import inputs
from _harness import TOL, assert_parity, assert_same_log, run_gpu, run_oracle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("batch,n_steps,hidden,w", [(100, 6, 8, 16), (300, 4, 32, 128)])
def test_hyper_cnf_float32_mode_against_the_exact_discrete_adjoint(batch, n_steps, hidden, w):
    wl = inputs.hyper_cnf(batch=batch, n_steps=n_steps, hidden=hidden, w=w)
    orc = run_oracle(wl, exact=True)
    gpu = run_gpu(wl, "f32", "none")
    assert_parity(gpu, orc, TOL["f32"])
    assert gpu["yT"].shape == (batch, 3) and np.any(gpu["yT"][:, 2] != 0)       # the log-density column is integrated


@pytest.mark.parametrize("low,scaling", [("f16", "dynamic"), ("bf16", "none"), ("f16", "none_safe")])
def test_hyper_cnf_mixed_precision_against_the_emulating_oracle(low, scaling):
    wl = inputs.hyper_cnf(batch=300, n_steps=5, hidden=32, w=128)
    orc = run_oracle(wl, low, scaling)
    gpu = run_gpu(wl, low, scaling)
    assert gpu["status"] == 0
    assert_parity(gpu, orc, TOL[low])
    if scaling == "dynamic":
        assert orc["log"].margin > 1e-4
        assert_same_log(gpu["log"], orc["log"])


def test_hyper_cnf_forced_overflow_gives_the_oracles_retry_sequence_and_other_tableaux_work():
    wl = inputs.hyper_cnf(batch=130, n_steps=4, hidden=16, w=32)
    orc = run_oracle(wl, "f16", "dynamic", k_max=40, init_scale_exp_override=30)
    gpu = run_gpu(wl, "f16", "dynamic", k_max=40, init_scale_exp_override=30)
    assert_parity(gpu, orc, TOL["f16"])
    assert_same_log(gpu["log"], orc["log"])
    assert max(gpu["log"]["attempts"]) > 1
    wl.solver = "heun"
    wl.tgrid = np.array([0.0, 0.15, 0.4, 0.8, 1.0], dtype=np.float32)
    assert_parity(run_gpu(wl, "f32", "none"), run_oracle(wl, exact=True), TOL["f32"])


def test_hyper_cnf_other_state_widths_take_the_general_kernels():
    wl = inputs.hyper_cnf(batch=70, n_steps=3, d=3, hidden=8, w=24)
    assert_parity(run_gpu(wl, "f32", "none"), run_oracle(wl, exact=True), TOL["f32"])
    gpu, orc = run_gpu(wl, "bf16", "none"), run_oracle(wl, "bf16", "none")
    assert_parity(gpu, orc, TOL["bf16"])


def test_hyper_cnf_wide_hypernetwork_output_goes_stage_by_stage_and_euler_takes_the_step_kernels():
    # 400 weight sets of a four-dimensional state: one stage's sets fit shared memory, four stages' do not, so every stage is a
    # launch of its own; both paths give the same numbers as the oracle
    wl = inputs.hyper_cnf(batch=50, n_steps=3, d=4, hidden=8, w=400)
    assert_parity(run_gpu(wl, "f32", "none"), run_oracle(wl, exact=True), TOL["f32"])
    gpu, orc = run_gpu(wl, "f16", "dynamic"), run_oracle(wl, "f16", "dynamic")
    assert_parity(gpu, orc, TOL["f16"])
    assert_same_log(gpu["log"], orc["log"])
    wl = inputs.hyper_cnf(batch=90, n_steps=7, hidden=16, w=64)
    wl.solver = "euler"
    gpu, orc = run_gpu(wl, "f16", "dynamic"), run_oracle(wl, "f16", "dynamic")
    assert_parity(gpu, orc, TOL["f16"])
    assert_same_log(gpu["log"], orc["log"])


def test_hyper_cnf_full_size():
    # the paper's setting: batch 1024, RK4 with 128 steps; the oracle runs all of it (the state is two-dimensional)
    wl = inputs.hyper_cnf()
    orc = run_oracle(wl)
    gpu = run_gpu(wl)
    assert gpu["status"] == 0
    assert_parity(gpu, orc, TOL[wl.low])
    assert_same_log(gpu["log"], orc["log"])
