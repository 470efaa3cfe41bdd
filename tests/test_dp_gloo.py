"""The multi-rank path of the benchmark on CPU: two gloo ranks shard the batch, run the oracle on their rows and sum
dL/dtheta with one all-reduce; the result must equal the single-process gradient, and dL/dy0 the matching rows."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import BY_NAME, Policy, make_velocity, odeint_backward, odeint_forward
    from paper_2510_23498_b200 import dp, inputs
    wl = inputs.mlp_block(batch=11, n_steps=3, d=8, hidden=16)
    lo, hi = dp.shard_rows(wl.batch, rank, world)
    vel, pol, tab = make_velocity(wl.vel), Policy(low="bf16"), BY_NAME["rk4"]
    traj, yT = odeint_forward(vel, wl.theta, wl.y0[lo:hi], wl.tgrid, tab, pol)
    # loss = mean over the GLOBAL batch: the local cotangent carries 1 / (B_global d)
    target = wl.extra["target"][lo:hi]
    dl = 2.0 * (yT - target) / (wl.batch * wl.vel["d"])
    a0, g, _ = odeint_backward(vel, wl.theta, traj, wl.tgrid, tab, pol, dl)
    gt = torch.from_numpy(g.copy())
    dp.allreduce_sum_(gt, world)
    tmax = dp.allreduce_max_float(1.0 + rank, world)
    if rank == 0:
        np.save(out, np.concatenate([gt.numpy(), [tmax, lo, hi]]))
    np.save(out + ".a%d.npy" % rank, a0)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_single_process_gradient(tmp_path):
    sys.path.insert(0, ROOT)
    from oracle import BY_NAME, Policy, make_velocity, odeint_backward, odeint_forward
    from paper_2510_23498_b200 import dp, inputs
    assert [dp.shard_rows(11, r, 2) for r in range(2)] == [(0, 6), (6, 11)]
    assert [dp.shard_rows(8, r, 4) for r in range(4)] == [(0, 2), (2, 4), (4, 6), (6, 8)]
    out = str(tmp_path / "g.npy")
    mp.spawn(_worker, args=(2, 29517 + os.getpid() % 1000, out), nprocs=2, join=True)
    got = np.load(out)
    wl = inputs.mlp_block(batch=11, n_steps=3, d=8, hidden=16)
    vel, pol, tab = make_velocity(wl.vel), Policy(low="bf16"), BY_NAME["rk4"]
    traj, yT = odeint_forward(vel, wl.theta, wl.y0, wl.tgrid, tab, pol)
    _, dl = wl.loss(yT)
    a_ref, g_ref, _ = odeint_backward(vel, wl.theta, traj, wl.tgrid, tab, pol, dl)
    g = got[:-3]
    assert got[-3] == 2.0                                   # max over ranks of the per-rank time stand-in
    assert np.linalg.norm(g - g_ref) <= 1e-6 * np.linalg.norm(g_ref)
    a = np.concatenate([np.load(out + ".a%d.npy" % r) for r in range(2)])
    assert np.linalg.norm(a - a_ref) <= 1e-6 * np.linalg.norm(a_ref)   # fp32-accumulated sums in a different order
