"""The backward pass on the library's static device workspace (mpode_backward_static_workspace).

That entry point exists for callers that cannot allocate device memory when they need a gradient (a host framework
whose allocator is locked during its step, a real-time loop, a process with a fixed memory budget).  It must give
what mpode_backward gives on a caller-provided workspace.  The static array is shared by every call and keeps the
previous call's contents, so the check is made on two calls in a row, the second one after another context has
dirtied the array.  This file is collected last on purpose: a run that stops at the first failure has then run every
other test already.
"""
import numpy as np
import pytest

from paper_2510_23498_b200 import inputs
from _harness import TOL, rel_l2

pytestmark = pytest.mark.gpu


def _forward_and_reference(wl):
    import torch
    from paper_2510_23498_b200 import binding
    ctx = binding.Context(wl.vel, wl.batch, wl.n_steps, low=wl.low, scaling=wl.scaling)
    assert ctx.workspace_bytes <= binding.STATIC_WORKSPACE_BYTES
    theta = torch.from_numpy(wl.theta).to(ctx.device)
    y0 = torch.from_numpy(wl.y0).to(ctx.device)
    _, yT = ctx.forward(theta, y0, wl.tgrid, wl.solver)
    _, dl = wl.loss(yT.cpu().numpy().astype(np.float64))
    dl = torch.from_numpy(dl.astype(np.float32)).to(ctx.device)
    a0, g, _, st = ctx.backward(dl)
    assert st == 0
    return ctx, dl, a0.cpu().numpy(), g.cpu().numpy(), (theta, y0)


def test_static_workspace_backward_matches_backward_on_two_calls_in_a_row():
    import torch
    from paper_2510_23498_b200 import binding
    wl = inputs.mlp_block(batch=200, n_steps=3, d=64, hidden=128)                    # fused tensor-core path, bf16
    wl2 = inputs.toy_mlp(batch=64, n_steps=4, hidden=16)                             # fp16, dynamic adjoint scaling
    ctx, dl, a_ref, g_ref, keep = _forward_and_reference(wl)
    ctx2, dl2, a_ref2, g_ref2, keep2 = _forward_and_reference(wl2)
    for call in range(2):
        a0, g, st = ctx.backward_static_workspace(dl)
        torch.cuda.synchronize()
        assert st == 0
        assert rel_l2(a0.cpu().numpy(), a_ref) <= TOL[wl.low] and rel_l2(g.cpu().numpy(), g_ref) <= TOL[wl.low], call
        # another context now leaves its own contents in the shared array
        b0, h, st2 = ctx2.backward_static_workspace(dl2)
        torch.cuda.synchronize()
        assert st2 == 0
        assert rel_l2(b0.cpu().numpy(), a_ref2) <= TOL[wl2.low] and rel_l2(h.cpu().numpy(), g_ref2) <= TOL[wl2.low], call
    ctx.close()
    ctx2.close()


def test_static_workspace_backward_allocates_no_device_memory_and_keeps_the_scale_log():
    # What the entry point is for: between two reads of the device's free memory, a call with preallocated outputs must not
    # change it.  One warm-up call comes first, because the CUDA runtime may load a kernel's code at its first launch.
    # The dynamic-scaling context also passes a scale log (it must equal mpode_backward's) and accumulates into a gradient.
    import ctypes as C
    import torch
    wl = inputs.toy_mlp(batch=64, n_steps=4, hidden=16)                              # fp16, dynamic adjoint scaling
    wl2 = inputs.mlp_block(batch=200, n_steps=3, d=64, hidden=128)                   # fused tensor-core path, bf16
    for w in (wl, wl2):
        ctx, dl, a_ref, g_ref, keep = _forward_and_reference(w)
        _, _, log_ref, _ = ctx.backward(dl)
        n = w.n_steps
        a0 = torch.empty((w.batch, ctx.D), dtype=torch.float32, device=ctx.device)
        g = torch.empty(ctx.p, dtype=torch.float32, device=ctx.device)
        arrays = ((C.c_int * n)(), (C.c_int * n)(), (C.c_ubyte * n)())
        ctx.backward_static_workspace(dl, out_a0=a0, out_g=g, log_arrays=arrays)     # warm-up: kernels loaded, address looked up
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        _, _, st = ctx.backward_static_workspace(dl, out_a0=a0, out_g=g, log_arrays=arrays)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert st == 0 and free1 == free0, (free0, free1)
        assert rel_l2(a0.cpu().numpy(), a_ref) <= TOL[w.low] and rel_l2(g.cpu().numpy(), g_ref) <= TOL[w.low]
        assert list(arrays[0]) == log_ref["exp_used"] and list(arrays[1]) == log_ref["attempts"]
        assert [int(x) for x in arrays[2]] == log_ref["doubled"]
        g.fill_(3.0)
        ctx.backward_static_workspace(dl, out_a0=a0, out_g=g, accumulate=True, log_arrays=arrays)
        torch.cuda.synchronize()
        assert np.allclose(g.cpu().numpy(), g_ref + 3.0, rtol=1e-5, atol=1e-6)
        ctx.close()


def test_static_workspace_dynamic_scaling_without_the_mapped_state_words():
    # Fused / layer-by-layer kernels (not the whole-solve kernel) under dynamic scaling with overflowing attempts.  A context
    # whose only backward calls go through this entry point has no mapped copy of the device's scale state (creating it would
    # allocate) and reads the decisions back after every step; the result and the scale log are those of mpode_backward.
    import ctypes as C
    import torch
    from paper_2510_23498_b200 import binding
    wl = inputs.mlp_block(batch=130, n_steps=3, d=72, hidden=200)
    kw = dict(low="f16", scaling="dynamic", k_max=40, init_scale_exp_override=24)
    outs = []
    for static in (False, True):
        ctx = binding.Context(wl.vel, wl.batch, wl.n_steps, **kw)
        assert ctx.workspace_bytes <= binding.STATIC_WORKSPACE_BYTES
        theta, y0 = torch.from_numpy(wl.theta).to(ctx.device), torch.from_numpy(wl.y0).to(ctx.device)
        _, yT = ctx.forward(theta, y0, wl.tgrid, wl.solver)
        _, dl = wl.loss(yT.cpu().numpy().astype(np.float64))
        dl = torch.from_numpy(dl.astype(np.float32)).to(ctx.device)
        if static:
            n = wl.n_steps
            arrays = ((C.c_int * n)(), (C.c_int * n)(), (C.c_ubyte * n)())
            a0, g, st = ctx.backward_static_workspace(dl, log_arrays=arrays)
            log = dict(exp_used=list(arrays[0]), attempts=list(arrays[1]), doubled=[int(x) for x in arrays[2]])
        else:
            a0, g, log, st = ctx.backward(dl)
        torch.cuda.synchronize()
        assert st == 0
        outs.append((a0.cpu().numpy(), g.cpu().numpy(), log, ctx.stats()))
        ctx.close()
    (a_ref, g_ref, log_ref, st_ref), (a_s, g_s, log_s, st_s) = outs
    assert np.array_equal(a_ref, a_s) and np.array_equal(g_ref, g_s)
    assert all(log_ref[k] == log_s[k] for k in ("exp_used", "attempts", "doubled")) and max(log_s["attempts"]) > 1
    assert st_ref["step_waits"] > 0 and st_s["step_waits"] == 0 and st_s["host_syncs"] >= wl.n_steps + st_s["retries"]


def test_static_workspace_refuses_invalid_calls_before_queueing_work():
    import torch
    from paper_2510_23498_b200 import binding
    wl = inputs.toy_mlp(batch=64, n_steps=4, hidden=16)
    ctx = binding.Context(wl.vel, wl.batch, wl.n_steps, low=wl.low, scaling=wl.scaling)
    with pytest.raises(binding.MpodeError) as ei:                                    # no forward pass yet
        ctx.backward_static_workspace(torch.zeros((wl.batch, ctx.D), device=ctx.device))
    assert ei.value.status == binding.ERR_BAD_STATE
    theta, y0 = torch.from_numpy(wl.theta).to(ctx.device), torch.from_numpy(wl.y0).to(ctx.device)
    ctx.forward(theta, y0, wl.tgrid, wl.solver)
    host = torch.zeros((wl.batch, ctx.D)).pin_memory()                               # not device memory
    with pytest.raises(binding.MpodeError) as ei:
        ctx.backward_static_workspace(host)
    assert ei.value.status == binding.ERR_INVALID_ARG
    ctx.close()


def test_static_workspace_rejects_contexts_that_need_more_than_it_holds():
    import torch
    from paper_2510_23498_b200 import binding
    wl = inputs.mlp_block(batch=4096, n_steps=1, d=256, hidden=1024)
    ctx = binding.Context(wl.vel, wl.batch, wl.n_steps, low=wl.low, scaling=wl.scaling)
    assert ctx.workspace_bytes > binding.STATIC_WORKSPACE_BYTES
    theta = torch.from_numpy(wl.theta).to(ctx.device)
    y0 = torch.from_numpy(wl.y0).to(ctx.device)
    _, yT = ctx.forward(theta, y0, wl.tgrid, wl.solver)
    with pytest.raises(binding.MpodeError) as ei:
        ctx.backward_static_workspace(torch.ones_like(yT))
    assert ei.value.status == binding.ERR_WORKSPACE_TOO_SMALL and "static workspace" in str(ei.value)
    ctx.close()
