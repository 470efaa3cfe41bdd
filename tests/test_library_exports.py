"""The C-ABI shared library builds without a GPU, loads, and exports every symbol include/mpode.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "mpode.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mpode_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_header_symbols():
    from paper_2510_23498_b200 import binding, build
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = _declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), "missing export %s" % n
    assert sorted(binding.EXPORTS) == names


def test_host_only_calls_work_without_a_device():
    from paper_2510_23498_b200 import binding
    lib = binding.load_library()
    assert lib.mpode_status_string(7).decode() == "dynamic adjoint scaling failed"
    rk4 = lib.mpode_tableau_rk4().contents
    assert rk4.stages == 4 and abs(sum(rk4.b[j] for j in range(4)) - 1.0) < 1e-15
    assert [rk4.c[j] for j in range(4)] == [0.0, 0.5, 0.5, 1.0]
    assert lib.mpode_tableau_euler().contents.stages == 1
    # context creation is host-side bookkeeping: sizes can be queried without a GPU
    import ctypes as C
    widths = (C.c_int * 4)(256, 1024, 1024, 256)
    desc = binding.VelocityDesc(0, 256, 3, C.cast(widths, C.POINTER(C.c_int)), 2, 1, 1, 0, 0, 0)
    pol = binding.Policy(1, 0, 0, 0, 0, binding.NO_OVERRIDE)
    h = C.c_void_p()
    assert lib.mpode_create(C.byref(h), C.byref(desc), 8192, 64, C.byref(pol)) == 0
    assert lib.mpode_param_count(h) == 1576192                       # 257*1024+1024 + 1024*1024+1024 + 1024*256+256
    assert lib.mpode_trajectory_bytes(h, 64) == 65 * 8192 * 256 * 2
    mixed = lib.mpode_workspace_bytes(h)
    lib.mpode_destroy(h)
    pol32 = binding.Policy(0, 0, 0, 0, 0, binding.NO_OVERRIDE)
    assert lib.mpode_create(C.byref(h), C.byref(desc), 8192, 64, C.byref(pol32)) == 0
    full = lib.mpode_workspace_bytes(h) + lib.mpode_trajectory_bytes(h, 64)
    lib.mpode_destroy(h)
    # every large buffer is in the low format: mixed mode needs about half of float32 mode
    assert (mixed + 65 * 8192 * 256 * 2) / full <= 0.55
    # The whole solve also holds the caller's float32 state, adjoint, terminal cotangent, parameters and gradient, the same in
    # both modes.  With them the ratio is 0.565: a KNOWN SHORTFALL against the 0.55 target (the fused backward's second cotangent
    # slots, two extra kappa slots and the slice partial sums of the weight gradient are what exceeds one half).  Asserted so that
    # it cannot grow unnoticed; the benchmark line reports the same figure as memory.ratio with memory.target.
    caller = 3 * 8192 * 256 * 4 + 2 * 1576192 * 4
    whole = (mixed + 65 * 8192 * 256 * 2 + caller) / (full + caller)
    assert 0.55 < whole <= 0.566, whole
    bad = binding.VelocityDesc(0, 256, 3, C.cast(widths, C.POINTER(C.c_int)), 2, 1, 1, 0, 0, 0)
    bad.d = 128
    assert lib.mpode_create(C.byref(h), C.byref(bad), 8, 4, C.byref(pol)) == 1


def test_cnf_workspace_has_no_float32_cotangent_scratch_where_the_epilogue_takes_the_activation_step():
    # c5 (2048 x 784, 785 -> 2048 -> 2048 -> 784): with a batch that is a multiple of 64 and widths of at least 64 the backward
    # step through an activation runs in the tensor-core epilogue, so mixed mode plans no [2 B, 2048] float32 buffer (33.5 MB);
    # a ragged batch keeps the two-kernel form and its buffer
    import ctypes as C
    from paper_2510_23498_b200 import binding
    lib = binding.load_library()
    widths = (C.c_int * 4)(784, 2048, 2048, 784)

    def sizes(batch, low):
        desc = binding.VelocityDesc(binding.KINDS["cnf"], 784, 3, C.cast(widths, C.POINTER(C.c_int)), binding.ACTS["softplus"], 1, 1,
                                    0, 0, 0, 0, 0)
        pol = binding.Policy(low, 0, 0, 0, 0, binding.NO_OVERRIDE)
        h = C.c_void_p()
        assert lib.mpode_create(C.byref(h), C.byref(desc), batch, 8, C.byref(pol)) == 0
        out = lib.mpode_workspace_bytes(h), lib.mpode_trajectory_bytes(h, 8)
        lib.mpode_destroy(h)
        return out

    ws16, traj16 = sizes(2048, 1)
    ws32, traj32 = sizes(2048, 0)
    assert traj16 * 2 == traj32 == 9 * 2048 * 784 * 4
    assert (ws16 + traj16) / (ws32 + traj32) <= 0.52
    ragged, _ = sizes(2047, 1)
    assert ragged > ws16 + 30e6 * 2047 / 2048

