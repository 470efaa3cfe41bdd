"""B200-native mixed-precision neural-ODE time stepping (forward RK loop + scaled discrete adjoint).

The CUDA library is loaded on first use by `paper_2510_23498_b200.binding`; importing this package
alone does not need a GPU.
"""
