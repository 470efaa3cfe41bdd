"""CPU oracle for the mixed-precision neural-ODE time loop (Alg. 1 and Alg. 2).

TEST INFRASTRUCTURE ONLY: plain numpy in fp64 with emulated 16-bit rounding.
Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this package; the CUDA path never does, and the two share no code.
"""
from .quantize import quantize, precision_bits, max_finite          # noqa: F401
from .tableau import Tableau, EULER, RK4, BY_NAME                    # noqa: F401
from .velocity import make_velocity                                  # noqa: F401
from .odeint import Policy, ScaleLog, odeint_forward, odeint_backward, initial_scale_exponent  # noqa: F401
