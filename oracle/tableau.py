"""Explicit Runge-Kutta tableaux: the increment functions Phi of Sec. 3.

TEST INFRASTRUCTURE ONLY (CPU oracle); shares no code with the CUDA path.

The paper's scheme is y_{i+1} = y_i + h_i Phi(f, y_i, t_i, h_i, theta) for an
explicit single-step method; it names forward Euler (Phi = f(t_i, y_i)) and
the classic fourth-order Runge-Kutta method (Sec. 3, Sec. 5).  In tableau
form Phi = sum_j b_j k_j with k_j = f(t_i + c_j h, y_i + h sum_{l<j} a_jl k_l).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Tableau:
    name: str
    a: np.ndarray  # [s, s], strictly lower triangular
    b: np.ndarray  # [s]
    c: np.ndarray  # [s]

    @property
    def stages(self) -> int:
        return int(self.b.shape[0])


def _mk(name, a, b, c) -> Tableau:
    a = np.array(a, dtype=np.float64)
    assert np.allclose(np.triu(a), 0.0), "explicit tableau must be strictly lower triangular"
    return Tableau(name, a, np.array(b, dtype=np.float64), np.array(c, dtype=np.float64))


EULER = _mk("euler", [[0.0]], [1.0], [0.0])
MIDPOINT = _mk("midpoint", [[0, 0], [0.5, 0]], [0.0, 1.0], [0.0, 0.5])
HEUN = _mk("heun", [[0, 0], [1.0, 0]], [0.5, 0.5], [0.0, 1.0])
KUTTA3 = _mk("kutta3", [[0, 0, 0], [0.5, 0, 0], [-1.0, 2.0, 0]], [1 / 6, 2 / 3, 1 / 6], [0.0, 0.5, 1.0])
RK4 = _mk("rk4", [[0, 0, 0, 0], [0.5, 0, 0, 0], [0, 0.5, 0, 0], [0, 0, 1.0, 0]],
          [1 / 6, 1 / 3, 1 / 3, 1 / 6], [0.0, 0.5, 0.5, 1.0])
RK38 = _mk("rk38", [[0, 0, 0, 0], [1 / 3, 0, 0, 0], [-1 / 3, 1.0, 0, 0], [1.0, -1.0, 1.0, 0]],
           [1 / 8, 3 / 8, 3 / 8, 1 / 8], [0.0, 1 / 3, 2 / 3, 1.0])

BY_NAME = {t.name: t for t in (EULER, MIDPOINT, HEUN, KUTTA3, RK4, RK38)}
