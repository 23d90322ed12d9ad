"""Seeded synthetic operands for the five benchmark/parity configurations.

Shared by the tests, the benchmark and the oracle-side checks; holds no step of
the method itself -- only random-number recipes.  Every array is float64 and
column-major (Fortran order), generated on the host with numpy's PCG64 so the CPU
oracle and the GPU path see bit-identical inputs.

Configurations (shape m, n, k; entry distribution; modulus set; substrate):
  1  256^3            U(-1,1)                         S  fp8   -- small, full oracle
  2  4096^3           (U(0,1)-0.5) exp(0.5 N(0,1))    S  fp8
  3  16384,16384,1024 U(-1,1); C also U(-1,1); C -= AB  E and S, fp8 (HPL trailing update, NB=1024)
  4  131072,128,4096  N(0,1)                          S  int8 and fp8 (tall/skinny block Krylov)
  5  10007,9973,5003  (U(0,1)-0.5) exp(2.0 N(0,1))    S  fp8   -- ragged, wide exponent spread
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Config:
    name: str
    m: int
    n: int
    k: int
    dist: str          # "uniform", "lognormal:<sigma>", "normal"
    seed: int
    sets: tuple        # modulus sets exercised, first is the default
    substrates: tuple  # "fp8" / "int8"
    alpha: float = 1.0
    beta: float = 0.0


CONFIGS = {
    1: Config("cfg1_256cube", 256, 256, 256, "uniform", 1001, ("S",), ("fp8",)),
    2: Config("cfg2_4096cube", 4096, 4096, 4096, "lognormal:0.5", 1002, ("S",), ("fp8",)),
    3: Config("cfg3_hpl_update_nb1024", 16384, 16384, 1024, "uniform", 1003, ("E", "S"), ("fp8",),
              alpha=-1.0, beta=1.0),
    4: Config("cfg4_tall_skinny", 131072, 128, 4096, "normal", 1004, ("S",), ("int8", "fp8")),
    5: Config("cfg5_ragged_wide", 10007, 9973, 5003, "lognormal:2.0", 1005, ("S",), ("fp8",)),
}


def _draw(rng: np.random.Generator, rows: int, cols: int, dist: str) -> np.ndarray:
    """rows x cols float64, column-major."""
    shape = (cols, rows)  # generate C-order transposed, view as F-order
    if dist == "uniform":
        x = 2.0 * rng.random(shape) - 1.0
    elif dist == "normal":
        x = rng.standard_normal(shape)
    elif dist.startswith("lognormal:"):
        sigma = float(dist.split(":")[1])
        x = (rng.random(shape) - 0.5) * np.exp(sigma * rng.standard_normal(shape))
    else:
        raise ValueError(dist)
    return x.T  # F-contiguous view, shape (rows, cols)


def operands(cfg: Config, m: int | None = None, n: int | None = None, k: int | None = None,
             want_c: bool = False):
    """A (m x k), B (k x n) [and C (m x n)] for a configuration; sizes may be cut
    down (same seed, same distribution) for oracle-sized cases."""
    m = cfg.m if m is None else m
    n = cfg.n if n is None else n
    k = cfg.k if k is None else k
    rng = np.random.default_rng(cfg.seed)
    A = _draw(rng, m, k, cfg.dist)
    B = _draw(rng, k, n, cfg.dist)
    if want_c:
        Cm = _draw(rng, m, n, "uniform")
        return A, B, Cm
    return A, B


def special_operands(kind: str, m: int, n: int, k: int, seed: int = 7):
    """Edge-case operands: exact small integers, zeros, subnormals, huge single entries."""
    rng = np.random.default_rng(seed)
    if kind == "small_integers":
        A = rng.integers(-2**20, 2**20, size=(k, m)).astype(np.float64).T
        B = rng.integers(-2**20, 2**20, size=(n, k)).astype(np.float64).T
    elif kind == "zero_lines":
        A = _draw(rng, m, k, "uniform")
        B = _draw(rng, k, n, "uniform")
        A[m // 2, :] = 0.0
        B[:, n // 3] = 0.0
        A[0, :] = -0.0
    elif kind == "subnormal":
        A = _draw(rng, m, k, "uniform") * 2.0**-1040
        B = _draw(rng, k, n, "uniform")
        A[1, :] *= 2.0**-30  # deep subnormals / underflow to zero
    elif kind == "spike":
        A = _draw(rng, m, k, "uniform")
        B = _draw(rng, k, n, "uniform")
        A[0, k // 2] = 3.0e40
        B[k // 3, 0] = -7.0e-35
    else:
        raise ValueError(kind)
    return np.asfortranarray(A), np.asfortranarray(B)
