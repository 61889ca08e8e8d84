"""Seeded synthetic inputs and the named workload configurations.

This module holds no Jacobi arithmetic.  It only produces the arrays (initial guess,
right-hand side, boundary values) that both the GPU library and the CPU checker are
given, so that neither side's result can depend on how the other draws its data.

Dense arrays are numpy float64 with shape (ny, nx) or (nz, ny, nx): the last axis is x.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


@dataclass(frozen=True)
class Workload:
    """One named problem: grid, decomposition, data recipe and the work to run on it."""
    name: str
    n: tuple            # global interior points (x, y[, z])
    b: tuple            # block interior points (x, y[, z])
    halo: int
    sweeps: int
    residual_every: int  # 0: only after the last sweep
    u0: str             # "zero" | "sine"
    f: str              # "none" | "uniform" | "normal"
    seed: int
    bvals: tuple = field(default=())  # Dirichlet value per face (-x,+x,-y,+y[,-z,+z]); () = all 0

    @property
    def ndim(self) -> int:
        return len(self.n)

    @property
    def has_f(self) -> bool:
        return self.f != "none"

    @property
    def points(self) -> int:
        return int(np.prod([int(x) for x in self.n], dtype=np.int64))

    @property
    def bytes_per_point(self) -> int:
        """Compulsory traffic of one sweep: read u, write u', plus read f where present."""
        return 24 if self.has_f else 16

    def boundary(self):
        return list(self.bvals) if self.bvals else [0.0] * (2 * self.ndim)


# The five configurations the library is measured and checked on.
HEATED_EDGE_256 = Workload("c1_heated_edge_256", (256, 256), (256, 256), 1, 100, 0,
                           "zero", "none", 0, (0.0, 0.0, 0.0, 1.0))
POISSON_4096 = Workload("c2_poisson_4096", (4096, 4096), (512, 512), 1, 1000, 10,
                        "zero", "uniform", 1)
EIGENMODE_16384 = Workload("c3_eigenmode_16384", (16384, 16384), (1024, 1024), 1, 200, 0,
                           "sine", "none", 0)
POISSON3D_1024 = Workload("c5_poisson3d_1024", (1024, 1024, 1024), (128, 128, 128), 1, 50, 10,
                          "zero", "normal", 3)
# The one domain shape the paper states (Section V-C, strong scaling): 1024 x 1024 x 768, here in
# 128^3 blocks with the recipe of POISSON3D_1024.  Context, not one of the five configurations.
PAPER_DOMAIN_1024x1024x768 = Workload("paper_domain_1024x1024x768", (1024, 1024, 768), (128, 128, 128), 1,
                                      50, 10, "zero", "normal", 3)
CONFIGS = {w.name: w for w in (HEATED_EDGE_256, POISSON_4096, EIGENMODE_16384, POISSON3D_1024,
                               PAPER_DOMAIN_1024x1024x768)}

# Halo pack/unpack microbenchmark: block edge B -> block grid G x G, so that every kind
# of face has interior instances; halo widths 1 and 4; data Uniform[-1,1], seed 2.
HALO_BENCH_SHAPES = {64: 64, 256: 32, 1024: 8, 4096: 4}
HALO_BENCH_WIDTHS = (1, 4)
HALO_BENCH_SEED = 2


def scaled(w: Workload, n, b=None, sweeps=None, name=None) -> Workload:
    """Same recipe on a smaller grid (parity cases the CPU checker finishes in seconds)."""
    return Workload(name or f"{w.name}_scaled", tuple(n), tuple(b or w.b), w.halo,
                    w.sweeps if sweeps is None else sweeps, w.residual_every, w.u0, w.f,
                    w.seed, w.bvals)


def _dense_shape(n):
    return tuple(int(x) for x in reversed(n))


def sine_mode(n, lo=None, hi=None, modes=None) -> np.ndarray:
    """prod_a sin(pi * m_a * i_a / (n_a + 1)) on 1-based interior indices, restricted to the
    0-based half-open box [lo, hi)."""
    ndim = len(n)
    lo = [0] * ndim if lo is None else lo
    hi = list(n) if hi is None else hi
    modes = [1] * ndim if modes is None else modes
    out = None
    for a in range(ndim):
        idx = np.arange(lo[a] + 1, hi[a] + 1, dtype=np.float64)
        s = np.sin(np.pi * modes[a] * idx / (n[a] + 1))
        shape = [1] * ndim
        shape[ndim - 1 - a] = s.size
        s = s.reshape(shape)
        out = s if out is None else out * s
    return np.ascontiguousarray(out)


def initial_u(w: Workload) -> np.ndarray:
    if w.u0 == "zero":
        return np.zeros(_dense_shape(w.n), dtype=np.float64)
    if w.u0 == "sine":
        return sine_mode(w.n)
    raise ValueError(w.u0)


def rhs(w: Workload):
    """Right-hand side drawn once, in dense x-fastest order, from numpy's default_rng(seed)."""
    if w.f == "none":
        return None
    rng = np.random.default_rng(w.seed)
    if w.f == "uniform":
        return rng.uniform(-1.0, 1.0, w.points).reshape(_dense_shape(w.n))
    if w.f == "normal":
        return rng.standard_normal(w.points).reshape(_dense_shape(w.n))
    raise ValueError(w.f)


def uniform_field(n, seed: int) -> np.ndarray:
    """Uniform[-1,1] values over a dense grid (halo microbenchmark data)."""
    rng = np.random.default_rng(seed)
    return rng.uniform(-1.0, 1.0, int(np.prod(n))).reshape(_dense_shape(n))


def linear_index_field(n) -> np.ndarray:
    """u = global linear index: any misplaced element of a pack/unpack is visible."""
    return np.arange(int(np.prod(n)), dtype=np.float64).reshape(_dense_shape(n))
