"""Pins for the oracle's sweep: closed forms, exact rational arithmetic on the textbook
matrix form, path enumeration, and invariants.  None of these re-types the oracle's
formula; each would fail on a dropped term, a wrong sign, a wrong constant or a
transposed operand."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

from paper_2210_01238_b200 import inputs

EPS = np.finfo(np.float64).eps


# ---------------------------------------------------------------- eigenmodes
@pytest.mark.parametrize("n,modes", [((7, 7), (1, 1)), ((16, 9), (1, 1)), ((31, 17), (2, 3)),
                                     ((5, 12), (5, 1)), ((256, 256), (1, 1))])
def test_eigenmode_2d_decays_by_lambda(orc, n, modes):
    """u0 = sin*sin is an eigenvector of the Jacobi iteration matrix with eigenvalue
    (cos(pi mx/(nx+1)) + cos(pi my/(ny+1)))/2, so k sweeps multiply it by lambda^k."""
    lam = sum(math.cos(math.pi * m / (nn + 1)) for m, nn in zip(modes, n)) / 2.0
    u0 = inputs.sine_mode(n, modes=modes)
    u = orc.mono_padded(n)
    u[1:-1, 1:-1] = u0
    k = 25
    got = orc.mono_sweep(u, None, k)[1:-1, 1:-1]
    want = (lam ** k) * u0
    assert np.max(np.abs(got - want)) <= 8 * k * EPS
    # sharper: one sweep, relative to lambda
    got1 = orc.mono_sweep(u, None, 1)[1:-1, 1:-1]
    assert np.max(np.abs(got1 - lam * u0)) <= 6 * EPS


@pytest.mark.parametrize("n,modes", [((5, 7, 3), (1, 1, 1)), ((8, 4, 6), (2, 1, 3)),
                                     ((3, 9, 5), (1, 4, 2))])
def test_eigenmode_3d_decays_by_lambda(orc, n, modes):
    """3D: eigenvalue (cos_x + cos_y + cos_z)/3; unequal sides and modes catch axis mix-ups."""
    lam = sum(math.cos(math.pi * m / (nn + 1)) for m, nn in zip(modes, n)) / 3.0
    u0 = inputs.sine_mode(n, modes=modes)
    u = orc.mono_padded(n)
    u[1:-1, 1:-1, 1:-1] = u0
    k = 20
    got = orc.mono_sweep(u, None, k)[1:-1, 1:-1, 1:-1]
    assert np.max(np.abs(got - (lam ** k) * u0)) <= 10 * k * EPS


# ------------------------------------------- exact rationals, textbook matrix form
def _lap1d(m):
    a = [[Fraction(0)] * m for _ in range(m)]
    for i in range(m):
        a[i][i] = Fraction(2)
        if i:
            a[i][i - 1] = Fraction(-1)
        if i + 1 < m:
            a[i][i + 1] = Fraction(-1)
    return a


def _exact_jacobi_step(n, u, f, bvals):
    """x' = x + D^-1 (b - A x) for A = the (2d+1)-point negative Laplacian assembled as a
    Kronecker sum of 1-D tridiag(-1, 2, -1) matrices; b = f + Dirichlet contributions.
    Everything in exact rationals; u, f indexed [(z,) y, x] as nested python lists."""
    ndim = len(n)
    pts = list(itertools.product(*[range(m) for m in reversed(n)]))  # (z,) y, x tuples
    L = [_lap1d(m) for m in n]  # per axis x, y, z

    def get(arr, p):
        for q in p:
            arr = arr[q]
        return arr

    out = {}
    diag = Fraction(2 * ndim)
    for p in pts:
        acc = Fraction(0)  # (A x)_p
        for a in range(ndim):
            pos = ndim - 1 - a  # position of axis a in the tuple
            for q in range(n[a]):
                c = L[a][p[pos]][q]
                if c:
                    pp = list(p)
                    pp[pos] = q
                    acc += c * get(u, pp)
        b = get(f, p) if f is not None else Fraction(0)
        for a in range(ndim):
            pos = ndim - 1 - a
            if p[pos] == 0:
                b += bvals[2 * a]
            if p[pos] == n[a] - 1:
                b += bvals[2 * a + 1]
        out[p] = get(u, p) + (b - acc) / diag
    return out


def _to_frac_nested(a):
    if a.ndim == 1:
        return [Fraction(float(x)) for x in a]
    return [_to_frac_nested(x) for x in a]


@pytest.mark.parametrize("n", [(1, 1), (2, 2), (3, 3), (4, 2), (1, 1, 1), (2, 2, 2), (3, 2, 4)])
@pytest.mark.parametrize("with_f", [False, True])
def test_tiny_grids_against_exact_rationals(orc, n, with_f):
    ndim = len(n)
    rng = np.random.default_rng(11)
    shape = tuple(reversed(n))
    u0 = rng.uniform(-1, 1, shape)
    f = rng.uniform(-1, 1, shape) if with_f else None
    bvals = [1.0, 2.0, 4.0, 8.0, 16.0, 32.0][: 2 * ndim]  # all different: catches a face mix-up
    u = orc.mono_padded(n, bvals)
    u[(slice(1, -1),) * ndim] = u0
    exact = _to_frac_nested(u0)
    fx = _to_frac_nested(f) if with_f else None
    for sweep in range(1, 4):
        u = orc.mono_sweep(u, f, 1)
        step = _exact_jacobi_step(n, exact, fx, [Fraction(b) for b in bvals])
        # back to nested lists
        arr = np.empty(shape, dtype=object)
        for p, v in step.items():
            arr[p] = v
        exact = arr.tolist()
        got = u[(slice(1, -1),) * ndim]
        for p, v in step.items():
            scale = max(1.0, abs(float(v)))
            # exact arithmetic vs 4-7 roundings per sweep
            assert abs(Fraction(float(got[p])) - v) <= 8 * sweep * EPS * scale, (p, sweep)


def test_single_cell_by_hand(orc):
    """1x1 grid: u' = (W + E + S + N + f)/4 with powers of two, exact in binary."""
    u = orc.mono_padded((1, 1), (1.0, 2.0, 4.0, 8.0))
    u[1, 1] = 123.0  # the centre has weight 0
    got = orc.mono_sweep(u, np.array([[16.0]]), 1)
    assert got[1, 1] == 31.0 / 4.0
    got = orc.mono_sweep(u, None, 1)
    assert got[1, 1] == 15.0 / 4.0


def test_single_cell_3d_by_hand(orc):
    """1x1x1: u' = fl( (sum of the six ghosts + f) * fl(1/6) ): one rounding of an exact product."""
    u = orc.mono_padded((1, 1, 1), (1.0, 2.0, 4.0, 8.0, 16.0, 32.0))
    u[1, 1, 1] = -55.0
    got = orc.mono_sweep(u, np.array([[[64.0]]]), 1)[1, 1, 1]
    want = float(Fraction(127) * Fraction(1.0 / 6.0))  # Fraction(float) is exact; float() rounds once
    assert got == want


# ------------------------------------------------ heated edge: path enumeration
def test_heated_edge_equals_random_walk_hitting_probability(orc):
    """u0 = 0, top ghost row (+y) = 1, others 0: after k sweeps u(i,j) is the probability that a
    simple random walk started at (i,j) leaves the grid through the top edge within k steps.
    Enumerate all 4^k walks; every value is a multiple of 4^-k and exact in binary."""
    nx, ny, k = 5, 4, 5
    u = orc.mono_padded((nx, ny), (0.0, 0.0, 0.0, 1.0))
    got = orc.mono_sweep(u, None, k)[1:-1, 1:-1]
    steps = ((1, 0), (-1, 0), (0, 1), (0, -1))
    for j0 in range(ny):
        for i0 in range(nx):
            hits = 0
            for walk in itertools.product(steps, repeat=k):
                i, j = i0, j0
                for di, dj in walk:
                    i += di
                    j += dj
                    if j >= ny:
                        hits += 1
                        break
                    if i < 0 or i >= nx or j < 0:
                        break
            assert got[j0, i0] == hits / 4.0 ** k, (i0, j0)


def test_heated_edge_256_hand_values_and_invariants(orc):
    """256^2, top edge 1: sweep 1 leaves exactly 0.25 on the top row and 0 elsewhere; information
    moves one row per sweep; the field is mirror-symmetric in x bit for bit, grows monotonically
    and stays within [0, 1] (round-to-nearest adds and multiplies are monotone)."""
    n = (256, 256)
    u = orc.mono_padded(n, (0.0, 0.0, 0.0, 1.0))
    u1 = orc.mono_sweep(u, None, 1)
    assert np.all(u1[-2, 1:-1] == 0.25) and np.all(u1[1:-2, 1:-1] == 0.0)
    prev = u1
    for k in range(2, 12):
        cur = orc.mono_sweep(prev, None, 1)
        inner = cur[1:-1, 1:-1]
        assert np.all(inner[: n[1] - k, :] == 0.0)
        assert np.all(inner[n[1] - k, :] > 0.0)
        assert np.array_equal(inner, inner[:, ::-1])
        assert np.all(inner >= prev[1:-1, 1:-1]) and np.all(inner <= 1.0)
        prev = cur


def test_four_rotated_edge_solutions_sum_to_one(orc):
    """Converged solutions for 'one edge at 1' over the four edges add up to the solution with
    all edges at 1, which is identically 1."""
    n = (8, 8)
    total = np.zeros((8, 8))
    for face in range(4):
        b = [0.0] * 4
        b[face] = 1.0
        total += orc.mono_sweep(orc.mono_padded(n, b), None, 900)[1:-1, 1:-1]
    assert np.max(np.abs(total - 1.0)) < 1e-14


def test_rhs_only_first_sweep(orc):
    """u0 = 0, zero boundary: the first sweep gives exactly f/4 (2D) and fl(f * fl(1/6)) (3D), which
    pins where f enters and its orientation on a non-square grid."""
    f = inputs.uniform_field((6, 3), 5)
    got = orc.mono_sweep(orc.mono_padded((6, 3)), f, 1)[1:-1, 1:-1]
    assert np.array_equal(got, f / 4.0)
    f3 = inputs.uniform_field((4, 3, 2), 6)
    got3 = orc.mono_sweep(orc.mono_padded((4, 3, 2)), f3, 1)[1:-1, 1:-1, 1:-1]
    assert np.array_equal(got3, f3 * (1.0 / 6.0))


# ------------------------------------------------ sub-window sampling
@pytest.mark.parametrize("n,k", [((23, 17), 4), ((9, 11, 7), 3)])
def test_window_sampling_matches_full_run_bitwise(orc, n, k):
    ndim = len(n)
    rng = np.random.default_rng(3)
    shape = tuple(reversed(n))
    u0 = rng.uniform(-1, 1, shape)
    f = rng.uniform(-1, 1, shape)
    bvals = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5][: 2 * ndim]
    u = orc.mono_padded(n, bvals)
    u[(slice(1, -1),) * ndim] = u0
    full = orc.mono_sweep(u, f, k)[(slice(1, -1),) * ndim]

    def box(arr):
        return lambda lo, hi: arr[tuple(slice(l, h) for l, h in zip(reversed(lo), reversed(hi)))]

    pts = [tuple(0 for _ in n), tuple(m - 1 for m in n), tuple(m // 2 for m in n),
           tuple((m // 3 if a else 1) for a, m in enumerate(n))]
    got = orc.sample_points(n, k, pts, box(u0), box(f), bvals)
    for p, g in zip(pts, got):
        assert g == full[tuple(reversed(p))]
