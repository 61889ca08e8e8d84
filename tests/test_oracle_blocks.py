"""Pins for the oracle's block decomposition, pack/unpack and residual."""
import math

import numpy as np
import pytest

from paper_2210_01238_b200 import inputs

EPS = np.finfo(np.float64).eps

SHAPES_2D = [((12, 8), (12, 8)), ((12, 8), (4, 4)), ((12, 8), (1, 1)), ((12, 8), (3, 2)),
             ((12, 8), (12, 1)), ((12, 8), (1, 8)), ((12, 8), (6, 4)), ((32, 24), (16, 8))]
SHAPES_3D = [((6, 4, 8), (3, 2, 4)), ((6, 4, 8), (1, 1, 1)), ((6, 4, 8), (6, 4, 8)),
             ((6, 4, 8), (2, 4, 2)), ((6, 4, 8), (6, 1, 4))]


def _halos(b):
    return [h for h in (1, 2, 3, 4, 8) if h <= min(b)]


def _block_box(B, blk):
    """numpy slices of block ``blk`` in the dense array, and its (x, y, z) block coordinates."""
    g = B.g + [1] * (3 - B.ndim)
    c = [blk % g[0], (blk // g[0]) % g[1], blk // (g[0] * g[1])][: B.ndim]
    sl = tuple(slice(c[a] * B.b[a], (c[a] + 1) * B.b[a]) for a in reversed(range(B.ndim)))
    return sl, c


# ---------------------------------------------------- blocked == monolithic
@pytest.mark.parametrize("n,b", SHAPES_2D + SHAPES_3D)
@pytest.mark.parametrize("with_f", [False, True])
def test_blocked_sweep_is_bit_identical_to_monolithic(orc, n, b, with_f):
    ndim = len(n)
    rng = np.random.default_rng(7)
    shape = tuple(reversed(n))
    u0 = rng.uniform(-1, 1, shape)
    f = rng.uniform(-1, 1, shape) if with_f else None
    bvals = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5][: 2 * ndim]
    m = orc.mono_padded(n, bvals)
    m[(slice(1, -1),) * ndim] = u0
    want = orc.mono_sweep(m, f, 5)[(slice(1, -1),) * ndim]
    for h in _halos(b):
        B = orc.Blocked(n, b, h, with_f)
        for face, v in enumerate(bvals):
            B.set_boundary(face, v)
        B.set_u(u0)
        if with_f:
            B.set_f(f)
        B.sweep(2)
        B.sweep(3)
        assert np.array_equal(B.get_u(), want), (n, b, h)
        B.close()


# ---------------------------------------------------- pack order and unpack placement
@pytest.mark.parametrize("n,b", SHAPES_2D + SHAPES_3D)
def test_pack_is_the_face_strip_in_memory_order(orc, n, b):
    """With u = global linear index every packed buffer must equal the numpy slice of the dense
    array: the h interior layers next to the face, other axes over the block interior."""
    ndim = len(n)
    dense = inputs.linear_index_field(n)
    for h in _halos(b):
        B = orc.Blocked(n, b, h)
        B.set_u(dense)
        B.pack()
        for blk in range(B.nblocks):
            sl, _ = _block_box(B, blk)
            mine = dense[sl]
            for face in range(2 * ndim):
                if B.neighbour(blk, face) < 0:
                    continue
                ax = ndim - 1 - face // 2
                idx = [slice(None)] * ndim
                idx[ax] = slice(b[face // 2] - h, None) if face & 1 else slice(0, h)
                assert np.array_equal(B.get_halo_buffer(blk, face), mine[tuple(idx)]), (blk, face, h)
        B.close()


@pytest.mark.parametrize("n,b", SHAPES_2D + SHAPES_3D)
def test_unpack_fills_ghosts_with_the_neighbours_strip_and_nothing_else(orc, n, b):
    ndim = len(n)
    dense = inputs.linear_index_field(n) + 1.0  # no zeros inside
    bvals = [-1.0, -2.0, -3.0, -4.0, -5.0, -6.0][: 2 * ndim]
    for h in _halos(b):
        B = orc.Blocked(n, b, h)
        for face, v in enumerate(bvals):
            B.set_boundary(face, v)
        B.set_u(dense)
        before = [B.get_block_padded(k) for k in range(B.nblocks)]
        B.pack()
        B.unpack()
        # the padded dense array: what every ghost should see
        full = np.zeros(tuple(s + 2 * h for s in dense.shape))
        full[(slice(h, -h),) * ndim] = dense
        for blk in range(B.nblocks):
            got = B.get_block_padded(blk)
            sl, c = _block_box(B, blk)
            inner = (slice(h, -h),) * ndim
            assert np.array_equal(got[inner], dense[sl])            # interior untouched
            expect = before[blk].copy()
            for face in range(2 * ndim):
                a = face // 2
                ax = ndim - 1 - a
                idx = [slice(h, -h)] * ndim
                idx[ax] = slice(-h, None) if face & 1 else slice(0, h)
                if B.neighbour(blk, face) < 0:
                    assert np.all(got[tuple(idx)] == bvals[face])   # Dirichlet ghosts untouched
                    continue
                # window of the padded dense array covering this padded block
                win = tuple(slice(c[q] * b[q], c[q] * b[q] + b[q] + 2 * h)
                            for q in reversed(range(ndim)))
                expect[tuple(idx)] = full[win][tuple(idx)]
            assert np.array_equal(got, expect), (blk, h)            # edges/corners untouched too
        B.close()


def test_pack_then_unpack_is_idempotent(orc):
    n, b = (12, 8), (4, 4)
    B = orc.Blocked(n, b, 2)
    B.set_u(inputs.uniform_field(n, 2))
    B.pack(); B.unpack()
    first = [B.get_block_padded(k) for k in range(B.nblocks)]
    B.pack(); B.unpack()
    for k in range(B.nblocks):
        assert np.array_equal(first[k], B.get_block_padded(k))


def test_create_rejects_bad_shapes(orc):
    # a remainder block narrower than the halo (13 = 3 * 4 + 1 < 2), h = 0, h > b, b = 0, b > n
    for n, b, h in [((13, 8), (4, 4), 2), ((12, 8), (4, 4), 0), ((12, 8), (4, 4), 5),
                    ((12, 8), (0, 4), 1), ((12, 8), (16, 4), 1)]:
        with pytest.raises(ValueError):
            orc.Blocked(n, b, h)


# ---------------------------------------------------- residual
@pytest.mark.parametrize("n", [(7, 7), (16, 9), (64, 64), (5, 7, 3), (8, 4, 6)])
def test_residual_of_eigenmode_closed_form(orc, n):
    """r = c (lambda - 1) u for an eigenmode, and ||sin-mode||_2^2 = prod (n_a + 1)/2."""
    ndim = len(n)
    c = 2.0 * ndim
    lam = sum(math.cos(math.pi / (m + 1)) for m in n) / ndim
    norm_u0 = math.sqrt(np.prod([(m + 1) / 2.0 for m in n]))
    u = orc.mono_padded(n)
    u[(slice(1, -1),) * ndim] = inputs.sine_mode(n)
    for k in (0, 3, 10):
        uk = orc.mono_sweep(u, None, k)
        want = c * (1.0 - lam) * lam ** k * norm_u0
        assert orc.mono_residual(uk) == pytest.approx(want, rel=1e-12 / (1.0 - lam))


def test_residual_2d_equals_four_times_the_next_update(orc):
    """2D: r_k = 4 (u_{k+1} - u_k) point-wise, exactly (x0.25 and x4 are exact), so the norm must
    agree with numpy's norm of the oracle's own consecutive iterates to rounding."""
    n = (33, 21)
    f = inputs.uniform_field(n, 1)
    u = orc.mono_padded(n, (0.5, -1.0, 2.0, 3.0))
    u[1:-1, 1:-1] = inputs.uniform_field(n, 4)
    for _ in range(3):
        nxt = orc.mono_sweep(u, f, 1)
        d = (4.0 * (nxt[1:-1, 1:-1] - u[1:-1, 1:-1])).astype(np.longdouble)
        want = float(np.sqrt(np.sum(d * d)))
        assert orc.mono_residual(u, f) == pytest.approx(want, rel=4 * EPS)
        u = nxt


@pytest.mark.parametrize("n", [(40, 24), (10, 6, 8)])
def test_residual_at_zero_is_norm_of_f(orc, n):
    f = inputs.uniform_field(n, 9)
    assert orc.mono_residual(orc.mono_padded(n), f) == pytest.approx(np.linalg.norm(f), rel=1e-14)


def test_residual_3d_against_exact_rationals(orc):
    """r = f + g - A u assembled from exact rationals on a 3x2x4 box (g = Dirichlet terms)."""
    from fractions import Fraction
    n = (3, 2, 4)
    rng = np.random.default_rng(5)
    u0 = rng.uniform(-1, 1, (4, 2, 3))
    f = rng.uniform(-1, 1, (4, 2, 3))
    bvals = [1.0, 2.0, 4.0, 8.0, 16.0, 32.0]
    u = orc.mono_padded(n, bvals)
    u[1:-1, 1:-1, 1:-1] = u0
    tot = Fraction(0)
    for k in range(4):
        for j in range(2):
            for i in range(3):
                def val(ii, jj, kk):
                    if ii < 0: return Fraction(bvals[0])
                    if ii >= 3: return Fraction(bvals[1])
                    if jj < 0: return Fraction(bvals[2])
                    if jj >= 2: return Fraction(bvals[3])
                    if kk < 0: return Fraction(bvals[4])
                    if kk >= 4: return Fraction(bvals[5])
                    return Fraction(float(u0[kk, jj, ii]))
                nb = (val(i - 1, j, k) + val(i + 1, j, k) + val(i, j - 1, k) + val(i, j + 1, k)
                      + val(i, j, k - 1) + val(i, j, k + 1))
                r = Fraction(float(f[k, j, i])) + nb - 6 * val(i, j, k)
                tot += r * r
    assert orc.mono_residual(u, f) == pytest.approx(math.sqrt(float(tot)), rel=1e-14)


def test_residual_vanishes_at_convergence_and_decreases(orc):
    n = (8, 8)
    f = inputs.uniform_field(n, 1)
    u = orc.mono_padded(n, (0.0, 0.0, 0.0, 1.0))
    last = orc.mono_residual(u, f)
    for _ in range(10):
        u = orc.mono_sweep(u, f, 10)
        cur = orc.mono_residual(u, f)
        assert cur < last
        last = cur
    u = orc.mono_sweep(u, f, 900)
    assert orc.mono_residual(u, f) < 1e-13


@pytest.mark.parametrize("n,b", [((12, 8), (4, 4)), ((12, 8), (3, 2)), ((6, 4, 8), (3, 2, 4))])
def test_blocked_residual_matches_monolithic(orc, n, b):
    ndim = len(n)
    rng = np.random.default_rng(8)
    shape = tuple(reversed(n))
    u0, f = rng.uniform(-1, 1, shape), rng.uniform(-1, 1, shape)
    bvals = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5][: 2 * ndim]
    m = orc.mono_padded(n, bvals)
    m[(slice(1, -1),) * ndim] = u0
    B = orc.Blocked(n, b, 1, True)
    for face, v in enumerate(bvals):
        B.set_boundary(face, v)
    B.set_u(u0); B.set_f(f)
    for _ in range(3):
        assert B.residual() == pytest.approx(orc.mono_residual(m, f), rel=4 * EPS)
        B.sweep(2)
        m = orc.mono_sweep(m, f, 2)
