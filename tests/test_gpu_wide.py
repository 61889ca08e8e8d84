"""GPU wide exchange (all h ghost layers with edges and corners) and groups of up to h sweeps
per exchange, against the CPU oracle: ghosts and packed wide faces bit-exact, interiors
bit-exact, residual within 1e-10."""
import numpy as np
import pytest

from paper_2210_01238_b200 import inputs

pytestmark = pytest.mark.gpu

BVALS = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5]
RESID_TOL = 1e-10

# (n, b, h): several blocks per axis, odd and even widths (scalar and 128-bit paths), single
# blocks along an axis, rows longer than one CTA tile, h up to 8
SHAPES = [((12, 8), (4, 4), 2), ((15, 9), (5, 3), 3), ((64, 48), (16, 8), 4), ((36, 24), (12, 8), 1),
          ((1100, 200), (550, 100), 2), ((130, 210), (130, 70), 3), ((32, 24), (16, 8), 8),
          ((640, 72), (640, 72), 2),
          ((6, 4, 8), (3, 2, 4), 2), ((24, 18, 12), (8, 6, 4), 3), ((48, 40, 20), (24, 20, 10), 2),
          ((132, 20, 36), (132, 10, 18), 4), ((16, 16, 16), (8, 8, 8), 8), ((20, 12, 40), (10, 12, 20), 1)]


@pytest.fixture(scope="module")
def jac():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_01238_b200 import jac as _jac
    _jac.lib()
    return _jac


def _pair(jac, orc, n, b, h, has_f, tsteps=0, seed=0):
    ndim = len(n)
    rng = np.random.default_rng(seed)
    shape = tuple(reversed(n))
    u0, f = rng.uniform(-1, 1, shape), rng.uniform(-1, 1, shape)
    J = jac.Jacobi(n, b, h, has_f, "wide", tsteps)
    B = orc.Blocked(n, b, h, has_f)
    for face in range(2 * ndim):
        J.set_boundary(face, BVALS[face])
        B.set_boundary(face, BVALS[face])
    J.set_u(u0); B.set_u(u0)
    if has_f:
        J.set_f(f); B.set_f(f)
    return J, B


@pytest.mark.parametrize("n,b,h", SHAPES)
def test_wide_exchange_ghosts_and_buffers_are_bit_exact(jac, orc, n, b, h):
    ndim = len(n)
    J = jac.Jacobi(n, b, h, False, "wide")
    B = orc.Blocked(n, b, h)
    dense = inputs.linear_index_field(n)
    for face in range(2 * ndim):
        J.set_boundary(face, BVALS[face]); B.set_boundary(face, BVALS[face])
    J.set_u(dense); B.set_u(dense)
    bufs = B.exchange_wide(keep_buffers=True)
    J.exchange_wide()
    for blk in range(B.nblocks):
        assert np.array_equal(J.get_block_padded(blk), B.get_block_padded(blk)), (blk,)
    # every face has its own send slot, so the packed faces of all axes are still there
    for (blk, face), want in bufs.items():
        assert np.array_equal(J.get_wide_buffer(blk, face), want), (blk, face)
    assert np.array_equal(J.get_u(), dense)
    J.close(); B.close()


@pytest.mark.parametrize("n,b,h", SHAPES)
@pytest.mark.parametrize("has_f", [False, True])
def test_wide_schedule_matches_oracle_bitwise(jac, orc, n, b, h, has_f):
    for k in sorted({1, 2, h, max(1, h - 1)} & set(range(1, h + 1))):
        J, B = _pair(jac, orc, n, b, h, has_f, tsteps=k)
        J.sweep(4); J.sweep(3)
        B.sweep_wide(4, k); B.sweep_wide(3, k)
        got, want = J.get_u(), B.get_u()
        assert np.array_equal(got, want), (n, b, h, k)
        # and equal to the schedule that exchanges before every sweep
        P = orc.Blocked(n, b, h, has_f)
        for face in range(2 * len(n)):
            P.set_boundary(face, BVALS[face])
        rng = np.random.default_rng(0)
        shape = tuple(reversed(n))
        u0, f = rng.uniform(-1, 1, shape), rng.uniform(-1, 1, shape)
        P.set_u(u0)
        if has_f:
            P.set_f(f)
        P.sweep(7)
        assert np.array_equal(got, P.get_u())
        r_got, r_want = J.residual(), B.residual()
        assert abs(r_got - r_want) <= RESID_TOL * r_want
        J.close(); B.close(); P.close()


def test_wide_schedule_default_group_is_h_and_counts_launches(jac, orc):
    n, b, h = (64, 48), (16, 8), 4
    J, B = _pair(jac, orc, n, b, h, True)
    before = J.launch_count()
    J.sweep(8)                      # two groups of 4: 2 x (4 exchange launches + 4 updates) + f's exchange
    assert J.launch_count() - before == 2 * (4 + 4) + 4
    B.sweep_wide(8)
    assert np.array_equal(J.get_u(), B.get_u())
    # a new right-hand side invalidates f's ghost layers
    f2 = np.random.default_rng(4).uniform(-1, 1, (48, 64))
    J.set_f(f2); B.set_f(f2)
    J.sweep(5); B.sweep_wide(5)
    assert np.array_equal(J.get_u(), B.get_u())
    J.close(); B.close()


def test_wide_sweep_with_fused_residual_and_solve(jac, orc):
    n, b, h = (48, 40, 20), (24, 20, 10), 2
    J, B = _pair(jac, orc, n, b, h, True)
    r = J.sweep_residual(5)
    B.sweep_wide(4)
    want = B.residual()
    assert abs(r - want) <= RESID_TOL * want
    B.sweep_wide(1)
    assert np.array_equal(J.get_u(), B.get_u())
    J.close(); B.close()


def test_wide_calls_need_a_wide_context(jac):
    with jac.Jacobi((12, 8), (4, 4), 2, False, "exchange") as J:
        with pytest.raises(jac.JacError) as e:
            J.exchange_wide()
        assert e.value.code == jac.EINVAL
    with pytest.raises(jac.JacError):
        jac.Jacobi((12, 8), (4, 4), 2, False, "wide", 3)


def test_plain_exchange_still_works_in_a_wide_context(jac, orc):
    n, b, h = (36, 24), (12, 8), 2
    J, B = _pair(jac, orc, n, b, h, False)
    J.pack_halos(); J.unpack_halos()
    B.pack(); B.unpack()
    for blk in range(B.nblocks):
        for face in range(4):
            if B.neighbour(blk, face) >= 0:
                assert np.array_equal(J.get_halo_buffer(blk, face), B.get_halo_buffer(blk, face))
        assert np.array_equal(J.get_block_padded(blk), B.get_block_padded(blk))
    J.close(); B.close()
