"""Grids that are not a multiple of the block size (remainder blocks at the high end of an axis):
every schedule against the CPU oracle — interiors, ghosts and packed faces bit-exact, residual
within 1e-10."""
import numpy as np
import pytest

from paper_2210_01238_b200 import inputs

pytestmark = pytest.mark.gpu

BVALS = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5]
RESID_TOL = 1e-10

# (n, b, h): remainder in x, in y, in both, of one point, odd remainders (scalar paths), remainders
# equal to h, rows longer than one CTA tile, 3D with remainders on every axis
SHAPES = [((13, 8), (4, 4), 1), ((12, 9), (4, 4), 1), ((14, 11), (4, 4), 2), ((13, 9), (6, 4), 1),
          ((10, 7), (3, 5), 1), ((1100, 210), (600, 100), 2), ((70, 51), (32, 16), 3),
          ((7, 6, 9), (3, 4, 4), 1), ((9, 5, 7), (4, 2, 3), 1), ((8, 8, 5), (4, 4, 4), 1),
          ((150, 30, 22), (128, 16, 10), 2), ((42, 26, 18), (20, 12, 8), 2)]
# shapes the temporal kernels accept: n[0] % 4 == 0 (2D), n[0] % 2 == 0 (3D)
TEMPORAL_SHAPES = [((264, 300), (128, 128), 1), ((136, 70), (64, 32), 1), ((1000, 530), (512, 256), 1),
                   ((72, 50, 40), (64, 48, 16), 1), ((140, 100, 70), (128, 64, 64), 1)]


@pytest.fixture(scope="module")
def jac():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_01238_b200 import jac as _jac
    _jac.lib()
    return _jac


def _pair(jac, orc, n, b, h, has_f, mode, tsteps=0, seed=0):
    ndim = len(n)
    rng = np.random.default_rng(seed)
    shape = tuple(reversed(n))
    u0, f = rng.uniform(-1, 1, shape), rng.uniform(-1, 1, shape)
    J = jac.Jacobi(n, b, h, has_f, mode, tsteps)
    B = orc.Blocked(n, b, h, has_f)
    for face in range(2 * ndim):
        J.set_boundary(face, BVALS[face]); B.set_boundary(face, BVALS[face])
    J.set_u(u0); B.set_u(u0)
    if has_f:
        J.set_f(f); B.set_f(f)
    return J, B


@pytest.mark.parametrize("n,b,h", SHAPES)
@pytest.mark.parametrize("mode", ["fused", "exchange", "pertask", "wide"])
@pytest.mark.parametrize("has_f", [False, True])
def test_sweeps_with_remainder_blocks(jac, orc, n, b, h, mode, has_f):
    J, B = _pair(jac, orc, n, b, h, has_f, mode)
    assert J.nblocks == B.nblocks
    J.sweep(3); J.sweep(4)
    B.sweep(7)
    assert np.array_equal(J.get_u(), B.get_u())
    r, want = J.residual(), B.residual()
    assert abs(r - want) <= RESID_TOL * want
    r = J.sweep_residual(2)
    B.sweep(1)
    want = B.residual()
    assert abs(r - want) <= RESID_TOL * want
    B.sweep(1)
    assert np.array_equal(J.get_u(), B.get_u())
    J.close(); B.close()


@pytest.mark.parametrize("n,b,h", SHAPES)
def test_exchange_with_remainder_blocks_is_bit_exact(jac, orc, n, b, h):
    ndim = len(n)
    J = jac.Jacobi(n, b, h, False, "wide")
    B = orc.Blocked(n, b, h)
    dense = inputs.linear_index_field(n)
    for face in range(2 * ndim):
        J.set_boundary(face, BVALS[face]); B.set_boundary(face, BVALS[face])
    J.set_u(dense); B.set_u(dense)
    J.pack_halos(); J.unpack_halos()
    B.pack(); B.unpack()
    for blk in range(B.nblocks):
        assert J.extent(blk) == B.extent(blk)
        for face in range(2 * ndim):
            if B.neighbour(blk, face) >= 0:
                assert np.array_equal(J.get_halo_buffer(blk, face), B.get_halo_buffer(blk, face)), (blk, face)
        assert np.array_equal(J.get_block_padded(blk), B.get_block_padded(blk)), blk
    bufs = B.exchange_wide(keep_buffers=True)
    J.exchange_wide()
    for (blk, face), want in bufs.items():
        assert np.array_equal(J.get_wide_buffer(blk, face), want), (blk, face)
    for blk in range(B.nblocks):
        assert np.array_equal(J.get_block_padded(blk), B.get_block_padded(blk)), blk
    assert np.array_equal(J.get_u(), dense)
    J.close(); B.close()


@pytest.mark.parametrize("n,b,h", TEMPORAL_SHAPES)
@pytest.mark.parametrize("has_f", [False, True])
def test_temporal_kernels_with_remainder_blocks(jac, orc, n, b, h, has_f):
    for tsteps in ([1, 2, 4, 8] if len(n) == 2 else [1, 2]):
        J, B = _pair(jac, orc, n, b, h, has_f, "temporal", tsteps)
        J.sweep(tsteps + 3)
        B.sweep(tsteps + 3)
        assert np.array_equal(J.get_u(), B.get_u()), (n, b, tsteps)
        r, want = J.residual(), B.residual()
        assert abs(r - want) <= RESID_TOL * want
        J.close(); B.close()


@pytest.mark.parametrize("n,b", [((72, 50), (32, 16)), ((264, 130), (128, 64)), ((20, 9), (8, 4))])
@pytest.mark.parametrize("has_f", [False, True])
def test_resident_schedule_with_remainder_blocks(jac, orc, n, b, has_f):
    J, B = _pair(jac, orc, n, b, 1, has_f, "resident")
    J.sweep(9); B.sweep(9)
    assert np.array_equal(J.get_u(), B.get_u())
    J.close(); B.close()


def test_device_resident_copies_with_remainder_blocks(jac, orc):
    import torch
    for n, b in [((13, 9), (6, 4)), ((70, 50), (32, 16)), ((9, 5, 7), (4, 2, 3))]:
        dense = inputs.linear_index_field(n)
        with jac.Jacobi(n, b, 1, True, "fused") as J:
            J.set_u_device(torch.from_numpy(dense).cuda())
            assert np.array_equal(J.get_u(), dense)
            J.set_u(dense * 2)
            assert np.array_equal(J.get_u_device().cpu().numpy(), dense * 2)


def test_remainder_narrower_than_the_halo_is_refused(jac):
    with pytest.raises(jac.JacError) as e:
        jac.Jacobi((13, 8), (4, 4), 2)
    assert e.value.code == jac.EINVAL
