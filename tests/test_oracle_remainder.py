"""Pins for grids that are not a multiple of the block size: the last block along such an axis
is a remainder block (n - (g-1)*b points), everything else is as for equal blocks."""
import numpy as np
import pytest

from paper_2210_01238_b200 import inputs

# (n, b): remainder in x only, y only, both; remainder of one point; three axes; remainder = h
SHAPES = [((13, 8), (4, 4)), ((12, 9), (4, 4)), ((14, 11), (4, 4)), ((13, 9), (6, 4)), ((10, 7), (3, 5)),
          ((7, 6, 9), (3, 4, 4)), ((9, 5, 7), (4, 2, 3)), ((8, 8, 5), (4, 4, 4))]
BVALS = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5]


def _halos(n, b):
    rem = [nn - (-(-nn // bb) - 1) * bb for nn, bb in zip(n, b)]
    return [h for h in (1, 2, 3) if h <= min(rem)]


def test_block_grid_and_extents(orc):
    B = orc.Blocked((14, 11), (4, 4), 1)
    assert B.g == [4, 3] and B.nblocks == 12
    assert B.extent(0) == [4, 4] and B.extent(3) == [2, 4] and B.extent(8) == [4, 3] and B.extent(11) == [2, 3]
    assert B.face_shape(0, 11) == (3, 1) and B.face_shape(2, 11) == (1, 2)
    assert B.padded_shape() == (6, 6)            # every block keeps a full-size padded array


@pytest.mark.parametrize("n,b", SHAPES)
@pytest.mark.parametrize("with_f", [False, True])
def test_sweeps_with_remainder_blocks_are_bit_identical_to_monolithic(orc, n, b, with_f):
    ndim = len(n)
    rng = np.random.default_rng(21)
    shape = tuple(reversed(n))
    u0 = rng.uniform(-1, 1, shape)
    f = rng.uniform(-1, 1, shape) if with_f else None
    bvals = BVALS[: 2 * ndim]
    m = orc.mono_padded(n, bvals)
    m[(slice(1, -1),) * ndim] = u0
    mono = orc.mono_sweep(m, f, 6)
    want = mono[(slice(1, -1),) * ndim]
    want_r = orc.mono_residual(mono, f)
    for h in _halos(n, b):
        for k in [0] + list(range(1, h + 1)):        # 0: exchange before every sweep; k: wide groups of k
            B = orc.Blocked(n, b, h, with_f)
            for face, v in enumerate(bvals):
                B.set_boundary(face, v)
            B.set_u(u0)
            if with_f:
                B.set_f(f)
            if k == 0:
                B.sweep(6)
            else:
                B.sweep_wide(4, k); B.sweep_wide(2, k)
            assert np.array_equal(B.get_u(), want), (n, b, h, k)
            r = B.residual()
            assert abs(r - want_r) <= 1e-13 * want_r
            B.close()


@pytest.mark.parametrize("n,b", SHAPES)
def test_pack_and_unpack_with_remainder_blocks(orc, n, b):
    """u = global linear index: packed faces are numpy slices of the block's part of the dense array,
    and after the exchange every ghost next to a neighbour holds the neighbour's cell."""
    ndim = len(n)
    dense = inputs.linear_index_field(n)
    for h in _halos(n, b):
        B = orc.Blocked(n, b, h)
        for face in range(2 * ndim):
            B.set_boundary(face, -(face + 1.5))
        B.set_u(dense)
        B.pack(); B.unpack()
        G = np.full(tuple(x + 2 * h for x in reversed(n)), np.nan)
        G[(slice(h, -h),) * ndim] = dense
        for face in range(2 * ndim):
            ax = ndim - 1 - face // 2
            idx = [slice(h, -h)] * ndim
            idx[ax] = slice(-h, None) if face & 1 else slice(0, h)
            G[tuple(idx)] = -(face + 1.5)
        for blk in range(B.nblocks):
            c, e = B.coords(blk), B.extent(blk)
            mine = dense[tuple(slice(c[a] * b[a], c[a] * b[a] + e[a]) for a in reversed(range(ndim)))]
            pad = B.get_block_padded(blk)
            # the part of the padded array the block uses: extent + 2h from the low corner
            used = pad[tuple(slice(0, e[a] + 2 * h) for a in reversed(range(ndim)))]
            win = G[tuple(slice(c[a] * b[a], c[a] * b[a] + e[a] + 2 * h) for a in reversed(range(ndim)))]
            known = ~np.isnan(win)
            for a in range(ndim):                  # edges and corners are not part of a face exchange
                pass
            faces_only = np.zeros(win.shape, dtype=bool)
            for face in range(2 * ndim):
                ax = ndim - 1 - face // 2
                idx = [slice(h, -h)] * ndim
                idx[ax] = slice(-h, None) if face & 1 else slice(0, h)
                faces_only[tuple(idx)] = True
            faces_only[(slice(h, -h),) * ndim] = True
            sel = known & faces_only
            assert np.array_equal(used[sel], win[sel]), (n, b, h, blk)
            for face in range(2 * ndim):
                if B.neighbour(blk, face) < 0:
                    continue
                ax = ndim - 1 - face // 2
                idx = [slice(None)] * ndim
                idx[ax] = slice(e[face // 2] - h, None) if face & 1 else slice(0, h)
                assert np.array_equal(B.get_halo_buffer(blk, face), mine[tuple(idx)]), (blk, face, h)
        B.close()


def test_wide_exchange_with_remainder_blocks_fills_corners(orc):
    n, b, h = (14, 11), (4, 4), 2
    dense = inputs.linear_index_field(n)
    B = orc.Blocked(n, b, h)
    B.set_u(dense)
    B.exchange_wide()
    G = np.zeros((11 + 4, 14 + 4))
    G[2:-2, 2:-2] = dense
    for blk in range(B.nblocks):
        c, e = B.coords(blk), B.extent(blk)
        used = B.get_block_padded(blk)[: e[1] + 4, : e[0] + 4]
        win = G[c[1] * 4: c[1] * 4 + e[1] + 4, c[0] * 4: c[0] * 4 + e[0] + 4]
        assert np.array_equal(used, win), blk      # all Dirichlet values are 0 here, corners included
