"""Pins for the oracle's wide exchange (all h ghost layers with edges and corners, filled axis
by axis) and for groups of up to h sweeps per exchange on shrinking extents."""
import numpy as np
import pytest

from paper_2210_01238_b200 import inputs

SHAPES_2D = [((12, 8), (4, 4)), ((12, 8), (3, 2)), ((12, 8), (12, 8)), ((12, 8), (6, 8)),
             ((20, 12), (5, 4)), ((16, 16), (4, 8))]
SHAPES_3D = [((6, 4, 8), (3, 2, 4)), ((6, 4, 8), (6, 4, 8)), ((8, 8, 8), (4, 4, 2)),
             ((9, 6, 6), (3, 3, 3))]
BVALS = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5]


def _halos(b):
    return [h for h in (1, 2, 3, 4) if h <= min(b)]


def _coords(B, blk):
    g = B.g + [1] * (3 - B.ndim)
    return [blk % g[0], (blk // g[0]) % g[1], blk // (g[0] * g[1])][: B.ndim]


def _global_padded(n, h, dense, bvals):
    """The whole domain with h layers around it: Dirichlet value of a face in all h layers outside
    that face (over the in-domain extent of the other axes); `known` is False where a position
    lies outside the domain in two or more axes (such cells are never read)."""
    ndim = len(n)
    G = np.zeros(tuple(x + 2 * h for x in reversed(n)))
    G[(slice(h, -h),) * ndim] = dense
    outside = np.zeros(G.shape, dtype=int)
    for face in range(2 * ndim):
        ax = ndim - 1 - face // 2
        idx = [slice(h, -h)] * ndim
        idx[ax] = slice(-h, None) if face & 1 else slice(0, h)
        G[tuple(idx)] = bvals[face]
    for a in range(ndim):
        idx = [slice(None)] * ndim
        for sl in (slice(0, h), slice(-h, None)):
            idx[a] = sl
            outside[tuple(idx)] += 1
    return G, outside <= 1


# ---------------------------------------------------- the point of it: k sweeps per exchange
@pytest.mark.parametrize("n,b", SHAPES_2D + SHAPES_3D)
@pytest.mark.parametrize("with_f", [False, True])
def test_wide_sweeps_are_bit_identical_to_monolithic(orc, n, b, with_f):
    ndim = len(n)
    rng = np.random.default_rng(11)
    shape = tuple(reversed(n))
    u0 = rng.uniform(-1, 1, shape)
    f = rng.uniform(-1, 1, shape) if with_f else None
    bvals = BVALS[: 2 * ndim]
    m = orc.mono_padded(n, bvals)
    m[(slice(1, -1),) * ndim] = u0
    want = orc.mono_sweep(m, f, 7)[(slice(1, -1),) * ndim]
    for h in _halos(b):
        for k in range(1, h + 1):
            B = orc.Blocked(n, b, h, with_f)
            for face, v in enumerate(bvals):
                B.set_boundary(face, v)
            B.set_u(u0)
            if with_f:
                B.set_f(f)
            B.sweep_wide(4, k)      # group sizes that do not divide the sweep counts
            B.sweep_wide(3, k)
            assert np.array_equal(B.get_u(), want), (n, b, h, k)
            B.close()


def test_groups_of_one_are_the_plain_schedule(orc):
    n, b, h = (12, 8), (4, 4), 2
    rng = np.random.default_rng(5)
    u0 = rng.uniform(-1, 1, (8, 12))
    A, B = orc.Blocked(n, b, h), orc.Blocked(n, b, h)
    A.set_u(u0); B.set_u(u0)
    A.sweep(3); B.sweep_wide(3, 1)
    assert np.array_equal(A.get_u(), B.get_u())


# ---------------------------------------------------- what the exchange leaves in the ghosts
@pytest.mark.parametrize("n,b", SHAPES_2D + SHAPES_3D)
def test_wide_exchange_fills_every_ghost_from_the_global_field(orc, n, b):
    """With u = global linear index, every padded block must equal the matching window of the
    padded global field: neighbours' interiors in the ghosts, edges and corners included, and
    the face's Dirichlet value outside the domain."""
    ndim = len(n)
    dense = inputs.linear_index_field(n)
    bvals = [-(face + 1.5) for face in range(2 * ndim)]
    for h in _halos(b):
        G, known = _global_padded(n, h, dense, bvals)
        B = orc.Blocked(n, b, h)
        for face, v in enumerate(bvals):
            B.set_boundary(face, v)
        B.set_u(dense)
        B.exchange_wide()
        assert np.array_equal(B.get_u(), dense)            # interiors untouched
        for blk in range(B.nblocks):
            c = _coords(B, blk)
            win = tuple(slice(c[a] * b[a], c[a] * b[a] + b[a] + 2 * h) for a in reversed(range(ndim)))
            got = B.get_block_padded(blk)
            assert np.array_equal(got[known[win]], G[win][known[win]]), (n, b, h, blk)
        B.close()


@pytest.mark.parametrize("n,b", SHAPES_2D + SHAPES_3D)
def test_wide_buffers_are_strips_in_memory_order(orc, n, b):
    """A packed wide face of axis a is the h interior layers next to the face over the whole
    padded extent of the other axes, x fastest.  Restricted to the interior extent of the axes
    exchanged later it must equal that slice of the final padded block (nothing written
    afterwards lies there)."""
    ndim = len(n)
    dense = inputs.linear_index_field(n)
    for h in _halos(b):
        B = orc.Blocked(n, b, h)
        B.set_u(dense)
        bufs = B.exchange_wide(keep_buffers=True)
        for (blk, face), buf in bufs.items():
            axis = face // 2
            assert buf.shape == B.wide_face_shape(face)
            pad = B.get_block_padded(blk)
            idx = [slice(None)] * ndim
            idx[ndim - 1 - axis] = slice(b[axis], b[axis] + h) if face & 1 else slice(h, 2 * h)
            strip = pad[tuple(idx)]
            later = [slice(None)] * ndim
            for a in range(axis + 1, ndim):
                later[ndim - 1 - a] = slice(h, -h)
            assert np.array_equal(buf[tuple(later)], strip[tuple(later)]), (n, b, h, blk, face)
        # faces on the domain boundary are not exchanged
        for blk in range(B.nblocks):
            for face in range(2 * ndim):
                assert ((blk, face) in bufs) == (B.neighbour(blk, face) >= 0)
        B.close()


# ---------------------------------------------------- the extended update
def test_extended_update_with_zero_extension_is_the_plain_update(orc):
    n, b, h = (12, 8), (4, 4), 2
    rng = np.random.default_rng(3)
    u0, f = rng.uniform(-1, 1, (8, 12)), rng.uniform(-1, 1, (8, 12))
    A, B = orc.Blocked(n, b, h, True), orc.Blocked(n, b, h, True)
    for X in (A, B):
        X.set_u(u0); X.set_f(f); X.set_boundary(1, 2.0)
        X.pack(); X.unpack()
    A.update(); B.update_ext(0)
    assert np.array_equal(A.get_u(), B.get_u())


def test_extended_update_keeps_values_outside_the_domain_and_rejects_too_wide(orc):
    n, b, h = (8, 8), (4, 4), 3
    B = orc.Blocked(n, b, h)
    for face in range(4):
        B.set_boundary(face, 10.0 + face)
    B.set_u(np.random.default_rng(2).uniform(-1, 1, (8, 8)))
    B.exchange_wide()
    before = [B.get_block_padded(k) for k in range(B.nblocks)]
    B.update_ext(2)
    # block 0 sits in the -x, -y corner: its -x and -y ghost layers lie outside the domain
    after = B.get_block_padded(0)
    # (the update wrote the window [h-2, h+b+2) of the other array; compare inside it)
    assert np.array_equal(after[h:-1, 1:h], before[0][h:-1, 1:h])   # -x ghosts, extended rows
    assert np.array_equal(after[1:h, h:-1], before[0][1:h, h:-1])   # -y ghosts
    assert np.all(after[h:h + 4, h - 1] == 10.0) and np.all(after[h - 1, h:h + 4] == 12.0)
    with pytest.raises(ValueError):
        B.update_ext(3)      # would read beyond the ghost layers
    with pytest.raises(ValueError):
        B.sweep_wide(2, 4)   # more sweeps per exchange than ghost layers


def test_extended_region_matches_the_neighbours_own_update(orc):
    """After one extended update the ghost layers inside the domain hold exactly what the owning
    block computed for those points (redundant computation, same bits)."""
    n, b, h = (12, 12, 6), (4, 6, 3), 2
    rng = np.random.default_rng(9)
    u0, f = rng.uniform(-1, 1, (6, 12, 12)), rng.uniform(-1, 1, (6, 12, 12))
    B = orc.Blocked(n, b, h, True)
    B.set_u(u0); B.set_f(f)
    B.exchange_wide()
    B.update_ext(1)
    dense = B.get_u()
    G, known = _global_padded(n, h, dense, [0.0] * 6)
    for blk in range(B.nblocks):
        c = _coords(B, blk)
        win = tuple(slice(c[a] * b[a], c[a] * b[a] + b[a] + 2 * h) for a in reversed(range(3)))
        inner = (slice(h - 1, -(h - 1)),) * 3     # interior extended by one layer
        got = B.get_block_padded(blk)[inner]
        assert np.array_equal(got[known[win][inner]], G[win][inner][known[win][inner]]), blk
