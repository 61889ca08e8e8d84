"""Pins of the oracle's slab form: a domain held as several blocked states cut along the slowest
axis, with the faces on the cuts packed, carried over and unpacked before every update, is the
monolithic run bit for bit; the packed cut planes are numpy slices of the field."""
import numpy as np
import pytest

from paper_2210_01238_b200 import inputs
from paper_2210_01238_b200.sharded import slab_of, slab_planes, slab_slice


def _slabs(orc, n, b, h, has_f, parts, u0, f, bvals):
    out = []
    for p in range(parts):
        n_slab, b_slab, _, _ = slab_of(n, b, p, parts)
        B = orc.Blocked(n_slab, b_slab, h, has_f)
        for face, v in enumerate(bvals):
            B.set_boundary(face, v)          # the values on the cut ends are overwritten by every unpack
        sl = slab_slice(n, b, p, parts)
        B.set_u(np.ascontiguousarray(u0[sl]))
        if has_f:
            B.set_f(np.ascontiguousarray(f[sl]))
        out.append(B)
    return out


def _exchange_cuts(slabs):
    planes = [(S.pack_cut(0), S.pack_cut(1)) for S in slabs]
    for i, S in enumerate(slabs):
        if i > 0:
            S.unpack_cut(0, planes[i - 1][1])
        if i + 1 < len(slabs):
            S.unpack_cut(1, planes[i + 1][0])


CASES = [((24, 18), (6, 3), 1, True, 3), ((20, 16), (5, 4), 2, False, 2), ((22, 17), (8, 4), 1, True, 4),
         ((12, 10, 12), (4, 5, 3), 1, True, 2), ((10, 10, 14), (4, 4, 2), 2, False, 3), ((8, 6, 9), (4, 3, 2), 1, True, 4),
         ((16, 8), (4, 4), 1, False, 2), ((6, 6, 6), (3, 3, 3), 1, True, 2)]


@pytest.mark.parametrize("n,b,h,has_f,parts", CASES)
def test_slabs_are_the_monolithic_run_bit_for_bit(orc, n, b, h, has_f, parts):
    rng = np.random.default_rng(31)
    shape = tuple(reversed(n))
    u0, f = rng.uniform(-1, 1, shape), rng.uniform(-1, 1, shape)
    bvals = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5][: 2 * len(n)]
    mono = orc.mono_padded(n, bvals)
    mono[(slice(1, -1),) * len(n)] = u0
    slabs = _slabs(orc, n, b, h, has_f, parts, u0, f, bvals)
    for _ in range(5):
        _exchange_cuts(slabs)
        for S in slabs:
            S.sweep(1)                       # the faces between its own blocks, then the update
        mono = orc.mono_sweep(mono, f if has_f else None, 1)
    got = np.concatenate([S.get_u() for S in slabs], axis=0)
    assert np.array_equal(got, mono[(slice(1, -1),) * len(n)])
    # residual of the whole domain: the root of the sum of the slabs' squares
    _exchange_cuts(slabs)
    total = np.sqrt(sum(S.residual() ** 2 for S in slabs))
    want = orc.mono_residual(mono, f if has_f else None)
    assert abs(total - want) <= 1e-12 * want


@pytest.mark.parametrize("n,b,h", [((12, 9), (4, 3), 1), ((12, 9), (4, 3), 2), ((8, 6, 8), (4, 3, 2), 1),
                                   ((10, 7, 6), (4, 4, 3), 2)])
def test_packed_cut_planes_are_slices_of_the_field(orc, n, b, h):
    ndim = len(n)
    field = inputs.linear_index_field(n)
    B = orc.Blocked(n, b, h)
    B.set_u(field)
    g = [-(-nn // bb) for nn, bb in zip(n, b)]
    per_plane = int(np.prod(g[: ndim - 1]))
    for side in (0, 1):
        plane = B.pack_cut(side)
        fe = plane.size // per_plane
        for m in range(per_plane):
            c = [m % g[0], m // g[0]][: ndim - 1]
            ext = [min(b[a], n[a] - c[a] * b[a]) for a in range(ndim - 1)]
            sl_fast = tuple(slice(c[a] * b[a], c[a] * b[a] + ext[a]) for a in reversed(range(ndim - 1)))
            slow = slice(n[ndim - 1] - h, n[ndim - 1]) if side else slice(0, h)
            want = field[(slow,) + sl_fast]
            assert np.array_equal(plane[m * fe: m * fe + want.size].reshape(want.shape), want), (side, m)


def test_unpack_cut_touches_only_the_ghost_layers_of_that_end(orc):
    n, b, h = (8, 6, 8), (4, 3, 2), 1
    B = orc.Blocked(n, b, h)
    B.set_u(inputs.linear_index_field(n))
    before = [B.get_block_padded(k) for k in range(B.nblocks)]
    plane = -1.0 - np.arange(B.cut_elems(), dtype=np.float64)
    B.unpack_cut(1, plane)
    per_plane = B.g[0] * B.g[1]
    fe = plane.size // per_plane
    for k in range(B.nblocks):
        after = B.get_block_padded(k)
        changed = after != before[k]
        if k < B.nblocks - per_plane:
            assert not changed.any()
            continue
        m = k - (B.nblocks - per_plane)
        want = np.zeros_like(changed)
        want[b[2] + h:, h:h + b[1], h:h + b[0]] = True
        assert np.array_equal(changed, want)
        assert np.array_equal(after[b[2] + h:, h:h + b[1], h:h + b[0]].ravel(), plane[m * fe:(m + 1) * fe])


def test_slab_planes_cover_the_block_planes_evenly():
    for planes in range(1, 20):
        for parts in range(1, planes + 1):
            runs = slab_planes(planes, parts)
            assert runs[0][0] == 0 and runs[-1][1] == planes
            assert all(a[1] == b[0] for a, b in zip(runs, runs[1:]))
            sizes = [hi - lo for lo, hi in runs]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        slab_planes(3, 4)
    # only the last slab can end in a remainder plane, and only inner ends are cuts
    n, b = (8, 8, 22), (4, 4, 4)
    assert [slab_of(n, b, p, 3) for p in range(3)] == [((8, 8, 8), b, 4, 0), ((8, 8, 8), b, 6, 8), ((8, 8, 6), b, 2, 16)]
    assert slab_of((8, 8, 22), b, 5, 6) == ((8, 8, 2), (4, 4, 2), 2, 20)     # a slab that is one remainder plane
