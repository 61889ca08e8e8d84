"""One domain as several slab contexts (the multi-GPU sharding, exercised on one device): every
slab is a context of its own on its own stream, the cut faces are packed by one slab and read in
place by its neighbour's unpack, and the result is the unpartitioned oracle's, bit for bit."""
import numpy as np
import pytest

from paper_2210_01238_b200 import inputs
from paper_2210_01238_b200.sharded import LocalSlabs, set_slab_boundary, slab_context, slab_of, slab_slice

pytestmark = pytest.mark.gpu

RESID_TOL = 1e-10


@pytest.fixture(scope="module")
def jac():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_01238_b200 import jac as _jac
    _jac.lib()
    return _jac


def _engines(n, b, h, has_f, mode, parts, u0, f, bvals):
    import torch
    out = []
    for p in range(parts):
        J = slab_context(n, b, h, has_f, mode, p, parts, stream=torch.cuda.Stream())
        set_slab_boundary(J, len(n), p, parts, bvals)
        sl = slab_slice(n, b, p, parts)
        J.set_u(np.ascontiguousarray(u0[sl]))
        if has_f:
            J.set_f(np.ascontiguousarray(f[sl]))
        out.append(J)
    return out


def _oracle(orc, n, b, h, has_f, u0, f, bvals, sweeps):
    B = orc.Blocked(n, b, h, has_f)
    for face, v in enumerate(bvals):
        B.set_boundary(face, v)
    B.set_u(u0)
    if has_f:
        B.set_f(f)
    B.sweep(sweeps)
    out = B.get_u(), B.residual()
    B.close()
    return out


CASES = [((96, 64), (32, 16), 1, True, 2), ((96, 64), (32, 16), 2, False, 4), ((100, 70), (32, 16), 1, True, 3),
         ((40, 24, 16), (20, 12, 4), 1, True, 2), ((40, 24, 16), (20, 12, 4), 1, False, 4),
         ((30, 20, 14), (8, 8, 4), 2, True, 3), ((64, 64, 48), (32, 32, 8), 1, True, 6),
         ((16, 16, 8), (8, 8, 4), 1, False, 2)]


@pytest.mark.parametrize("mode", ["fused", "exchange"])
@pytest.mark.parametrize("n,b,h,has_f,parts", CASES)
def test_slab_contexts_match_the_unpartitioned_oracle(jac, orc, n, b, h, has_f, parts, mode):
    rng = np.random.default_rng(41)
    shape = tuple(reversed(n))
    u0, f = rng.uniform(-1, 1, shape), rng.uniform(-1, 1, shape)
    bvals = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5][: 2 * len(n)]
    sweeps = 7
    want, want_r = _oracle(orc, n, b, h, has_f, u0, f, bvals, sweeps)
    engines = _engines(n, b, h, has_f, mode, parts, u0, f, bvals)
    S = LocalSlabs(engines)
    S.sweep(3)
    S.sweep(sweeps - 3)
    got = np.concatenate([J.get_u() for J in engines], axis=0)
    assert np.array_equal(got, want)
    r = S.residual(lambda J: J.residual_sumsq())
    assert abs(r - want_r) <= RESID_TOL * want_r
    for J in engines:
        J.close()


def test_packed_cut_planes_and_cut_ghosts_are_the_oracle_s(jac, orc):
    """The planes a slab packs equal the oracle's packed cut planes, and after the exchange the
    ghost layers on a cut hold the neighbouring slab's interior layers."""
    n, b, h, parts = (48, 40, 24), (16, 20, 4), 2, 3
    field = inputs.linear_index_field(n)
    engines = _engines(n, b, h, False, "exchange", parts, field, None, [0.0] * 6)
    S = LocalSlabs(engines)
    S.start()
    for p, J in enumerate(engines):
        n_slab, b_slab, _, _ = slab_of(n, b, p, parts)
        O = orc.Blocked(n_slab, b_slab, h)
        O.set_u(np.ascontiguousarray(field[slab_slice(n, b, p, parts)]))
        per_plane = O.g[0] * O.g[1]
        for side in (0, 1):
            if (side == 0 and p == 0) or (side == 1 and p == parts - 1):
                continue
            got = J.cut_send(side).cpu().numpy().reshape(per_plane, -1)
            want = O.pack_cut(side).reshape(per_plane, -1)
            assert np.array_equal(got[:, : want.shape[1]], want), (p, side)
        # ghosts on the cuts: the padded global field's window
        J.stream.synchronize()
        first = slab_of(n, b, p, parts)[3]
        for blk in range(J.nblocks):
            pb = J.get_block_padded(blk)
            c = [blk % O.g[0], (blk // O.g[0]) % O.g[1], blk // per_plane]
            x0, y0 = c[0] * b_slab[0], c[1] * b_slab[1]
            if c[2] == 0 and p > 0:
                want = field[first - h:first, y0:y0 + b_slab[1], x0:x0 + b_slab[0]]
                assert np.array_equal(pb[:h, h:-h, h:-h], want), (p, blk)
            if c[2] == O.g[2] - 1 and p + 1 < parts:
                z1 = first + n_slab[2]
                want = field[z1:z1 + h, y0:y0 + b_slab[1], x0:x0 + b_slab[0]]
                assert np.array_equal(pb[-h:, h:-h, h:-h], want), (p, blk)
        O.close()
    for J in engines:
        J.close()


def test_calls_out_of_order_are_refused(jac):
    import ctypes as C
    L = jac.lib()
    with jac.Jacobi((32, 32), (16, 16), 1, False, "fused") as J:       # no cuts
        assert L.jac_sweep_begin(J._ctx) == jac.EINVAL
        assert L.jac_pack_cut(J._ctx) == jac.EINVAL
        assert L.jac_cut_info(J._ctx, 0, None, None, None, None) == jac.EINVAL
    with jac.Jacobi((32, 32), (16, 16), 1, False, "fused", flags=jac.FLAG_CUT_HI) as J:
        assert L.jac_sweep(J._ctx, 1) == jac.EINVAL                     # a slab sweeps in two halves
        assert L.jac_sweep_begin(J._ctx) == jac.EINVAL                  # cut ghosts not current yet
        assert L.jac_sweep_end(J._ctx, None, None, None, None) == jac.EINVAL
        assert L.jac_set_boundary(J._ctx, 3, C.c_double(1.0)) == jac.EINVAL   # the cut is no domain face
        assert L.jac_cut_info(J._ctx, 0, None, None, None, None) == jac.EINVAL
        out = C.c_double(0.0)
        assert L.jac_residual(J._ctx, C.byref(out)) == jac.EINVAL
        J.pack_cut(); J.unpack_cut()
        J.sweep_begin()
        assert L.jac_sweep_begin(J._ctx) == jac.EINVAL
        assert L.jac_pack_cut(J._ctx) == jac.EINVAL
        J.sweep_end()
    for mode in ("temporal", "wide", "pertask", "resident"):
        with pytest.raises(jac.JacError):
            jac.workspace_bytes(jac.make_desc((32, 32), (16, 16), 1, False, mode, flags=jac.FLAG_CUT_LO))


def test_config5_recipe_at_256_and_the_paper_shape_at_a_quarter(jac, orc):
    """Config 5's recipe at 256^3 in 64^3 blocks as 2 and 4 slabs, and the paper's strong-scaling
    shape at a quarter of its edge (256 x 256 x 192 in 32^3 blocks) as 3 slabs."""
    for n, b, parts in (((256, 256, 256), (64, 64, 64), 2), ((256, 256, 256), (64, 64, 64), 4),
                        ((256, 256, 192), (32, 32, 32), 3)):
        w = inputs.scaled(inputs.POISSON3D_1024, n, b, sweeps=20)
        f = inputs.rhs(w)
        u0 = inputs.initial_u(w)
        want, want_r = _oracle(orc, n, b, 1, True, u0, f, [0.0] * 6, w.sweeps)
        engines = _engines(n, b, 1, True, "fused", parts, u0, f, [0.0] * 6)
        S = LocalSlabs(engines)
        S.sweep(w.sweeps)
        got = np.concatenate([J.get_u() for J in engines], axis=0)
        assert np.array_equal(got, want), (n, parts)
        r = S.residual(lambda J: J.residual_sumsq())
        assert abs(r - want_r) <= RESID_TOL * want_r
        for J in engines:
            J.close()
