"""The resident schedule (whole grid in the shared memory of one thread-block cluster, all
sweeps of a call in one launch) against the CPU oracle: bit-exact interiors, residual 1e-10."""
import numpy as np
import pytest

from paper_2210_01238_b200 import inputs

pytestmark = pytest.mark.gpu

BVALS = [0.5, -1.0, 2.0, 3.0]
RESID_TOL = 1e-10

# (n, b, halo): one block; many blocks; fewer rows than CTAs in the cluster; row counts that do
# not divide by the cluster size (a short last slab, empty CTAs); slabs of more rows than one
# work item marches (8); a grid that needs a cluster of 16; the widest rows that still fit
SHAPES = [((12, 8), (12, 8), 1), ((12, 4), (4, 4), 1), ((64, 48), (16, 8), 2), ((36, 21), (12, 7), 1),
          ((256, 256), (256, 256), 1), ((256, 256), (64, 32), 1), ((130, 70), (130, 70), 1),
          ((20, 9), (10, 3), 3), ((512, 256), (128, 64), 1), ((1400, 64), (700, 32), 1),
          ((32, 200), (16, 50), 1), ((6, 1), (2, 1), 1)]


@pytest.fixture(scope="module")
def jac():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_01238_b200 import jac as _jac
    _jac.lib()
    return _jac


@pytest.mark.parametrize("n,b,h", SHAPES)
@pytest.mark.parametrize("has_f", [False, True])
def test_resident_schedule_matches_oracle_bitwise(jac, orc, n, b, h, has_f):
    rng = np.random.default_rng(1)
    shape = tuple(reversed(n))
    u0, f = rng.uniform(-1, 1, shape), rng.uniform(-1, 1, shape)
    try:
        J = jac.Jacobi(n, b, h, has_f, "resident")
    except jac.JacError as e:          # only the capacity rule may refuse one of these shapes
        assert e.code == jac.EINVAL and has_f and n == (1400, 64)
        return
    B = orc.Blocked(n, b, h, has_f)
    for face in range(4):
        J.set_boundary(face, BVALS[face]); B.set_boundary(face, BVALS[face])
    J.set_u(u0); B.set_u(u0)
    if has_f:
        J.set_f(f); B.set_f(f)
    before = J.launch_count()
    J.sweep(1); J.sweep(6); J.sweep(13)
    assert J.launch_count() - before == 3          # one launch per call, however many sweeps
    B.sweep(20)
    assert np.array_equal(J.get_u(), B.get_u())
    r, want = J.residual(), B.residual()
    assert abs(r - want) <= RESID_TOL * want
    # the lagged residual rides on one ordinary launch after the resident one
    r = J.sweep_residual(5)
    B.sweep(4)
    want = B.residual()
    assert abs(r - want) <= RESID_TOL * want
    B.sweep(1)
    assert np.array_equal(J.get_u(), B.get_u())
    J.close(); B.close()


def test_resident_heated_edge_256_100_sweeps(jac, orc):
    w = inputs.CONFIGS["c1_heated_edge_256"]
    with jac.Jacobi(w.n, w.b, w.halo, w.has_f, "resident") as J:
        B = orc.Blocked(w.n, w.b, w.halo, w.has_f)
        for face, v in enumerate(w.boundary()):
            J.set_boundary(face, v); B.set_boundary(face, v)
        J.set_u(inputs.initial_u(w)); B.set_u(inputs.initial_u(w))
        J.sweep(w.sweeps); B.sweep(w.sweeps)
        got = J.get_u()
        assert np.array_equal(got, B.get_u())
        assert np.array_equal(got, got[:, ::-1])            # mirror symmetry holds bit for bit
        assert abs(J.residual() - B.residual()) <= RESID_TOL * B.residual()
        B.close()


def test_resident_refusals(jac):
    for n, b in [((1024, 1024), (512, 512)), ((15, 8), (5, 4)), ((12, 8, 8), (4, 4, 4))]:
        with pytest.raises(jac.JacError) as e:
            jac.Jacobi(n, b, 1, False, "resident")
        assert e.value.code == jac.EINVAL


def test_a_given_up_wait_is_reported_and_sticks(jac):
    """The status word a CTA raises when it has polled its mbarrier to the limit is what the host
    looks at after it has waited for the stream: raise it by hand (no kernel is made to wait) and the
    next such call returns JAC_ETIMEOUT, as does every call after it."""
    import ctypes as C
    import torch
    with jac.Jacobi((64, 64), (64, 64), 1, False, "resident") as J:
        J.sweep(3)
        assert J.residual() >= 0.0
        word = int(J.layout.off_scratch) // 8 + int(J.layout.partials) + 4
        J.stream.synchronize()
        J.workspace.view(torch.int32)[2 * word] = 1
        out = C.c_double(0.0)
        L = jac.lib()
        assert L.jac_residual(J._ctx, C.byref(out)) == jac.ETIMEOUT
        assert L.jac_sweep(J._ctx, 1) == jac.ETIMEOUT
        assert "wait" in jac.strerror(jac.ETIMEOUT)
