"""The entry point for callers that cannot allocate device memory.

``jac_residual_dense_static`` takes the solver's dense arrays and needs no context and no
workspace: its scratch is a fixed array inside the library image.  A caller inside another
framework's memory pool, or a monitoring hook that must not stall the solver with a cudaMalloc,
can therefore still ask how far from converged a grid is.

The check: its result must agree with the CPU oracle's residual of the same padded grid, and with
``jac_residual`` (the context-based entry point, which reduces the same per-point residuals from
a caller-provided workspace), within the tolerance the other residual tests use, on two calls in
a row -- the second call finds the first call's numbers still in the shared scratch and must not
be disturbed by them.  This file sorts last so that a run stopping at the first failure has
already gone through every other test.
"""
import ctypes as C

import numpy as np
import pytest

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


def _reference(jac, n, b, u, f, bvals):
    with jac.Jacobi(n, b, 1, f is not None) as J:
        for face, v in enumerate(bvals):
            J.set_boundary(face, v)
        J.set_u(u)
        if f is not None:
            J.set_f(f)
        return J.residual()


# the second case is larger than the first, the third smaller again: each call meets scratch
# left behind by a call of a different size
CASES = [((300, 170), (100, 85), True), ((1024, 1536), (256, 256), False), ((40, 24, 36), (20, 12, 18), True),
         ((9, 5), (9, 5), False)]


def _oracle(orc, n, u, f, bvals):
    """The oracle's residual norm of the dense grid inside its ring of Dirichlet values."""
    padded = orc.mono_padded(n, bvals)
    padded[(slice(1, -1),) * len(n)] = u
    return orc.mono_residual(padded, f)


def test_matches_oracle_and_context_residual_on_consecutive_calls(jac, orc):
    import torch
    for n, b, has_f in CASES:
        rng = np.random.default_rng(21)
        shape = tuple(reversed(n))
        u = rng.uniform(-1, 1, shape)
        f = rng.uniform(-1, 1, shape) if has_f else None
        bvals = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5][: 2 * len(n)]
        want = _oracle(orc, n, u, f, bvals)
        by_context = _reference(jac, n, b, u, f, bvals)
        assert abs(by_context - want) <= RESID_TOL * want, (n, by_context, want)
        ud = torch.from_numpy(u).cuda()
        fd = torch.from_numpy(f).cuda() if has_f else None
        first = jac.residual_dense_static(ud, fd, bvals)
        second = jac.residual_dense_static(ud, fd, bvals)
        assert abs(first - want) <= RESID_TOL * want, (n, first, want)
        assert abs(second - want) <= RESID_TOL * want, (n, second, want)
        assert abs(first - by_context) <= RESID_TOL * by_context, (n, first, by_context)
        assert first == second            # fixed reduction order: repeatable bit for bit
        assert np.array_equal(ud.cpu().numpy(), u)   # inputs are only read


def test_zero_boundary_default_and_norm_of_f(jac):
    import torch
    f = np.random.default_rng(22).uniform(-1, 1, (64, 96))
    z = torch.zeros((64, 96), dtype=torch.float64, device="cuda")
    got = jac.residual_dense_static(z, torch.from_numpy(f).cuda(), None)
    assert got == pytest.approx(np.linalg.norm(f), rel=1e-13)


def test_rejects_bad_arguments_and_oversized_grids(jac):
    import torch
    L = jac.lib()
    u = torch.zeros((8, 8), dtype=torch.float64, device="cuda")
    out = C.c_double(-1.0)
    n_ok = (C.c_int64 * 3)(8, 8, 1)
    assert L.jac_residual_dense_static(2, n_ok, None, None, None, None, C.byref(out)) == jac.EINVAL
    assert L.jac_residual_dense_static(4, n_ok, u.data_ptr(), None, None, None, C.byref(out)) == jac.EINVAL
    assert L.jac_residual_dense_static(2, n_ok, u.data_ptr(), None, None, None, None) == jac.EINVAL
    n_zero = (C.c_int64 * 3)(8, 0, 1)
    assert L.jac_residual_dense_static(2, n_zero, u.data_ptr(), None, None, None, C.byref(out)) == jac.EINVAL
    # one point more than the fixed scratch covers: refused before anything is read
    n_big = (C.c_int64 * 3)(1 << 15, (1 << 14) + 1, 1)
    assert L.jac_residual_dense_static(2, n_big, u.data_ptr(), None, None, None, C.byref(out)) == jac.ELIMIT
    n_big3 = (C.c_int64 * 3)(1 << 10, 1 << 10, (1 << 9) + 1)
    assert L.jac_residual_dense_static(3, n_big3, u.data_ptr(), None, None, None, C.byref(out)) == jac.ELIMIT
    assert out.value == -1.0
    assert "scratch" in jac.strerror(jac.ELIMIT)
