"""GPU library vs CPU oracle, element by element, on small shapes that span several tiles and
ragged tails: sweep (every schedule), pack, unpack, residual, boundary values, data in/out.
Bars: halos and ghosts bit-exact; sweep bit-exact (the bar the library is held to is
max|du| <= 1e-12 max|u|; identical operation order makes it 0); residual rel. error <= 1e-10."""
import numpy as np
import pytest

from paper_2210_01238_b200 import inputs

pytestmark = pytest.mark.gpu

SWEEP_TOL = 1e-12
RESID_TOL = 1e-10
BVALS = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5]

# (n, b, halo): single block, many tiny blocks, odd widths (scalar path), rows longer than one
# CTA tile (x tiles), more rows than one strip (y tiles), halo 1..4
SHAPES_2D = [((12, 8), (12, 8), 1), ((12, 8), (4, 4), 1), ((12, 8), (1, 1), 1), ((15, 9), (5, 3), 1),
             ((15, 9), (5, 3), 3), ((64, 48), (16, 8), 4), ((640, 72), (640, 72), 1),
             ((1100, 200), (550, 100), 2), ((130, 210), (130, 70), 1), ((36, 24), (12, 8), 2),
             ((32, 24), (16, 8), 8), ((30, 21), (10, 7), 7)]
SHAPES_3D = [((6, 4, 8), (3, 2, 4), 1), ((6, 4, 8), (1, 1, 1), 1), ((6, 4, 8), (6, 4, 8), 2),
             ((20, 12, 40), (10, 12, 20), 1), ((132, 20, 36), (132, 10, 18), 1),
             ((24, 18, 12), (8, 6, 4), 3), ((48, 40, 20), (24, 20, 10), 2), ((16, 16, 16), (8, 8, 8), 8)]
MODES = ["fused", "exchange", "pertask"]


@pytest.fixture(scope="module")
def jac():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_01238_b200 import jac as _jac
    _jac.lib()  # raises if the library was not built
    return _jac


def _random_problem(n, seed=0):
    rng = np.random.default_rng(seed)
    shape = tuple(reversed(n))
    return rng.uniform(-1, 1, shape), rng.uniform(-1, 1, shape)


def _setup_pair(jac, orc, n, b, h, has_f, mode, seed=0, tsteps=0):
    ndim = len(n)
    u0, f = _random_problem(n, seed)
    J = jac.Jacobi(n, b, h, has_f, mode, tsteps)
    B = orc.Blocked(n, b, h, has_f)
    for face in range(2 * ndim):
        J.set_boundary(face, BVALS[face])
        B.set_boundary(face, BVALS[face])
    J.set_u(u0)
    B.set_u(u0)
    if has_f:
        J.set_f(f)
        B.set_f(f)
    return J, B


def _assert_sweep_close(got, want):
    scale = np.max(np.abs(want))
    assert np.max(np.abs(got - want)) <= SWEEP_TOL * scale
    assert np.array_equal(got, want), "same operation order should give identical bits"


@pytest.mark.parametrize("n,b,h", SHAPES_2D + SHAPES_3D)
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("has_f", [False, True])
def test_sweep_matches_oracle(jac, orc, n, b, h, mode, has_f):
    J, B = _setup_pair(jac, orc, n, b, h, has_f, mode)
    for nsw in (1, 2, 4):
        J.sweep(nsw)
        B.sweep(nsw)
        _assert_sweep_close(J.get_u(), B.get_u())
    r_gpu, r_cpu = J.residual(), B.residual()
    assert abs(r_gpu - r_cpu) <= RESID_TOL * r_cpu
    # a residual call must not disturb the state
    J.sweep(1)
    B.sweep(1)
    _assert_sweep_close(J.get_u(), B.get_u())
    J.close()
    B.close()


@pytest.mark.parametrize("n,b,h", SHAPES_2D + SHAPES_3D)
@pytest.mark.parametrize("mode", ["fused", "pertask"])
def test_pack_and_unpack_are_bit_exact(jac, orc, n, b, h, mode):
    ndim = len(n)
    J = jac.Jacobi(n, b, h, False, mode)
    B = orc.Blocked(n, b, h, False)
    dense = inputs.uniform_field(n, inputs.HALO_BENCH_SEED)
    for face in range(2 * ndim):
        J.set_boundary(face, BVALS[face])
        B.set_boundary(face, BVALS[face])
    J.set_u(dense)
    B.set_u(dense)
    J.pack_halos()
    B.pack()
    for blk in range(B.nblocks):
        for face in range(2 * ndim):
            if B.neighbour(blk, face) >= 0:
                assert np.array_equal(J.get_halo_buffer(blk, face), B.get_halo_buffer(blk, face)), (blk, face)
    J.unpack_halos()
    B.unpack()
    for blk in range(B.nblocks):
        assert np.array_equal(J.get_block_padded(blk), B.get_block_padded(blk)), blk
    J.close()
    B.close()


def test_fused_sweep_needs_no_exchange_and_leaves_ghosts_alone(jac, orc):
    """The fused schedule reads neighbour interiors directly.  No exchange ever runs here, so the
    inter-block ghosts stay at their initial zeros: a kernel that read them would get wrong values."""
    for n, b, h in [((36, 24), (12, 8), 2), ((24, 18, 12), (8, 6, 4), 3), ((15, 9), (5, 3), 1)]:
        J, B = _setup_pair(jac, orc, n, b, h, True, "fused", seed=3)
        J.sweep(3)
        B.sweep(3)
        assert np.array_equal(J.get_u(), B.get_u()), n
        J.close()
        B.close()


def test_device_resident_set_and_get(jac, orc):
    import torch
    n, b = (130, 70), (26, 14)
    u0, f = _random_problem(n, 5)
    J = jac.Jacobi(n, b, 1, True)
    J.set_u_device(torch.from_numpy(u0).cuda())
    J.set_f_device(torch.from_numpy(f).cuda())
    assert np.array_equal(J.get_u_device().cpu().numpy(), u0)
    assert np.array_equal(J.get_u(), u0)
    B = orc.Blocked(n, b, 1, True)
    B.set_u(u0)
    B.set_f(f)
    J.sweep(3)
    B.sweep(3)
    _assert_sweep_close(J.get_u_device().cpu().numpy(), B.get_u())
    J.close()


def test_residual_is_repeatable_and_matches_norm_of_f_at_zero(jac):
    n, b = (96, 80), (32, 16)
    _, f = _random_problem(n, 6)
    J = jac.Jacobi(n, b, 1, True)
    J.set_f(f)
    r = [J.residual() for _ in range(3)]
    assert r[0] == r[1] == r[2]
    assert r[0] == pytest.approx(np.linalg.norm(f), rel=1e-13)
    J.close()


def test_empty_and_error_paths(jac):
    import ctypes as C
    J = jac.Jacobi((8, 8), (4, 4))
    J.sweep(0)
    with pytest.raises(jac.JacError):
        J.sweep(-1)
    with pytest.raises(jac.JacError):
        J.set_boundary(4, 1.0)       # no z faces in 2D
    with pytest.raises(jac.JacError):
        J.get_halo_buffer(99, 0)
    with pytest.raises(jac.JacError):
        J.set_f(np.zeros((8, 8)))    # created without f
    assert jac.lib().jac_residual(J._ctx, None) == jac.EINVAL
    # undersized / misaligned workspace
    import torch
    d = jac.make_desc((8, 8), (4, 4))
    need = jac.workspace_bytes(d)
    ws = torch.empty(need + 512, dtype=torch.uint8, device="cuda")
    ctx = C.c_void_p()
    assert jac.lib().jac_create(C.byref(d), ws.data_ptr(), need - 1, C.byref(ctx)) == jac.ENOMEM
    assert jac.lib().jac_create(C.byref(d), ws.data_ptr() + 8, need, C.byref(ctx)) == jac.ENOMEM
    assert not ctx.value
    J.close()


def test_launch_counts_per_schedule(jac):
    """fused: one launch per sweep; exchange: three; per-task: one per
    block face with a neighbour, twice, plus one per block."""
    n, b = (32, 24), (8, 8)   # 4 x 3 blocks, interior faces: 2*(3*3 + 4*2) = 34
    counts = {}
    for mode in MODES:
        J = jac.Jacobi(n, b, 1, False, mode)
        J.set_u(np.zeros((24, 32)))
        c0 = J.launch_count()
        J.sweep(5)
        counts[mode] = J.launch_count() - c0
        J.close()
    assert counts["fused"] == 5
    assert counts["exchange"] == 2 * 5
    assert counts["pertask"] == 5 * (2 * 34 + 12)


# temporal blocking: widths that leave ragged strips (120 columns per warp), several row strips,
# blocks narrower and wider than a strip, every depth, sweep counts that leave a remainder
TEMPORAL_SHAPES = [((8, 8), (4, 4)), ((120, 40), (60, 20)), ((124, 33), (124, 33)),
                   ((256, 100), (64, 25)), ((1100, 200), (220, 50)), ((36, 24), (12, 8)),
                   ((480, 96), (4, 1)), ((2048, 300), (1024, 150))]


@pytest.mark.parametrize("n,b", TEMPORAL_SHAPES)
@pytest.mark.parametrize("tsteps", [1, 2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("has_f", [False, True])
def test_temporal_blocking_matches_oracle(jac, orc, n, b, tsteps, has_f):
    J, B = _setup_pair(jac, orc, n, b, 1, has_f, "temporal", seed=2, tsteps=tsteps)
    for nsw in (1, 4, 17):
        J.sweep(nsw)
        B.sweep(nsw)
        _assert_sweep_close(J.get_u(), B.get_u())
    r_gpu, r_cpu = J.residual(), B.residual()
    assert abs(r_gpu - r_cpu) <= RESID_TOL * r_cpu
    J.sweep(5)
    B.sweep(5)
    _assert_sweep_close(J.get_u(), B.get_u())
    J.close()
    B.close()


# 3D: tiles are 60 (T = 3: 56) x (32 - 2T) outputs wide and stream z in chunks: shapes with ragged
# tiles in x and y, several z chunks, blocks smaller and larger than a tile, nonzero Dirichlet values
TEMPORAL_SHAPES_3D = [((8, 8, 8), (4, 4, 4)), ((24, 18, 12), (8, 6, 4)), ((64, 48, 40), (32, 24, 20)),
                      ((130, 100, 36), (130, 50, 18)), ((132, 20, 70), (66, 10, 35)),
                      ((256, 128, 24), (128, 128, 8)), ((62, 46, 20), (2, 2, 2)), ((120, 56, 300), (60, 28, 100)),
                      ((58, 27, 9), (58, 27, 9))]


@pytest.mark.parametrize("n,b", TEMPORAL_SHAPES_3D)
@pytest.mark.parametrize("tsteps", [1, 2, 3])
@pytest.mark.parametrize("has_f", [False, True])
def test_temporal_blocking_3d_matches_oracle(jac, orc, n, b, tsteps, has_f):
    J, B = _setup_pair(jac, orc, n, b, 1, has_f, "temporal", seed=4, tsteps=tsteps)
    for nsw in (1, 2, 5):
        J.sweep(nsw)
        B.sweep(nsw)
        _assert_sweep_close(J.get_u(), B.get_u())
    r_gpu, r_cpu = J.residual(), B.residual()
    assert abs(r_gpu - r_cpu) <= RESID_TOL * r_cpu
    J.sweep(4)
    B.sweep(4)
    _assert_sweep_close(J.get_u(), B.get_u())
    J.close()
    B.close()


def test_temporal_mode_rejects_unsupported_shapes(jac):
    with pytest.raises(jac.JacError):
        jac.Jacobi((12, 8), (6, 4), mode="temporal")          # 2D: bx % 4 != 0
    with pytest.raises(jac.JacError):
        jac.Jacobi((9, 8, 8), (3, 4, 4), mode="temporal")     # 3D: bx % 2 != 0
    with pytest.raises(jac.JacError):
        jac.Jacobi((8, 8, 8), (4, 4, 4), mode="temporal", tsteps=4)   # 3D: at most 3 sweeps per launch


def test_partial_exchange_by_face_mask(jac, orc):
    """x faces first, then y (and z): the result equals one full exchange; bad masks are refused."""
    for n, b, h in [((36, 24), (12, 8), 2), ((24, 18, 12), (8, 6, 4), 1)]:
        ndim = len(n)
        dense = inputs.uniform_field(n, 4)
        J = jac.Jacobi(n, b, h, False, "exchange")
        B = orc.Blocked(n, b, h, False)
        J.set_u(dense)
        B.set_u(dense)
        B.pack()
        B.unpack()
        J.pack_faces(0b11)
        J.unpack_faces(0b11)
        # only x ghosts are filled so far
        for blk in range(B.nblocks):
            got, want = J.get_block_padded(blk), B.get_block_padded(blk)
            sl = [slice(h, -h)] * ndim
            assert np.array_equal(got[tuple(sl)][..., :], want[tuple(sl)][..., :])
            ysl = list(sl); ysl[ndim - 2] = slice(0, h)
            assert np.all(got[tuple(ysl)] == 0.0)
        rest = (1 << (2 * ndim)) - 1 - 0b11
        J.pack_faces(rest)
        J.unpack_faces(rest)
        for blk in range(B.nblocks):
            assert np.array_equal(J.get_block_padded(blk), B.get_block_padded(blk))
        with pytest.raises(jac.JacError):
            J.pack_faces(1 << (2 * ndim))
        J.close()
        B.close()


def test_sweeps_per_launch_query(jac):
    cases = [(dict(n=(64, 64), b=(32, 32), mode="exchange"), 1),
             (dict(n=(64, 64), b=(32, 32), mode="temporal", tsteps=3), 3),
             (dict(n=(64, 64), b=(32, 32), mode="temporal"), 4),            # small grid: 4
             (dict(n=(64, 64), b=(32, 32), mode="temporal", has_f=True), 6),
             (dict(n=(16, 16, 16), b=(8, 8, 8), mode="temporal"), 3)]
    for kw, want in cases:
        with jac.Jacobi(**kw) as J:
            assert J.sweeps_per_launch() == want, kw


FUSED_RESIDUAL_CASES = [((36, 24), (12, 8), 1), ((256, 100), (64, 25), 1), ((1100, 200), (220, 50), 2),
                        ((24, 18, 12), (8, 6, 4), 1), ((130, 100, 36), (130, 50, 18), 1),
                        ((64, 48, 40), (32, 24, 20), 2)]


@pytest.mark.parametrize("n,b,h", FUSED_RESIDUAL_CASES)
@pytest.mark.parametrize("mode", ["fused", "exchange", "pertask", "temporal"])
@pytest.mark.parametrize("has_f", [False, True])
def test_sweep_with_fused_residual(jac, orc, n, b, h, mode, has_f):
    """jac_sweep_residual(k): state after k sweeps, norm of the residual of the state after k - 1."""
    J, B = _setup_pair(jac, orc, n, b, h, has_f, mode, seed=6)
    for k in (1, 3, 6):
        B.sweep(k - 1)
        want_r = B.residual()
        B.sweep(1)
        got_r = J.sweep_residual(k)
        assert abs(got_r - want_r) <= RESID_TOL * want_r, (k, got_r, want_r)
        _assert_sweep_close(J.get_u(), B.get_u())
    # an ordinary residual afterwards still works and agrees
    assert abs(J.residual() - B.residual()) <= RESID_TOL * B.residual()
    J.close()
    B.close()


@pytest.mark.parametrize("n,b,h", FUSED_RESIDUAL_CASES + [((480, 96), (4, 1), 1), ((120, 56, 70), (60, 28, 35), 1)])
@pytest.mark.parametrize("mode,tsteps", [("fused", 0), ("exchange", 0), ("pertask", 0), ("temporal", 0), ("temporal", 2),
                                         ("temporal", 1), ("wide", 0)])
@pytest.mark.parametrize("has_f", [False, True])
def test_residual_from_the_first_sweep_s_pass(jac, orc, n, b, h, mode, tsteps, has_f):
    """jac_residual_sweep_async(k): the norm of the residual of the state BEFORE the k sweeps, then the
    state after them."""
    import torch
    J, B = _setup_pair(jac, orc, n, b, h, has_f, mode, seed=8, tsteps=tsteps)
    norms = torch.zeros(3, dtype=torch.float64).pin_memory()
    want = []
    for i, k in enumerate((1, 4, 10)):
        want.append(B.residual())
        B.sweep(k)
        J.residual_sweep_async(k, norms[i:i + 1])
    got_u = J.get_u()              # waits for the stream
    _assert_sweep_close(got_u, B.get_u())
    for got_r, want_r in zip(norms.tolist(), want):
        assert abs(got_r - want_r) <= RESID_TOL * want_r, (got_r, want_r)
    assert abs(J.residual() - B.residual()) <= RESID_TOL * B.residual()
    J.close()
    B.close()


# (n, b, mode, tsteps, nsweeps, every): norms due inside launches (every > T, no multiple of T), at
# launch borders (every = T), every < T (group by group), nothing due (nsweeps <= every), many norms
NORM_CASES = [((120, 40), (60, 20), "temporal", 3, 23, 5), ((256, 100), (64, 25), "temporal", 8, 50, 10),
              ((256, 100), (64, 25), "temporal", 6, 31, 10), ((1100, 200), (220, 50), "temporal", 4, 17, 4),
              ((36, 24), (12, 8), "temporal", 4, 9, 2), ((36, 24), (12, 8), "temporal", 0, 7, 7),
              ((120, 40), (60, 20), "temporal", 2, 110, 2),      # 54 norms: more than travel in one copy
              ((36, 24), (12, 8), "fused", 0, 11, 3), ((36, 24), (12, 8), "exchange", 0, 7, 2),
              ((64, 48), (64, 48), "resident", 0, 9, 4),
              ((40, 36, 30), (20, 12, 10), "temporal", 3, 22, 5), ((40, 36, 30), (20, 12, 10), "temporal", 2, 9, 3),
              ((40, 36, 30), (20, 12, 10), "temporal", 3, 10, 3), ((24, 18, 12), (8, 6, 4), "fused", 0, 7, 3)]


@pytest.mark.parametrize("n,b,mode,tsteps,nsweeps,every", NORM_CASES)
@pytest.mark.parametrize("has_f", [False, True])
def test_norms_every_k_sweeps_from_the_sweeps_own_passes(jac, orc, n, b, mode, tsteps, nsweeps, every, has_f):
    """jac_sweep_norms_async: the norm of the state after every, 2 * every, ... sweeps equals the oracle's
    residual at that point, whichever level of whichever launch measures it, and the sweeps themselves
    leave the oracle's bits."""
    import torch
    J, B = _setup_pair(jac, orc, n, b, 1, has_f, mode, seed=9, tsteps=tsteps)
    need = (nsweeps - 1) // every
    out = torch.full((max(need, 1) + 1,), -7.0, dtype=torch.float64).pin_memory()
    J.sweep_norms_async(nsweeps, every, out if need else None)
    torch.cuda.synchronize()
    want = []
    done = 0
    while done < nsweeps:
        k = min(every, nsweeps - done)
        B.sweep(k)
        done += k
        if done < nsweeps:
            want.append(B.residual())
    assert len(want) == need
    for m in range(need):
        assert abs(float(out[m]) - want[m]) <= RESID_TOL * want[m], (m, float(out[m]), want[m])
    assert float(out[need]) == -7.0                       # nothing written past the norms that are due
    _assert_sweep_close(J.get_u(), B.get_u())
    r, w = J.residual(), B.residual()
    assert abs(r - w) <= RESID_TOL * w
    J.close()
    B.close()


@pytest.mark.parametrize("mode", ["temporal", "fused", "exchange", "pertask", "resident", "wide"])
def test_solve_stops_after_the_group_that_meets_the_tolerance(jac, orc, mode):
    """Groups of 3 sweeps, the tolerance met in the middle of a batch of queued groups (and, with a
    loose tolerance, in the very first group); a tolerance never met runs max_sweeps, the last
    group shorter."""
    n, b = (48, 40), (24, 20)
    u0, f = _random_problem(n, 10)

    def oracle_after(k):
        B = orc.Blocked(n, b, 1, True)
        B.set_u(u0)
        B.set_f(f)
        B.sweep(k - 1)
        r = B.residual()
        B.sweep(1)
        out = B.get_u(), r
        B.close()
        return out

    with jac.Jacobi(n, b, 1, True, mode) as J:
        J.set_u(u0); J.set_f(f)
        r0 = J.residual()
    for tol, max_sweeps in ((0.12 * r0, 500), (10.0 * r0, 500), (0.0, 20)):
        with jac.Jacobi(n, b, 1, True, mode) as J:
            J.set_u(u0); J.set_f(f)
            done, res = J.solve(max_sweeps, 3, tol)
            got = J.get_u()
            after = J.residual()
        want_u, want_r = oracle_after(done)
        assert res <= tol or done == max_sweeps
        assert done % 3 == 0 or done == max_sweeps
        assert abs(res - want_r) <= RESID_TOL * want_r
        assert np.array_equal(got, want_u), (mode, tol, done)
        assert after > 0
        if tol == 10.0 * r0:
            assert done == 3
        if tol == 0.12 * r0:
            assert done == 33          # the eleventh group: the third of the second batch of queued groups
            prev_u, prev_r = oracle_after(done - 3)     # the group before had not met it yet
            assert prev_r > tol


def test_solve_stops_at_the_tolerance(jac, orc):
    n, b = (48, 40), (24, 20)
    u0, f = _random_problem(n, 9)
    for mode in ("temporal", "fused"):
        J = jac.Jacobi(n, b, 1, True, mode)
        J.set_u(u0)
        J.set_f(f)
        r0 = J.residual()
        done, res = J.solve(100000, 50, 1e-6 * r0)
        assert res <= 1e-6 * r0 and done % 50 == 0 and 50 <= done < 100000
        # the oracle at the same sweep count: the reported norm is that of the state one sweep earlier
        B = orc.Blocked(n, b, 1, True)
        B.set_u(u0)
        B.set_f(f)
        B.sweep(done - 1)
        want = B.residual()
        B.sweep(1)
        assert abs(res - want) <= RESID_TOL * want
        assert np.array_equal(J.get_u(), B.get_u())
        # a cap below convergence is honoured
        J.set_u(u0)
        done2, res2 = J.solve(30, 8, 0.0)
        assert done2 == 30 and res2 > 0.0
        with pytest.raises(jac.JacError):
            J.solve(0, 8, 1.0)
        J.close()
        B.close()


def test_work_is_issued_on_the_callers_stream(jac, orc):
    """A context created on a side stream runs there: results are right, and two contexts on two
    streams do not disturb each other."""
    import torch
    n, b, h = (130, 70), (130, 70), 1
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    u0, f = _random_problem(n, 3)
    B = orc.Blocked(n, b, h, True)
    B.set_u(u0); B.set_f(f)
    J1 = jac.Jacobi(n, b, h, True, "fused", stream=s1)
    J2 = jac.Jacobi(n, b, h, True, "exchange", stream=s2)
    assert J1.desc.stream == s1.cuda_stream and J2.desc.stream == s2.cuda_stream
    for J in (J1, J2):
        J.set_u(u0); J.set_f(f)
    for _ in range(5):          # interleave the two streams' launches
        J1.sweep(1); J2.sweep(1)
    B.sweep(5)
    want = B.get_u()
    assert np.array_equal(J1.get_u(), want) and np.array_equal(J2.get_u(), want)
    r = B.residual()
    assert abs(J1.residual() - r) <= RESID_TOL * r and abs(J2.residual() - r) <= RESID_TOL * r
    J1.close(); J2.close(); B.close()


def test_asynchronous_copies_and_residual_pipeline(jac, orc):
    """jac_set_u_async / jac_get_u_async / jac_residual_async on two contexts and two streams,
    several jobs in flight with no host wait in between: every job's solution and norm are those
    of the blocking calls, bit for bit."""
    import torch
    n, b, h = (256, 140), (128, 70), 1
    rng = np.random.default_rng(5)
    f = rng.uniform(-1, 1, (140, 256))
    inputs_u = [rng.uniform(-1, 1, (140, 256)) for _ in range(4)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    ctxs = [jac.Jacobi(n, b, h, True, "temporal", stream=s) for s in streams]
    for J in ctxs:
        J.set_f(f)
    host_in = [torch.from_numpy(u).pin_memory() for u in inputs_u]
    host_out = [torch.empty(140, 256, dtype=torch.float64).pin_memory() for _ in range(4)]
    norms = [torch.zeros(1, dtype=torch.float64).pin_memory() for _ in range(4)]
    for k in range(4):
        J = ctxs[k % 2]
        J.set_u_async(host_in[k])
        J.sweep(9)
        J.residual_async(norms[k])
        J.get_u_async(host_out[k])
    for s in streams:
        s.synchronize()
    for k in range(4):
        B = orc.Blocked(n, b, h, True)
        B.set_u(inputs_u[k]); B.set_f(f)
        B.sweep(9)
        assert np.array_equal(host_out[k].numpy(), B.get_u()), k
        want = B.residual()
        assert abs(float(norms[k][0]) - want) <= RESID_TOL * want
        B.close()
    # the asynchronous norm has the bits of the blocking one
    J = ctxs[0]
    J.set_u(inputs_u[0]); J.sweep(3)
    r = J.residual()
    J.residual_async(norms[0]); streams[0].synchronize()
    assert float(norms[0][0]) == r
    with pytest.raises(AssertionError):
        J.set_u_async(torch.from_numpy(inputs_u[0]))      # pageable memory is refused by the binding
    for J in ctxs:
        J.close()


@pytest.mark.parametrize("n,b,h", SHAPES_2D + SHAPES_3D + [((14, 11), (4, 4), 2), ((9, 5, 7), (4, 2, 3), 1)])
def test_one_launch_exchange_leaves_what_pack_and_unpack_leave(jac, orc, n, b, h):
    ndim = len(n)
    dense = inputs.linear_index_field(n)
    A = jac.Jacobi(n, b, h, False, "exchange")
    B = orc.Blocked(n, b, h)
    for face in range(2 * ndim):
        A.set_boundary(face, BVALS[face]); B.set_boundary(face, BVALS[face])
    A.set_u(dense); B.set_u(dense)
    A.exchange_halos()
    B.pack(); B.unpack()
    for blk in range(B.nblocks):
        for face in range(2 * ndim):
            if B.neighbour(blk, face) >= 0:
                assert np.array_equal(A.get_halo_buffer(blk, face), B.get_halo_buffer(blk, face)), (blk, face)
        assert np.array_equal(A.get_block_padded(blk), B.get_block_padded(blk)), blk
    assert np.array_equal(A.get_u(), dense)
    A.close(); B.close()
