"""Host <-> device copies through the dense staging arrays (JAC_FLAG_HOST_STAGING): the same bits
as the per-block copies, queued back to back, with the copy in running on the context's own stream."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def jac():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_01238_b200 import jac as _jac
    _jac.lib()
    return _jac


SHAPES = [((96, 64), (32, 16), 1, True), ((100, 50), (32, 16), 2, False), ((45, 31), (16, 8), 1, True),
          ((40, 24, 16), (20, 12, 8), 1, True), ((30, 20, 10), (8, 8, 4), 2, False), ((1024, 768), (256, 256), 1, False)]


@pytest.mark.parametrize("n,b,h,has_f", SHAPES)
def test_staged_copies_round_trip_and_feed_the_same_sweeps(jac, orc, n, b, h, has_f):
    rng = np.random.default_rng(5)
    shape = tuple(reversed(n))
    u0, f = rng.uniform(-1, 1, shape), rng.uniform(-1, 1, shape)
    B = orc.Blocked(n, b, h, has_f)
    B.set_u(u0)
    if has_f:
        B.set_f(f)
    B.sweep(5)
    want, want_r = B.get_u(), B.residual()
    with jac.Jacobi(n, b, h, has_f, "fused", flags=jac.FLAG_HOST_STAGING) as J:
        J.set_u(u0)
        assert np.array_equal(J.get_u(), u0)                 # in and out again, bit for bit
        for blk in range(J.nblocks):                         # and nothing but interiors was written
            pb = J.get_block_padded(blk)
            e = J.extent(blk)
            inner = tuple(slice(h, h + x) for x in reversed(e))
            mask = np.ones(pb.shape, dtype=bool)
            mask[inner] = False
            assert np.all(pb[mask] == 0.0), blk
        if has_f:
            J.set_f(f)
        J.sweep(5)
        assert np.array_equal(J.get_u(), want)
        assert abs(J.residual() - want_r) <= 1e-10 * want_r


def test_jobs_queued_back_to_back_from_pinned_memory(jac, orc):
    """Three jobs through one context without waiting in between: each copies its own input in,
    sweeps, and copies its solution out; the third reads its input from the array the first one's
    solution is still being copied into."""
    import torch
    n, b, sweeps = (512, 384), (128, 128), 7
    rng = np.random.default_rng(6)
    ins = [torch.from_numpy(rng.uniform(-1, 1, (n[1], n[0]))).pin_memory() for _ in range(2)]
    outs = [torch.zeros((n[1], n[0]), dtype=torch.float64).pin_memory() for _ in range(3)]
    norms = torch.zeros(3, dtype=torch.float64).pin_memory()

    def oracle(u0, k):
        B = orc.Blocked(n, b, 1)
        B.set_u(u0)
        B.sweep(k)
        return B.get_u(), B.residual()

    w0, r0 = oracle(ins[0].numpy(), sweeps)
    w1, r1 = oracle(ins[1].numpy(), sweeps)
    w2, r2 = oracle(w0, sweeps)                 # the third job continues from the first job's solution
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        with jac.Jacobi(n, b, 1, False, "temporal", stream=stream, flags=jac.FLAG_HOST_STAGING) as J:
            J.set_u_async(ins[0]); J.sweep(sweeps); J.residual_async(norms[0:1]); J.get_u_async(outs[0])
            J.set_u_async(ins[1]); J.sweep(sweeps); J.residual_async(norms[1:2]); J.get_u_async(outs[1])
            J.set_u_async(outs[0]); J.sweep(sweeps); J.residual_async(norms[2:3]); J.get_u_async(outs[2])
            stream.synchronize()
    assert np.array_equal(outs[0].numpy(), w0)
    assert np.array_equal(outs[1].numpy(), w1)
    assert np.array_equal(outs[2].numpy(), w2)
    for got, want in zip(norms.tolist(), (r0, r1, r2)):
        assert abs(got - want) <= 1e-10 * want


def test_first_copy_in_does_not_overtake_the_clearing_of_the_workspace(jac):
    """jac_create clears the workspace on the caller's stream; a copy in from pinned memory right
    after it runs on the context's own stream and must still come after that clearing.  With a
    workspace of a few GB the clearing takes long enough for a copy that overtook it to lose data:
    at u = 0 the residual norm is the norm of f, to the last bit of the reduction."""
    import torch
    n, b = (384, 384, 384), (128, 128, 128)
    f = np.random.default_rng(9).standard_normal((n[2], n[1], n[0]))
    fp = torch.from_numpy(f).pin_memory()
    with jac.Jacobi(n, b, 1, True, "temporal", flags=jac.FLAG_HOST_STAGING) as J:
        J._call("jac_set_f", jac.lib().jac_set_f(J._ctx, fp.data_ptr()))
        got = J.residual()
    want = float(np.sqrt(np.sum(f * f)))
    assert abs(got - want) <= 1e-12 * want
