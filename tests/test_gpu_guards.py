"""Out-of-bounds evidence without a sanitizer: the workspace sits inside a larger allocation between
two guard bands, and every byte of it that no call is entitled to write is filled with a pattern.
After every schedule the guards, the padding between the arrays, the unused tail of every block,
the ghost cells nobody fills (edges and corners), the gaps between send slots and the scratch
beyond the partial sums must still hold the pattern, bit for bit."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

GUARD = 1 << 20
PATTERN = np.array([0x7FF8DEADBEEF0001], dtype=np.uint64).view(np.float64)[0]     # a NaN with a payload


@pytest.fixture(scope="module")
def jac():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_01238_b200 import jac as _jac
    _jac.lib()
    return _jac


def _allowed_mask(J, wide):
    """Doubles of the workspace a call may write: interiors, the ghost strips of faces (all ghost
    layers in the wide schedule), the four-cell x margins next to them, f, the used part of every
    send slot, the partial sums and the result words."""
    L, d = J.layout, J.desc
    ndim, h = J.ndim, d.halo
    nd = int(L.total_bytes) // 8
    ok = np.zeros(nd, dtype=bool)
    PX, PY, PZ = int(L.pad[0]), int(L.pad[1]), int(L.pad[2])
    xpad, bs, origin = int(L.xpad), int(L.block_stride), int(L.origin)
    hz = h if ndim == 3 else 0
    arrays = [int(L.off_u[0]) // 8, int(L.off_u[1]) // 8] + ([int(L.off_f) // 8] if d.has_f else [])
    for blk in range(J.nblocks):
        e = J.extent(blk) + [1] * (3 - ndim)
        blockmask = np.zeros((PZ, PY, PX), dtype=bool)
        z0, y0, x0 = hz, h, xpad
        if wide:
            # every ghost layer, edges and corners included
            blockmask[max(z0 - hz, 0):z0 + e[2] + hz, y0 - h:y0 + e[1] + h, x0 - h:x0 + e[0] + h] = True
            blockmask[z0:z0 + e[2], y0:y0 + e[1], x0 - xpad:x0 + e[0] + xpad] = True      # plain x unpack: margin sector
        else:
            blockmask[z0:z0 + e[2], y0:y0 + e[1], x0:x0 + e[0]] = True                    # interior
            blockmask[z0:z0 + e[2], y0:y0 + e[1], x0 - xpad:x0 + e[0] + xpad] = True      # x ghosts and their margin sector
            blockmask[z0:z0 + e[2], y0 - h:y0 + e[1] + h, x0:x0 + e[0]] = True            # y ghosts
            if ndim == 3:
                blockmask[z0 - h:z0 + e[2] + h, y0:y0 + e[1], x0:x0 + e[0]] = True        # z ghosts
        flat = blockmask.ravel()
        for a in arrays:
            ok[a + blk * bs: a + blk * bs + flat.size] |= flat
    send0, ss = int(L.off_send) // 8, int(L.send_stride)
    for blk in range(J.nblocks):
        for face in range(2 * ndim):
            ne = int(L.wide_face_elems[face] if wide else L.face_elems[face])
            o = send0 + blk * ss + int(L.face_offset[face])
            ok[o:o + ne] = True
    sc = int(L.off_scratch) // 8
    ok[sc:sc + int(L.partials) + 32] = True
    return ok


CASES = [((96, 64), (32, 16), 1, True), ((100, 70), (32, 16), 2, False), ((44, 36), (12, 8), 4, True),
         ((40, 24, 16), (20, 12, 8), 1, True), ((30, 20, 14), (8, 8, 4), 2, False), ((36, 28, 12), (12, 8, 4), 3, True)]
MODES = ["fused", "exchange", "pertask", "temporal", "wide", "resident"]


@pytest.mark.parametrize("n,b,h,has_f", CASES)
@pytest.mark.parametrize("mode", MODES)
def test_nothing_outside_the_entitled_cells_is_written(jac, n, b, h, has_f, mode):
    import torch
    try:
        desc = jac.make_desc(n, b, h, has_f, mode)
        nbytes = jac.workspace_bytes(desc)
    except jac.JacError:
        pytest.skip("the schedule does not take this shape")
    big = torch.empty(nbytes + 2 * GUARD, dtype=torch.uint8, device="cuda")
    pat = torch.from_numpy(np.full(1, PATTERN)).cuda()
    big.view(torch.float64)[:] = pat                              # guards and workspace alike
    ws = big[GUARD:GUARD + nbytes]
    J = jac.Jacobi(n, b, h, has_f, mode, workspace=ws)
    J.stream.synchronize()
    ws.view(torch.float64)[:] = pat                               # jac_create cleared it: pattern again
    sc = int(J.layout.off_scratch) // 8                           # except the scratch, whose status words
    ws.view(torch.float64)[sc:sc + int(J.layout.partials) + 32] = 0.0   # the library expects as it left them
    rng = np.random.default_rng(17)
    shape = tuple(reversed(n))
    for face in range(2 * len(n)):
        J.set_boundary(face, 0.25 * (face + 1))
    J.set_u(rng.uniform(-1, 1, shape))
    if has_f:
        J.set_f(rng.uniform(-1, 1, shape))
    # every entry point of the hot path, in the context's schedule
    J.pack_halos(); J.unpack_halos(); J.exchange_halos()
    J.pack_faces(0b0011); J.unpack_faces(0b1100)
    if mode == "wide":
        J.exchange_wide()
    J.sweep(1); J.sweep(5)
    J.residual()
    J.sweep_residual(3)
    out = torch.zeros(1, dtype=torch.float64).pin_memory()
    J.residual_sweep_async(4, out)
    norms = torch.zeros(4, dtype=torch.float64).pin_memory()
    J.sweep_norms_async(9, 2, norms)
    J.sweep_norms_async(17, 8, norms)
    J.solve(7, 2, 0.0)
    J.get_u()
    J.stream.synchronize()
    after = big.cpu().numpy().view(np.uint64)
    pat_bits = np.array([PATTERN]).view(np.uint64)[0]
    g = GUARD // 8
    assert np.all(after[:g] == pat_bits), "guard band before the workspace was written"
    assert np.all(after[g + nbytes // 8:] == pat_bits), "guard band after the workspace was written"
    inside = after[g:g + nbytes // 8]
    ok = _allowed_mask(J, mode == "wide")
    assert (~ok).sum() > 0.02 * ok.size          # there is something to watch: cells no call may write
    touched = inside != pat_bits
    stray = np.flatnonzero(touched & ~ok)
    assert stray.size == 0, f"{stray.size} doubles written outside the entitled cells, first at double {stray[:5]}"
    # and the entitled cells were really reached: interiors hold numbers now
    assert touched[ok].mean() > 0.1
    J.close()
