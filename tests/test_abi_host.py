"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and its pure-host queries (validation, layout, error strings) behave."""
import ctypes as C
import re
from pathlib import Path

import numpy as np
import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def jac():
    from paper_2210_01238_b200 import build, jac as _jac
    build.build()
    return _jac


def _declared_symbols():
    names = set()
    for hdr in sorted((ROOT / "include").glob("*.h")):
        text = re.sub(r"/\*.*?\*/", "", hdr.read_text(), flags=re.S)
        names |= set(re.findall(r"\b(jac_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol(jac):
    L = C.CDLL(str(jac.LIB_PATH))
    declared = _declared_symbols()
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(L, name), f"{name} is declared in include/ but not exported"
    assert sorted(jac.EXPORTS) == declared


def test_strerror(jac):
    assert jac.strerror(0) == "ok"
    for code in (-1, -2, -3, -4, -5, -6):
        assert jac.strerror(code) not in ("ok", "unknown error code")
    assert jac.strerror(-99) == "unknown error code"


@pytest.mark.parametrize("kw", [
    dict(n=(13, 8), b=(4, 4), halo=2),    # remainder block (1 point) narrower than the halo
    dict(n=(14, 8), b=(4, 4), mode="temporal"),                 # temporal 2D wants n[0] % 4 == 0 ...
    dict(n=(14, 8), b=(4, 4), mode="resident", halo=1, tsteps=3),  # a cluster size that is neither 8 nor 16
    dict(n=(12, 8), b=(4, 4), halo=0),
    dict(n=(12, 8), b=(4, 4), halo=5),    # wider than the block
    dict(n=(12, 8), b=(4, 4), halo=9),
    dict(n=(12, 8), b=(0, 4)),
    dict(n=(12, 8), b=(24, 8)),
    dict(n=(12, 8), b=(4, 4), mode=7),
    dict(n=(12, 8), b=(4, 4), tsteps=9),
    dict(n=(12,), b=(4,)),                # ndim 1
    dict(n=(12, 8), b=(4, 4), halo=2, mode="wide", tsteps=3),   # more sweeps per exchange than ghost layers
    dict(n=(12, 8, 8), b=(4, 4, 4), mode="resident"),           # the resident schedule is 2D only,
    dict(n=(15, 8), b=(5, 4), mode="resident"),                 # wants an even block width
    dict(n=(1024, 1024), b=(512, 512), mode="resident"),        # and a grid that fits a cluster's shared memory
])
def test_invalid_descriptors_are_rejected(jac, kw):
    d = jac.make_desc(**kw)
    with pytest.raises(jac.JacError) as e:
        jac.workspace_bytes(d)
    assert e.value.code == jac.EINVAL


def test_null_arguments(jac):
    L = jac.lib()
    d = jac.make_desc((8, 8), (4, 4))
    out = C.c_size_t(123)
    assert L.jac_workspace_bytes(None, C.byref(out)) == jac.EINVAL
    assert L.jac_workspace_bytes(C.byref(d), None) == jac.EINVAL
    assert out.value == 123
    assert L.jac_sweep(None, 1) == jac.EINVAL
    assert L.jac_destroy(None) == jac.EINVAL
    ctx = C.c_void_p()
    assert L.jac_create(C.byref(d), None, 1 << 20, C.byref(ctx)) == jac.ENOMEM
    assert not ctx.value


@pytest.mark.parametrize("n,b,h,has_f", [((16384, 16384), (1024, 1024), 1, False),
                                          ((4096, 4096), (512, 512), 1, True),
                                          ((1024, 1024, 1024), (128, 128, 128), 1, True),
                                          ((12, 8), (3, 2), 2, True), ((9, 5, 7), (3, 5, 1), 1, False),
                                          ((14, 11), (4, 4), 2, True), ((10, 9, 7), (4, 4, 3), 1, False),
                                          ((256, 256), (64, 64), 4, False)])
def test_layout_is_aligned_and_disjoint(jac, n, b, h, has_f):
    d = jac.make_desc(n, b, h, has_f)
    L = jac.get_layout(d)
    ndim = len(n)
    assert L.nblocks == int(np.prod([-(-nn // bb) for nn, bb in zip(n, b)]))
    assert L.xpad >= h and L.xpad % 4 == 0
    assert L.pad[0] == b[0] + 2 * L.xpad and L.pad[1] == b[1] + 2 * h
    assert L.pad[2] == (b[2] + 2 * h if ndim == 3 else 1)
    assert L.block_stride % 16 == 0 and L.block_stride >= L.pad[0] * L.pad[1] * L.pad[2]
    # first interior point of a block row starts a 32-byte sector when the row pitch allows it
    assert (L.origin - ((h if ndim == 3 else 0) * L.pad[1] + h) * L.pad[0]) == L.xpad
    offs = [L.off_u[0], L.off_u[1]] + ([L.off_f] if has_f else []) + [L.off_send, L.off_scratch]
    assert all(o % 256 == 0 for o in offs) and offs == sorted(offs)
    assert (L.off_f == -1) == (not has_f)
    assert L.off_u[1] - L.off_u[0] >= L.nblocks * L.block_stride * 8
    assert L.total_bytes == jac.workspace_bytes(d) and L.total_bytes > offs[-1]
    for fc in range(6):
        axis = fc // 2
        want = 0 if axis >= ndim else h * int(np.prod([b[a] for a in range(ndim) if a != axis]))
        assert L.face_elems[fc] == want
        assert L.face_offset[fc] % 16 == 0
    assert L.send_stride >= sum(L.face_elems)


@pytest.mark.parametrize("n,b,h", [((12, 8), (3, 2), 2), ((9, 5, 7), (3, 5, 1), 1), ((256, 256), (64, 64), 4),
                                   ((1024, 1024, 1024), (128, 128, 128), 2)])
def test_wide_layout_holds_the_wide_faces(jac, n, b, h):
    ndim = len(n)
    narrow = jac.get_layout(jac.make_desc(n, b, h, False, "exchange"))
    L = jac.get_layout(jac.make_desc(n, b, h, False, "wide"))
    for fc in range(6):
        axis = fc // 2
        want = 0 if axis >= ndim else h * int(np.prod([b[a] + 2 * h for a in range(ndim) if a != axis]))
        assert L.wide_face_elems[fc] == want == narrow.wide_face_elems[fc]
        assert L.face_elems[fc] == narrow.face_elems[fc]       # the plain faces are what they were
        assert L.face_offset[fc] % 16 == 0
        if fc < 2 * ndim - 1:
            assert L.face_offset[fc + 1] - L.face_offset[fc] >= L.wide_face_elems[fc]
    assert L.send_stride >= sum(L.wide_face_elems) and L.send_stride >= narrow.send_stride
    assert L.off_scratch - L.off_send >= L.nblocks * L.send_stride * 8


@pytest.mark.parametrize("n,b,has_f", [((16384, 16384), (1024, 1024), False), ((10, 9, 7), (4, 4, 3), True),
                                        ((14, 11), (4, 4), True)])
def test_host_staging_flag_adds_two_dense_arrays(jac, n, b, has_f):
    plain = jac.get_layout(jac.make_desc(n, b, 1, has_f))
    L = jac.get_layout(jac.make_desc(n, b, 1, has_f, flags=jac.FLAG_HOST_STAGING))
    dense = -(-int(np.prod(n)) * 8 // 256) * 256
    assert plain.off_stage_in == -1 and plain.off_stage_out == -1
    assert L.off_stage_in == plain.total_bytes and L.off_stage_out == L.off_stage_in + dense
    assert L.total_bytes == plain.total_bytes + 2 * dense
    assert L.off_stage_in % 256 == 0 and L.off_stage_out % 256 == 0
    for name in ("off_u", "off_f", "off_send", "off_scratch", "block_stride", "origin"):
        a, c = getattr(plain, name), getattr(L, name)
        assert (list(a) == list(c)) if hasattr(a, "__len__") else (a == c), name
    with pytest.raises(jac.JacError) as e:          # a flag bit the library does not know
        jac.workspace_bytes(jac.make_desc(n, b, 1, has_f, flags=8))
    assert e.value.code == jac.EINVAL


def test_resident_schedule_accepts_what_fits_a_cluster(jac):
    # 256 x 256 with f: slabs of 32 rows in 8 CTAs; 512 x 256 needs 16 CTAs; both are accepted
    for n, b, f in [((256, 256), (256, 256), True), ((512, 256), (128, 64), False), ((12, 4), (4, 4), True)]:
        assert jac.workspace_bytes(jac.make_desc(n, b, 1, f, "resident")) > 0


def test_footprints_of_the_named_configs(jac):
    gib = 1 << 30
    assert jac.workspace_bytes(jac.make_desc((16384, 16384), (1024, 1024))) < 4.5 * gib
    assert jac.workspace_bytes(jac.make_desc((1024,) * 3, (128,) * 3, 1, True)) < 30 * gib


def test_binding_refuses_to_run_without_a_gpu(jac):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        jac.Jacobi((8, 8), (4, 4))


def test_product_code_never_touches_the_oracle():
    """The oracle is test infrastructure: nothing in the package (binding, build, inputs, kernels)
    may import, load or name it, and the oracle may not reach into the package's CUDA side."""
    pkg = ROOT / "paper_2210_01238_b200"
    for path in list(pkg.rglob("*.py")) + list(pkg.rglob("*.cu*")) + list(pkg.rglob("*.h")):
        text = path.read_text()
        assert "oracle" not in text.lower() and "liborc" not in text, path
    for path in (ROOT / "oracle").glob("*"):
        if path.suffix in (".py", ".c"):
            text = path.read_text()
            assert "libjac" not in text and "import jac" not in text and "csrc" not in text, path
