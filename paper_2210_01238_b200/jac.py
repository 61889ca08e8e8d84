"""ctypes binding of ``libjac.so`` -- argument marshalling only.

Every step of the hot path (sweep, pack, unpack, residual) runs in the library's CUDA
kernels; PyTorch is used here for nothing but device memory and the stream.  There is no
CPU fallback: if the shared library is missing, or a call is made without a CUDA device,
an exception is raised.

    from paper_2210_01238_b200 import jac
    J = jac.Jacobi(n=(4096, 4096), b=(512, 512), halo=1, has_f=True)
    J.set_f(f); J.sweep(10); r = J.residual(); u = J.get_u()
"""
from __future__ import annotations

import ctypes as C
import os
from pathlib import Path

import numpy as np

_PKG = Path(__file__).resolve().parent
# JAC_LIB selects another build of the same library (e.g. one compiled with different tile sizes)
LIB_PATH = Path(os.environ["JAC_LIB"]) if os.environ.get("JAC_LIB") else _PKG / "libjac.so"

MODE_FUSED, MODE_PERTASK, MODE_TEMPORAL, MODE_EXCHANGE, MODE_WIDE, MODE_RESIDENT = 0, 1, 2, 3, 4, 5
MODES = {"fused": MODE_FUSED, "pertask": MODE_PERTASK, "temporal": MODE_TEMPORAL,
         "exchange": MODE_EXCHANGE, "wide": MODE_WIDE, "resident": MODE_RESIDENT}

OK, EINVAL, ENOMEM, ECUDA, ENODEV, ELIMIT, ETIMEOUT = 0, -1, -2, -3, -4, -5, -6
FLAG_HOST_STAGING, FLAG_CUT_LO, FLAG_CUT_HI = 1, 2, 4

EXPORTS = [
    "jac_workspace_bytes", "jac_get_layout", "jac_create", "jac_destroy",
    "jac_set_u", "jac_set_f", "jac_get_u", "jac_set_u_device", "jac_set_f_device",
    "jac_get_u_device", "jac_set_boundary", "jac_get_block_padded", "jac_get_halo_buffer",
    "jac_pack_halos", "jac_unpack_halos", "jac_pack_faces", "jac_unpack_faces", "jac_sweep", "jac_residual", "jac_launch_count",
    "jac_last_cuda_error", "jac_strerror", "jac_residual_dense_static", "jac_sweeps_per_launch",
    "jac_sweep_residual", "jac_solve", "jac_exchange_wide", "jac_get_wide_buffer",
    "jac_set_u_async", "jac_get_u_async", "jac_residual_async", "jac_exchange_halos",
    "jac_pack_cut", "jac_unpack_cut", "jac_sweep_begin", "jac_sweep_end", "jac_cut_info",
    "jac_residual_sumsq_async", "jac_residual_sweep_async", "jac_debug_bounds", "jac_debug_shrink_bounds",
    "jac_sweep_norms_async",
]


class Desc(C.Structure):
    _fields_ = [("ndim", C.c_int32), ("halo", C.c_int32), ("has_f", C.c_int32),
                ("mode", C.c_int32), ("tsteps", C.c_int32), ("flags", C.c_int32),
                ("n", C.c_int64 * 3), ("b", C.c_int64 * 3), ("stream", C.c_void_p)]


class Layout(C.Structure):
    _fields_ = [("g", C.c_int64 * 3), ("nblocks", C.c_int64), ("pad", C.c_int64 * 3),
                ("xpad", C.c_int64), ("origin", C.c_int64), ("block_stride", C.c_int64),
                ("face_elems", C.c_int64 * 6), ("face_offset", C.c_int64 * 6),
                ("send_stride", C.c_int64), ("partials", C.c_int64), ("off_u", C.c_int64 * 2),
                ("off_f", C.c_int64), ("off_send", C.c_int64), ("off_scratch", C.c_int64),
                ("total_bytes", C.c_int64), ("wide_face_elems", C.c_int64 * 6),
                ("off_stage_in", C.c_int64), ("off_stage_out", C.c_int64), ("cut_elems", C.c_int64),
                ("off_cut_send", (C.c_int64 * 2) * 2), ("off_cut_recv", C.c_int64 * 2)]


class JacError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} ({code})")


_lib = None


def lib() -> C.CDLL:
    """The loaded shared library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2210_01238_b200.build`")
        L = C.CDLL(str(LIB_PATH))
        dp, vp = C.POINTER(C.c_double), C.c_void_p
        L.jac_workspace_bytes.argtypes = [C.POINTER(Desc), C.POINTER(C.c_size_t)]
        L.jac_get_layout.argtypes = [C.POINTER(Desc), C.POINTER(Layout)]
        L.jac_create.argtypes = [C.POINTER(Desc), vp, C.c_size_t, C.POINTER(vp)]
        L.jac_destroy.argtypes = [vp]
        for name in ("jac_set_u", "jac_set_f", "jac_get_u", "jac_set_u_device",
                     "jac_set_f_device", "jac_get_u_device", "jac_set_u_async", "jac_get_u_async",
                     "jac_residual_async", "jac_residual_sumsq_async"):
            getattr(L, name).argtypes = [vp, vp]
        L.jac_pack_cut.argtypes = [vp]
        L.jac_sweep_begin.argtypes = [vp]
        L.jac_unpack_cut.argtypes = [vp, vp, vp, vp, vp]
        L.jac_sweep_end.argtypes = [vp, vp, vp, vp, vp]
        L.jac_cut_info.argtypes = [vp, C.c_int, C.POINTER(vp), C.POINTER(vp), C.POINTER(C.c_size_t), C.POINTER(vp)]
        L.jac_set_boundary.argtypes = [vp, C.c_int, C.c_double]
        L.jac_get_block_padded.argtypes = [vp, C.c_int64, vp]
        L.jac_get_halo_buffer.argtypes = [vp, C.c_int64, C.c_int, vp]
        L.jac_exchange_wide.argtypes = [vp]
        L.jac_get_wide_buffer.argtypes = [vp, C.c_int64, C.c_int, vp]
        L.jac_exchange_halos.argtypes = [vp]
        L.jac_pack_halos.argtypes = [vp]
        L.jac_unpack_halos.argtypes = [vp]
        L.jac_pack_faces.argtypes = [vp, C.c_uint]
        L.jac_unpack_faces.argtypes = [vp, C.c_uint]
        L.jac_sweep.argtypes = [vp, C.c_int]
        L.jac_residual.argtypes = [vp, dp]
        L.jac_sweep_residual.argtypes = [vp, C.c_int, dp]
        L.jac_residual_sweep_async.argtypes = [vp, C.c_int, vp]
        L.jac_sweep_norms_async.argtypes = [vp, C.c_int, C.c_int, vp]
        L.jac_solve.argtypes = [vp, C.c_int, C.c_int, C.c_double, C.POINTER(C.c_int), dp]
        L.jac_launch_count.argtypes = [vp, C.POINTER(C.c_int64)]
        L.jac_sweeps_per_launch.argtypes = [vp, C.POINTER(C.c_int)]
        L.jac_last_cuda_error.argtypes = [vp]
        L.jac_debug_bounds.argtypes = [vp, C.POINTER(C.c_int), C.POINTER(C.c_uint64)]
        L.jac_debug_shrink_bounds.argtypes = [vp, C.c_int, C.c_int64]
        L.jac_strerror.argtypes = [C.c_int]
        L.jac_residual_dense_static.argtypes = [C.c_int, C.POINTER(C.c_int64), vp, vp,
                                                C.POINTER(C.c_double), vp, dp]
        L.jac_strerror.restype = C.c_char_p
        for name in EXPORTS:
            if name != "jac_strerror":
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().jac_strerror(int(code)).decode()


def make_desc(n, b, halo=1, has_f=False, mode=MODE_FUSED, tsteps=0, stream=0, flags=0) -> Desc:
    ndim = len(n)
    d = Desc()
    d.ndim, d.halo, d.has_f = ndim, int(halo), int(bool(has_f))
    d.mode = MODES[mode] if isinstance(mode, str) else int(mode)
    d.tsteps, d.flags = int(tsteps), int(flags)
    for a in range(3):
        d.n[a] = int(n[a]) if a < ndim else 1
        d.b[a] = int(b[a]) if a < ndim else 1
    d.stream = stream or None
    return d


def workspace_bytes(desc: Desc) -> int:
    out = C.c_size_t(0)
    rc = lib().jac_workspace_bytes(C.byref(desc), C.byref(out))
    if rc:
        raise JacError(rc, "jac_workspace_bytes")
    return out.value


def get_layout(desc: Desc) -> Layout:
    out = Layout()
    rc = lib().jac_get_layout(C.byref(desc), C.byref(out))
    if rc:
        raise JacError(rc, "jac_get_layout")
    return out


def residual_dense_static(u, f=None, bvals=None, stream=None) -> float:
    """Residual norm of dense CUDA tensors ``u`` (and ``f``) of shape (ny, nx) / (nz, ny, nx)
    through the entry point that allocates nothing (no context, no workspace).

    For callers that may not allocate device memory; see ``jac_residual_dense_static`` in
    ``include/jac.h`` for the size limit (2^29 points) and the rule that calls on one device
    must not overlap.  The first call on a device should be made outside stream capture.
    """
    import torch
    assert u.is_cuda and u.dtype == torch.float64 and u.is_contiguous() and u.dim() in (2, 3)
    if f is not None:
        assert f.is_cuda and f.dtype == torch.float64 and f.is_contiguous() and f.shape == u.shape
    ndim = u.dim()
    n = (C.c_int64 * 3)(*(list(reversed(u.shape)) + [1] * (3 - ndim)))
    bv = None
    if bvals is not None:
        assert len(bvals) == 2 * ndim
        bv = (C.c_double * 6)(*([float(x) for x in bvals] + [0.0] * (6 - 2 * ndim)))
    st = stream if stream is not None else torch.cuda.current_stream()
    out = C.c_double(0.0)
    rc = lib().jac_residual_dense_static(ndim, n, u.data_ptr(), f.data_ptr() if f is not None else None,
                                         bv, st.cuda_stream or None, C.byref(out))
    if rc:
        raise JacError(rc, "jac_residual_dense_static")
    return out.value


def _host_ptr(a: np.ndarray):
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


class Jacobi:
    """One context of the library over a torch-owned workspace on the current CUDA device.

    n, b: global / block interior points in (x, y[, z]) order.  ``workspace``: a uint8 CUDA tensor to
    use instead of allocating one (256-byte aligned, ``workspace_bytes`` long).  Dense arrays are numpy float64
    of shape (ny, nx) / (nz, ny, nx), or torch CUDA float64 tensors of that shape for the
    ``*_device`` calls.
    """

    def __init__(self, n, b, halo=1, has_f=False, mode="fused", tsteps=0, stream=None, flags=0, workspace=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2210_01238_b200.jac needs a CUDA device; there is no CPU path")
        self._torch = torch
        self.n, self.b = tuple(int(x) for x in n), tuple(int(x) for x in b)
        self.ndim = len(self.n)
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        self.desc = make_desc(n, b, halo, has_f, mode, tsteps, self.stream.cuda_stream, flags)
        self.layout = get_layout(self.desc)
        nbytes = workspace_bytes(self.desc)
        if workspace is not None:
            # the caller's memory: a contiguous uint8 CUDA tensor of at least the size the library asks for
            assert workspace.is_cuda and workspace.dtype == torch.uint8 and workspace.is_contiguous()
            assert workspace.numel() >= nbytes and workspace.data_ptr() % 256 == 0
            self.workspace = workspace
        else:
            with torch.cuda.stream(self.stream):
                self.workspace = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        self._ctx = C.c_void_p()
        self._call("jac_create", lib().jac_create(C.byref(self.desc), self.workspace.data_ptr(),
                                                  nbytes, C.byref(self._ctx)))

    # ---- plumbing
    def _call(self, what: str, rc: int):
        if rc:
            detail = ""
            if rc == ECUDA and self._ctx:
                detail = f" [cudaError {lib().jac_last_cuda_error(self._ctx)}]"
            raise JacError(rc, what + detail)

    def bounds_record(self):
        """(does this build of the library check its kernels' addresses, record of the first access
        outside its array or 0) -- see ``jac_debug_bounds``."""
        checked, rec = C.c_int(0), C.c_uint64(0)
        self._call("jac_debug_bounds", lib().jac_debug_bounds(self._ctx, C.byref(checked), C.byref(rec)))
        return bool(checked.value), int(rec.value)

    def close(self):
        if getattr(self, "_ctx", None):
            # a checked build (JAC_LIB pointing at one) speaks up when a context is closed
            checked, rec = C.c_int(0), C.c_uint64(0)
            rc = lib().jac_debug_bounds(self._ctx, C.byref(checked), C.byref(rec))
            lib().jac_destroy(self._ctx)
            self._ctx = C.c_void_p()
            self.workspace = None
            if rc == OK and checked.value and rec.value:
                raise JacError(EINVAL, f"a kernel reached outside its array: kernel {rec.value >> 56}, array "
                                       f"{(rec.value >> 52) & 15}, byte offset {rec.value & ((1 << 52) - 1):#x}")

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    @property
    def dense_shape(self):
        return tuple(reversed(self.n))

    @property
    def nblocks(self) -> int:
        return int(self.layout.nblocks)

    def _dev_ptr(self, t):
        assert t.is_cuda and t.dtype == self._torch.float64 and t.is_contiguous()
        assert tuple(t.shape) == self.dense_shape
        return t.data_ptr()

    # ---- data in / out
    def set_u(self, dense: np.ndarray):
        d = np.ascontiguousarray(dense, dtype=np.float64)
        assert d.shape == self.dense_shape
        self._call("jac_set_u", lib().jac_set_u(self._ctx, _host_ptr(d)))

    def set_f(self, dense: np.ndarray):
        d = np.ascontiguousarray(dense, dtype=np.float64)
        assert d.shape == self.dense_shape
        self._call("jac_set_f", lib().jac_set_f(self._ctx, _host_ptr(d)))

    def get_u(self, out: np.ndarray | None = None) -> np.ndarray:
        if out is None:
            out = np.empty(self.dense_shape, dtype=np.float64)
        assert out.shape == self.dense_shape
        self._call("jac_get_u", lib().jac_get_u(self._ctx, _host_ptr(out)))
        return out

    def set_u_device(self, t):
        self._call("jac_set_u_device", lib().jac_set_u_device(self._ctx, self._dev_ptr(t)))

    def set_f_device(self, t):
        self._call("jac_set_f_device", lib().jac_set_f_device(self._ctx, self._dev_ptr(t)))

    def get_u_device(self, out=None):
        if out is None:
            with self._torch.cuda.stream(self.stream):
                out = self._torch.empty(self.dense_shape, dtype=self._torch.float64, device="cuda")
        self._call("jac_get_u_device", lib().jac_get_u_device(self._ctx, self._dev_ptr(out)))
        return out

    def set_u_pinned(self, t):
        """``t``: pinned host torch tensor of the dense shape (asynchronous DMA source)."""
        assert not t.is_cuda and t.dtype == self._torch.float64 and t.is_contiguous()
        self._call("jac_set_u", lib().jac_set_u(self._ctx, t.data_ptr()))

    def get_u_pinned(self, t):
        assert not t.is_cuda and t.dtype == self._torch.float64 and t.is_contiguous()
        self._call("jac_get_u", lib().jac_get_u(self._ctx, t.data_ptr()))
        return t

    # ---- the same without waiting (pinned host tensors; synchronise the stream before reuse)
    def _pinned_ptr(self, t, shape=None):
        assert not t.is_cuda and t.is_pinned() and t.dtype == self._torch.float64 and t.is_contiguous()
        assert shape is None or tuple(t.shape) == shape
        return t.data_ptr()

    def set_u_async(self, t):
        self._call("jac_set_u_async", lib().jac_set_u_async(self._ctx, self._pinned_ptr(t, self.dense_shape)))

    def get_u_async(self, t):
        self._call("jac_get_u_async", lib().jac_get_u_async(self._ctx, self._pinned_ptr(t, self.dense_shape)))
        return t

    def residual_async(self, out):
        """``out``: pinned float64 tensor with one element; holds the norm once the stream got there."""
        assert out.numel() == 1
        self._call("jac_residual_async", lib().jac_residual_async(self._ctx, self._pinned_ptr(out)))
        return out

    def residual_sumsq_async(self, out):
        """As residual_async, but the sum of squares (slabs of one domain add theirs, then take the root)."""
        assert out.numel() == 1
        self._call("jac_residual_sumsq_async", lib().jac_residual_sumsq_async(self._ctx, self._pinned_ptr(out)))
        return out

    def residual_sumsq(self) -> float:
        """Sum of squares of the residual of the current state (waits for the stream)."""
        out = self._torch.zeros(1, dtype=self._torch.float64).pin_memory()
        self.residual_sumsq_async(out)
        self.stream.synchronize()
        return float(out[0])

    # ---- slab contexts (flags FLAG_CUT_LO / FLAG_CUT_HI)
    def cut_info(self, side: int):
        """(send pointer of the last pack, receive pointer, bytes, ready event) of cut ``side``."""
        send, recv, ev, nbytes = C.c_void_p(), C.c_void_p(), C.c_void_p(), C.c_size_t(0)
        self._call("jac_cut_info", lib().jac_cut_info(self._ctx, int(side), C.byref(send), C.byref(recv),
                                                      C.byref(nbytes), C.byref(ev)))
        return send.value, recv.value, nbytes.value, ev.value

    def _cut_view(self, ptr: int, nbytes: int):
        """The workspace bytes [ptr, ptr + nbytes) as a float64 tensor (no copy)."""
        off = ptr - self.workspace.data_ptr()
        return self.workspace[off:off + nbytes].view(self._torch.float64)

    def cut_send(self, side: int):
        send, _, nbytes, _ = self.cut_info(side)
        return self._cut_view(send, nbytes)

    def cut_recv(self, side: int):
        _, recv, nbytes, _ = self.cut_info(side)
        return self._cut_view(recv, nbytes)

    def pack_cut(self):
        self._call("jac_pack_cut", lib().jac_pack_cut(self._ctx))

    def unpack_cut(self, src_lo=None, ready_lo=None, src_hi=None, ready_hi=None):
        self._call("jac_unpack_cut", lib().jac_unpack_cut(self._ctx, src_lo, ready_lo, src_hi, ready_hi))

    def sweep_begin(self):
        self._call("jac_sweep_begin", lib().jac_sweep_begin(self._ctx))

    def sweep_end(self, src_lo=None, ready_lo=None, src_hi=None, ready_hi=None):
        self._call("jac_sweep_end", lib().jac_sweep_end(self._ctx, src_lo, ready_lo, src_hi, ready_hi))

    def set_boundary(self, face: int, value: float):
        self._call("jac_set_boundary", lib().jac_set_boundary(self._ctx, int(face), float(value)))

    def get_block_padded(self, blk: int) -> np.ndarray:
        h = self.desc.halo
        out = np.empty(tuple(x + 2 * h for x in reversed(self.b)), dtype=np.float64)
        self._call("jac_get_block_padded",
                   lib().jac_get_block_padded(self._ctx, int(blk), _host_ptr(out)))
        return out

    def extent(self, blk: int):
        """Interior points of block ``blk`` per axis: b, or the remainder for the last block of an axis."""
        g = [int(self.layout.g[a]) for a in range(3)]
        c = [blk % g[0], (blk // g[0]) % g[1], blk // (g[0] * g[1])][: self.ndim]
        return [min(bb, nn - cc * bb) for nn, bb, cc in zip(self.n, self.b, c)]

    def get_halo_buffer(self, blk: int, face: int) -> np.ndarray:
        """Packed face of (block, face); a remainder block's face is correspondingly smaller."""
        raw = np.empty(int(self.layout.face_elems[face]), dtype=np.float64)
        self._call("jac_get_halo_buffer",
                   lib().jac_get_halo_buffer(self._ctx, int(blk), int(face), _host_ptr(raw)))
        dims = self.extent(blk)
        dims[face // 2] = self.desc.halo
        return raw[: int(np.prod(dims))].reshape(tuple(reversed(dims))).copy()

    # ---- the hot path
    def pack_halos(self):
        self._call("jac_pack_halos", lib().jac_pack_halos(self._ctx))

    def unpack_halos(self):
        self._call("jac_unpack_halos", lib().jac_unpack_halos(self._ctx))

    def exchange_halos(self):
        """pack_halos + unpack_halos as one launch."""
        self._call("jac_exchange_halos", lib().jac_exchange_halos(self._ctx))

    def pack_faces(self, face_mask: int):
        self._call("jac_pack_faces", lib().jac_pack_faces(self._ctx, int(face_mask)))

    def unpack_faces(self, face_mask: int):
        self._call("jac_unpack_faces", lib().jac_unpack_faces(self._ctx, int(face_mask)))

    def exchange_wide(self):
        """All h ghost layers, edges and corners included (contexts created with mode "wide")."""
        self._call("jac_exchange_wide", lib().jac_exchange_wide(self._ctx))

    def get_wide_buffer(self, blk: int, face: int) -> np.ndarray:
        h = self.desc.halo
        raw = np.empty(int(self.layout.wide_face_elems[face]), dtype=np.float64)
        self._call("jac_get_wide_buffer",
                   lib().jac_get_wide_buffer(self._ctx, int(blk), int(face), _host_ptr(raw)))
        dims = [x + 2 * h for x in self.extent(blk)]
        dims[face // 2] = h
        return raw[: int(np.prod(dims))].reshape(tuple(reversed(dims))).copy()

    def sweep(self, nsweeps: int = 1):
        self._call("jac_sweep", lib().jac_sweep(self._ctx, int(nsweeps)))

    def sweep_residual(self, nsweeps: int) -> float:
        """nsweeps sweeps; returns the residual norm of the state before the last of them."""
        out = C.c_double(0.0)
        self._call("jac_sweep_residual", lib().jac_sweep_residual(self._ctx, int(nsweeps), C.byref(out)))
        return out.value

    def residual_sweep_async(self, nsweeps: int, out):
        """The residual norm of the current state (into the pinned 1-element tensor ``out`` when the
        stream gets there), then nsweeps sweeps; the norm comes out of the first sweep's pass."""
        assert out.numel() == 1
        self._call("jac_residual_sweep_async",
                   lib().jac_residual_sweep_async(self._ctx, int(nsweeps), self._pinned_ptr(out)))
        return out

    def sweep_norms_async(self, nsweeps: int, every: int, out=None):
        """nsweeps sweeps; the pinned tensor ``out`` receives, when the stream gets there, the residual
        norms of the states after every, 2 * every, ... (< nsweeps) sweeps: (nsweeps - 1) // every values."""
        need = (int(nsweeps) - 1) // int(every) if nsweeps >= 1 and every >= 1 else 0
        if need > 0:
            assert out is not None and out.numel() >= need
        ptr = self._pinned_ptr(out) if out is not None else None
        self._call("jac_sweep_norms_async",
                   lib().jac_sweep_norms_async(self._ctx, int(nsweeps), int(every), ptr))
        return out

    def solve(self, max_sweeps: int, check_every: int, tol: float):
        """Sweeps until the lagged residual norm is <= tol; returns (sweeps done, last norm)."""
        done, res = C.c_int(0), C.c_double(0.0)
        self._call("jac_solve", lib().jac_solve(self._ctx, int(max_sweeps), int(check_every), float(tol),
                                                C.byref(done), C.byref(res)))
        return done.value, res.value

    def residual(self) -> float:
        out = C.c_double(0.0)
        self._call("jac_residual", lib().jac_residual(self._ctx, C.byref(out)))
        return out.value

    def sweeps_per_launch(self) -> int:
        out = C.c_int(0)
        self._call("jac_sweeps_per_launch", lib().jac_sweeps_per_launch(self._ctx, C.byref(out)))
        return out.value

    def launch_count(self) -> int:
        out = C.c_int64(0)
        self._call("jac_launch_count", lib().jac_launch_count(self._ctx, C.byref(out)))
        return out.value
