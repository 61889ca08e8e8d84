"""ctypes front end of the CPU oracle (``jacobi_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  Nothing here touches the GPU library, and the
GPU library never touches this.

The arithmetic lives in the C file; this module only marshals numpy arrays and, in
``sample_points``, chooses which sub-window of a huge domain the monolithic sweep is
run on (the sweep itself is still the C routine).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import sys
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "jacobi_oracle.c"
_LIB = _HERE / "liborc.so"

_i64p = C.POINTER(C.c_int64)
_f64p = C.POINTER(C.c_double)


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no FMA contraction, OpenMP over rows/blocks)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        cmd = ["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-fPIC", "-shared", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        # ORC_LIB lets the mutation test point the pins at a deliberately broken build
        override = os.environ.get("ORC_LIB")
        if override:
            L = C.CDLL(override)
        else:
            build()
            L = C.CDLL(str(_LIB))
        L.orc_sweep_mono.argtypes = [C.c_int, _i64p, _f64p, _f64p, _f64p]
        L.orc_residual_mono.argtypes = [C.c_int, _i64p, _f64p, _f64p, _f64p]
        L.orc_blocked_create.argtypes = [C.c_int, _i64p, _i64p, C.c_int64, C.c_int,
                                         C.POINTER(C.c_void_p)]
        L.orc_blocked_destroy.argtypes = [C.c_void_p]
        L.orc_blocked_set_boundary.argtypes = [C.c_void_p, C.c_int, C.c_double]
        L.orc_blocked_set_u.argtypes = [C.c_void_p, _f64p]
        L.orc_blocked_set_f.argtypes = [C.c_void_p, _f64p]
        L.orc_blocked_get_u.argtypes = [C.c_void_p, _f64p]
        L.orc_blocked_get_block_padded.argtypes = [C.c_void_p, C.c_int64, _f64p]
        L.orc_blocked_get_halo_buffer.argtypes = [C.c_void_p, C.c_int64, C.c_int, _f64p]
        L.orc_blocked_pack.argtypes = [C.c_void_p]
        L.orc_blocked_unpack.argtypes = [C.c_void_p]
        L.orc_blocked_update.argtypes = [C.c_void_p]
        L.orc_blocked_sweep.argtypes = [C.c_void_p, C.c_int64]
        L.orc_blocked_residual.argtypes = [C.c_void_p, _f64p]
        L.orc_blocked_exchange_wide.argtypes = [C.c_void_p, _f64p]
        L.orc_blocked_update_ext.argtypes = [C.c_void_p, C.c_int64]
        L.orc_blocked_sweep_wide.argtypes = [C.c_void_p, C.c_int64, C.c_int64]
        L.orc_blocked_wide_face_elems.argtypes = [C.c_void_p, C.c_int64, C.c_int]
        L.orc_blocked_face_elems.argtypes = [C.c_void_p, C.c_int64, C.c_int]
        L.orc_blocked_face_elems.restype = C.c_int64
        L.orc_blocked_wide_face_elems.restype = C.c_int64
        L.orc_blocked_wide_max_face.argtypes = [C.c_void_p]
        L.orc_blocked_wide_max_face.restype = C.c_int64
        L.orc_blocked_cut_elems.argtypes = [C.c_void_p]
        L.orc_blocked_cut_elems.restype = C.c_int64
        L.orc_blocked_pack_cut.argtypes = [C.c_void_p, C.c_int, _f64p]
        L.orc_blocked_unpack_cut.argtypes = [C.c_void_p, C.c_int, _f64p]
        _lib = L
    return _lib


def _ptr(a: np.ndarray | None):
    if a is None:
        return None
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_f64p)


def _dims(v, ndim):
    v = [int(x) for x in v]
    assert len(v) == ndim
    return (C.c_int64 * 3)(*(v + [1] * (3 - ndim)))


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle {what} failed with code {rc}")


def set_threads(n: int) -> None:
    """OpenMP thread count for subsequent oracle calls (timing only; results do not depend on it)."""
    omp = C.CDLL("libgomp.so.1")
    omp.omp_set_num_threads(int(n))


def max_threads() -> int:
    omp = C.CDLL("libgomp.so.1")
    return int(omp.omp_get_max_threads())


# --------------------------------------------------------------------------- #
# Monolithic form.  Arrays are numpy with shape (ny+2, nx+2) or (nz+2, ny+2, nx+2):
# numpy's last axis is x (fastest).
# --------------------------------------------------------------------------- #

def mono_padded(n, bvals=None) -> np.ndarray:
    """Zero padded array with Dirichlet values (face order -x,+x,-y,+y,-z,+z) in the ghost ring."""
    ndim = len(n)
    shape = tuple(int(x) + 2 for x in reversed(n))
    u = np.zeros(shape, dtype=np.float64)
    if bvals is not None:
        for face, val in enumerate(bvals[: 2 * ndim]):
            axis_np = ndim - 1 - face // 2
            idx = [slice(1, -1)] * ndim
            idx[axis_np] = -1 if face & 1 else 0
            u[tuple(idx)] = val
    return u


def mono_sweep(u: np.ndarray, f: np.ndarray | None = None, nsweeps: int = 1) -> np.ndarray:
    """nsweeps Jacobi sweeps of the padded array ``u``; returns a new padded array."""
    ndim = u.ndim
    n = [s - 2 for s in reversed(u.shape)]
    a = np.ascontiguousarray(u, dtype=np.float64).copy()
    b = a.copy()
    if f is not None:
        f = np.ascontiguousarray(f, dtype=np.float64)
        assert f.size == int(np.prod(n))
    for _ in range(int(nsweeps)):
        _check(lib().orc_sweep_mono(ndim, _dims(n, ndim), _ptr(a), _ptr(f), _ptr(b)), "sweep_mono")
        a, b = b, a
    return a


def mono_residual(u: np.ndarray, f: np.ndarray | None = None) -> float:
    ndim = u.ndim
    n = [s - 2 for s in reversed(u.shape)]
    u = np.ascontiguousarray(u, dtype=np.float64)
    if f is not None:
        f = np.ascontiguousarray(f, dtype=np.float64)
    out = C.c_double(0.0)
    _check(lib().orc_residual_mono(ndim, _dims(n, ndim), _ptr(u), _ptr(f), C.byref(out)),
           "residual_mono")
    return out.value


# --------------------------------------------------------------------------- #
# Blocked form.
# --------------------------------------------------------------------------- #

class Blocked:
    """Block-decomposed state: per-block padded arrays, send buffers, optional f.

    n, b: global and block interior sizes in (x, y[, z]) order; h: ghost width.
    Dense arrays passed in/out have numpy shape (ny, nx) or (nz, ny, nx).
    """

    def __init__(self, n, b, h: int = 1, has_f: bool = False):
        self.ndim = len(n)
        self.n = [int(x) for x in n]
        self.b = [int(x) for x in b]
        self.h = int(h)
        self.has_f = bool(has_f)
        self._p = C.c_void_p()
        _check(lib().orc_blocked_create(self.ndim, _dims(n, self.ndim), _dims(b, self.ndim),
                                        self.h, int(has_f), C.byref(self._p)), "create")
        self.g = [-(-nn // bb) for nn, bb in zip(self.n, self.b)]
        self.nblocks = int(np.prod(self.g))

    def close(self):
        if self._p:
            lib().orc_blocked_destroy(self._p)
            self._p = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _dense_shape(self):
        return tuple(reversed(self.n))

    def padded_shape(self):
        return tuple(x + 2 * self.h for x in reversed(self.b))

    def coords(self, blk: int):
        g = self.g + [1] * (3 - self.ndim)
        return [blk % g[0], (blk // g[0]) % g[1], blk // (g[0] * g[1])][: self.ndim]

    def extent(self, blk: int):
        """Interior points of block ``blk`` per axis: b, or the remainder for the last block of an axis."""
        return [min(bb, nn - c * bb) for nn, bb, c in zip(self.n, self.b, self.coords(blk))]

    def face_shape(self, face: int, blk: int = 0):
        """numpy shape of a packed face: (ez, ey, h) for x, (ez, h, ex) for y, (h, ey, ex) for z (2D drops z),
        e = the block's interior extent."""
        dims = self.extent(blk)
        dims[face // 2] = self.h
        return tuple(reversed(dims))

    def set_boundary(self, face: int, value: float):
        _check(lib().orc_blocked_set_boundary(self._p, face, float(value)), "set_boundary")

    def set_u(self, dense: np.ndarray):
        d = np.ascontiguousarray(dense, dtype=np.float64)
        assert d.shape == self._dense_shape()
        _check(lib().orc_blocked_set_u(self._p, _ptr(d)), "set_u")

    def set_f(self, dense: np.ndarray):
        d = np.ascontiguousarray(dense, dtype=np.float64)
        assert d.shape == self._dense_shape()
        _check(lib().orc_blocked_set_f(self._p, _ptr(d)), "set_f")

    def get_u(self) -> np.ndarray:
        out = np.empty(self._dense_shape(), dtype=np.float64)
        _check(lib().orc_blocked_get_u(self._p, _ptr(out)), "get_u")
        return out

    def get_block_padded(self, blk: int) -> np.ndarray:
        out = np.empty(self.padded_shape(), dtype=np.float64)
        _check(lib().orc_blocked_get_block_padded(self._p, blk, _ptr(out)), "get_block_padded")
        return out

    def get_halo_buffer(self, blk: int, face: int) -> np.ndarray:
        out = np.empty(self.face_shape(face, blk), dtype=np.float64)
        assert out.size == int(lib().orc_blocked_face_elems(self._p, blk, face))
        _check(lib().orc_blocked_get_halo_buffer(self._p, blk, face, _ptr(out)), "get_halo_buffer")
        return out

    def pack(self):
        _check(lib().orc_blocked_pack(self._p), "pack")

    def unpack(self):
        _check(lib().orc_blocked_unpack(self._p), "unpack")

    def update(self):
        _check(lib().orc_blocked_update(self._p), "update")

    def sweep(self, nsweeps: int = 1):
        _check(lib().orc_blocked_sweep(self._p, int(nsweeps)), "sweep")

    def residual(self) -> float:
        out = C.c_double(0.0)
        _check(lib().orc_blocked_residual(self._p, C.byref(out)), "residual")
        return out.value

    # ---- wide exchange: all h ghost layers including edges and corners, axis by axis
    def wide_face_shape(self, face: int, blk: int = 0):
        """numpy shape of a packed wide face: h layers along the face's axis, extent + 2h along the others."""
        dims = [x + 2 * self.h for x in self.extent(blk)]
        dims[face // 2] = self.h
        return tuple(reversed(dims))

    def exchange_wide(self, keep_buffers: bool = False):
        """Wide exchange of the current state; with ``keep_buffers`` returns {(blk, face): packed wide face}."""
        if not keep_buffers:
            _check(lib().orc_blocked_exchange_wide(self._p, None), "exchange_wide")
            return None
        wmax = int(lib().orc_blocked_wide_max_face(self._p))
        raw = np.zeros((self.nblocks, 6, wmax), dtype=np.float64)
        _check(lib().orc_blocked_exchange_wide(self._p, _ptr(raw)), "exchange_wide")
        out = {}
        for blk in range(self.nblocks):
            for face in range(2 * self.ndim):
                if self.neighbour(blk, face) < 0:
                    continue
                shp = self.wide_face_shape(face, blk)
                ne = int(lib().orc_blocked_wide_face_elems(self._p, blk, face))
                assert ne == int(np.prod(shp))
                out[(blk, face)] = raw[blk, face, :ne].reshape(shp).copy()
        return out

    def update_ext(self, e: int):
        """The update over every block's interior extended by e layers (no exchange)."""
        _check(lib().orc_blocked_update_ext(self._p, int(e)), "update_ext")

    def sweep_wide(self, nsweeps: int, k: int | None = None):
        """nsweeps sweeps with one wide exchange per group of k (default h) sweeps."""
        _check(lib().orc_blocked_sweep_wide(self._p, int(nsweeps), int(self.h if k is None else k)), "sweep_wide")

    # ---- slabs: the faces that cross a cut along the slowest axis
    def cut_elems(self) -> int:
        return int(lib().orc_blocked_cut_elems(self._p))

    def pack_cut(self, side: int) -> np.ndarray:
        """The h interior layers next to the low (0) / high (1) end of the slowest axis, packed."""
        out = np.zeros(self.cut_elems(), dtype=np.float64)
        _check(lib().orc_blocked_pack_cut(self._p, int(side), _ptr(out)), "pack_cut")
        return out

    def unpack_cut(self, side: int, plane: np.ndarray):
        """A plane packed by the neighbouring slab -> the ghost layers at that end."""
        plane = np.ascontiguousarray(plane, dtype=np.float64)
        assert plane.size == self.cut_elems()
        _check(lib().orc_blocked_unpack_cut(self._p, int(side), _ptr(plane)), "unpack_cut")

    def neighbour(self, blk: int, face: int) -> int:
        """Block across ``face`` or -1 at the domain boundary (host-side convenience for tests)."""
        c = [blk % self.g[0], (blk // self.g[0]) % self.g[1] if self.ndim > 1 else 0,
             blk // (self.g[0] * self.g[1]) if self.ndim > 2 else 0]
        a = face // 2
        c[a] += 1 if face & 1 else -1
        if c[a] < 0 or c[a] >= self.g[a]:
            return -1
        g = self.g + [1] * (3 - self.ndim)
        return (c[2] * g[1] + c[1]) * g[0] + c[0]


# --------------------------------------------------------------------------- #
# Sampled outputs of a domain too large to sweep on the CPU.
#
# After k sweeps the value at a point depends only on initial data within
# Manhattan distance k.  So the monolithic sweep run on the sub-box of radius k
# around the point (clipped at the domain, where the true Dirichlet ghosts take
# over) gives, at the centre, bit for bit what the full-domain run gives there:
# wrong values injected at the artificial box edge move inwards by one cell per
# sweep and have not reached the centre after k sweeps.
# --------------------------------------------------------------------------- #

def sample_points(n, nsweeps: int, points, u0_fn, f_fn=None, bvals=None) -> np.ndarray:
    """Values after ``nsweeps`` sweeps at the given 0-based interior ``points`` [(i, j[, k]), ...].

    u0_fn(lo, hi) / f_fn(lo, hi) return the dense initial data / right-hand side on the
    0-based half-open interior index box [lo, hi) (x, y[, z] order), numpy shape reversed.
    """
    ndim = len(n)
    bvals = list(bvals) if bvals is not None else [0.0] * (2 * ndim)
    out = np.empty(len(points), dtype=np.float64)
    for q, pt in enumerate(points):
        lo = [max(0, int(pt[a]) - nsweeps) for a in range(ndim)]
        hi = [min(int(n[a]), int(pt[a]) + nsweeps + 1) for a in range(ndim)]
        size = [hi[a] - lo[a] for a in range(ndim)]
        u = np.zeros(tuple(s + 2 for s in reversed(size)), dtype=np.float64)
        for face in range(2 * ndim):
            a = face // 2
            on_boundary = (hi[a] == n[a]) if face & 1 else (lo[a] == 0)
            if on_boundary:
                idx = [slice(1, -1)] * ndim
                idx[ndim - 1 - a] = -1 if face & 1 else 0
                u[tuple(idx)] = bvals[face]
        u[(slice(1, -1),) * ndim] = u0_fn(lo, hi)
        f = None if f_fn is None else np.ascontiguousarray(f_fn(lo, hi), dtype=np.float64)
        u = mono_sweep(u, f, nsweeps)
        centre = tuple(int(pt[a]) - lo[a] + 1 for a in reversed(range(ndim)))
        out[q] = u[centre]
    return out


if __name__ == "__main__":
    build(force="--force" in sys.argv)
    print(_LIB)
