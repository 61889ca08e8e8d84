"""One domain over several GPUs: slabs of whole block planes along the slowest axis.

The paper's proxy application (Section V-C) spreads its blocks over many GPUs; per iteration the
faces of neighbouring blocks travel as messages, and the paper credits its gains to overlapping
those messages with kernel work.  Here every GPU owns one *slab* -- a contiguous run of block
planes along the slowest axis (y in 2D, z in 3D) -- as a library context of its own
(``FLAG_CUT_LO`` / ``FLAG_CUT_HI``).  Between slabs only the faces on the cut planes travel, once
per sweep; the residual norm needs one 8-byte sum.

This module is plumbing only: it decides who owns which planes and moves packed cut planes between
neighbours.  Packing, unpacking, the update and its overlap with the transfer
(``jac_sweep_begin`` / ``jac_sweep_end``) run in the library.

Two ways to move a plane:

* ``SlabRank`` -- one process per GPU under ``torch.distributed``: the packed plane goes to the
  neighbour rank with a point-to-point send/recv (NCCL between GPUs) straight between the
  contexts' cut buffers, and the residual is one ``all_reduce`` of a double.
* ``LocalSlabs`` -- several slabs in one process: a slab's unpack kernel reads the neighbour's send
  buffer in place (ordinary loads; on another device this needs peer access), ordered by the event
  the neighbour records after packing.  No copy at all.

An *engine* is what a slab runs on: ``jac.Jacobi`` with cut flags, or any object with the same
``pack_cut / cut_send / cut_recv / unpack_cut / sweep_begin / sweep_end`` methods.
"""
from __future__ import annotations

import math

FLAG_CUT_LO, FLAG_CUT_HI = 2, 4


def slab_planes(planes: int, parts: int):
    """[(first plane, one past the last plane)] for each part: contiguous, sizes differing by at
    most one, larger ones first.  Every part gets at least one plane."""
    if parts < 1 or planes < parts:
        raise ValueError(f"{planes} block planes cannot be cut into {parts} slabs")
    base, extra = divmod(planes, parts)
    out, lo = [], 0
    for p in range(parts):
        hi = lo + base + (1 if p < extra else 0)
        out.append((lo, hi))
        lo = hi
    return out


def slab_of(n, b, part: int, parts: int):
    """The slab of part ``part``: (its extent n_slab, its block size, its cut flags, its first point
    along the slowest axis).  The block size is ``b``, except that a last slab that is a single
    remainder plane has blocks as thin as that plane."""
    n, b = [int(x) for x in n], [int(x) for x in b]
    sa = len(n) - 1
    planes = -(-n[sa] // b[sa])
    lo, hi = slab_planes(planes, parts)[part]
    first = lo * b[sa]
    last = min(n[sa], hi * b[sa])
    n_slab = list(n)
    n_slab[sa] = last - first
    b_slab = list(b)
    b_slab[sa] = min(b[sa], n_slab[sa])
    flags = (FLAG_CUT_LO if part > 0 else 0) | (FLAG_CUT_HI if part + 1 < parts else 0)
    return tuple(n_slab), tuple(b_slab), flags, first


def slab_slice(n, b, part: int, parts: int):
    """Index of the slab inside a dense array of shape (ny, nx) / (nz, ny, nx)."""
    n_slab, _, _, first = slab_of(n, b, part, parts)
    return (slice(first, first + n_slab[len(n) - 1]),)


class SlabRank:
    """One rank's slab under ``torch.distributed`` (one process per GPU).

    ``engine``: the slab's context; ``dist``: the ``torch.distributed`` module (or a stand-in with
    ``P2POp``, ``isend``, ``irecv``, ``batch_isend_irecv``, ``all_reduce``); ``sumsq``: a callable
    returning the slab's sum of squared residuals of the current state as a 1-element tensor on the
    device the group communicates on.
    """

    def __init__(self, engine, rank: int, world: int, dist, sumsq, group=None):
        self.engine, self.rank, self.world, self.dist, self.group = engine, int(rank), int(world), dist, group
        self.sumsq = sumsq
        self.lo = self.rank - 1 if self.rank > 0 else None         # neighbour below / above
        self.hi = self.rank + 1 if self.rank + 1 < self.world else None
        self.started = False

    def transfer(self):
        """Packed cut planes to the neighbours, theirs into the receive buffers."""
        d, ops = self.dist, []
        for side, peer in ((0, self.lo), (1, self.hi)):
            if peer is None:
                continue
            ops.append(d.P2POp(d.isend, self.engine.cut_send(side), peer, self.group))
            ops.append(d.P2POp(d.irecv, self.engine.cut_recv(side), peer, self.group))
        if ops:
            for req in d.batch_isend_irecv(ops):
                req.wait()

    def start(self):
        """The cut exchange of the initial state (every later one rides on a sweep)."""
        if self.world > 1:
            self.engine.pack_cut()
            self.transfer()
            self.engine.unpack_cut()
        self.started = True

    def sweep(self, nsweeps: int = 1):
        if self.world == 1:
            self.engine.sweep(nsweeps)
            return
        if not self.started:
            self.start()
        for _ in range(int(nsweeps)):
            self.engine.sweep_begin()      # cut planes first, their faces packed, the rest meanwhile
            self.transfer()                # the faces travel while the rest of the slab is updated
            self.engine.sweep_end()        # neighbours' faces into the ghost layers of the new state

    def residual(self) -> float:
        """L2 norm of the residual over the whole domain: one sum over the slabs' sums of squares."""
        if self.world > 1 and not self.started:
            self.start()
        t = self.sumsq()
        if self.world > 1:
            self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM, group=self.group)
        return math.sqrt(float(t.item()))


class LocalSlabs:
    """Several slabs of one domain in ONE process (engines on one device, or on devices with peer
    access): every slab's unpack reads its neighbours' send buffers in place."""

    def __init__(self, engines):
        self.engines = list(engines)
        self.started = False

    def _neighbour_planes(self, i):
        """(src_lo, ready_lo, src_hi, ready_hi) for slab i: what its neighbours packed towards it."""
        src_lo = ready_lo = src_hi = ready_hi = None
        if i > 0:
            src_lo, _, _, ready_lo = self.engines[i - 1].cut_info(1)
        if i + 1 < len(self.engines):
            src_hi, _, _, ready_hi = self.engines[i + 1].cut_info(0)
        return src_lo, ready_lo, src_hi, ready_hi

    def start(self):
        if len(self.engines) > 1:
            for e in self.engines:
                e.pack_cut()
            for i, e in enumerate(self.engines):
                e.unpack_cut(*self._neighbour_planes(i))
        self.started = True

    def sweep(self, nsweeps: int = 1):
        if len(self.engines) == 1:
            self.engines[0].sweep(nsweeps)
            return
        if not self.started:
            self.start()
        for _ in range(int(nsweeps)):
            for e in self.engines:
                e.sweep_begin()
            for i, e in enumerate(self.engines):
                e.sweep_end(*self._neighbour_planes(i))

    def residual(self, sumsq_of) -> float:
        """``sumsq_of(engine)`` -> that slab's sum of squared residuals (a float)."""
        if len(self.engines) > 1 and not self.started:
            self.start()
        return math.sqrt(sum(float(sumsq_of(e)) for e in self.engines))


def slab_context(n, b, halo, has_f, mode, part: int, parts: int, stream=None, flags: int = 0):
    """The library context of slab ``part`` of ``parts`` of the domain ``n`` in blocks ``b``
    (mode "fused" or "exchange"; with one part, any mode: it is then the whole domain)."""
    from . import jac
    n_slab, b_slab, cut_flags, _ = slab_of(n, b, part, parts)
    return jac.Jacobi(n_slab, b_slab, halo, has_f, mode, stream=stream, flags=flags | cut_flags)


def set_slab_boundary(engine, ndim: int, part: int, parts: int, bvals):
    """Dirichlet values of the domain faces this slab touches (a cut is not a domain face)."""
    for face, v in enumerate(bvals):
        on_cut = face // 2 == ndim - 1 and ((face & 1 and part + 1 < parts) or (not face & 1 and part > 0))
        if not on_cut:
            engine.set_boundary(face, v)
