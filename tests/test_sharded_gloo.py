"""The multi-rank protocol of the slab sharding on CPU (gloo, world sizes 2 and 3): which rank owns
which block planes, which packed cut plane goes to which neighbour, and the one-number reduction of
the residual.  Every rank runs ``SlabRank`` -- the class the GPU ranks run -- over an engine that
keeps its slab in the CPU oracle, so the gathered result can be held against the oracle's run of the
unpartitioned domain, bit for bit."""
import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import numpy as np
import torch
import torch.distributed as dist
from oracle import orc
from paper_2210_01238_b200.sharded import SlabRank, slab_of, slab_slice

world = int(sys.argv[3])
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%s" % sys.argv[2],
                        rank=int(os.environ["RANK"]), world_size=world)
rank = dist.get_rank()


class OracleEngine:
    # a slab kept in the CPU oracle, with the method names of the library's slab context
    def __init__(self, n_slab, b_slab, h, has_f, flags):
        self.B = orc.Blocked(n_slab, b_slab, h, has_f)
        self.cut = [bool(flags & 2), bool(flags & 4)]
        self.send = [torch.zeros(self.B.cut_elems(), dtype=torch.float64) for _ in range(2)]
        self.recv = [torch.zeros(self.B.cut_elems(), dtype=torch.float64) for _ in range(2)]
    def pack_cut(self):
        for side in (0, 1):
            if self.cut[side]:
                self.send[side].copy_(torch.from_numpy(self.B.pack_cut(side)))
    def cut_send(self, side): return self.send[side]
    def cut_recv(self, side): return self.recv[side]
    def unpack_cut(self):
        for side in (0, 1):
            if self.cut[side]:
                self.B.unpack_cut(side, self.recv[side].numpy())
    def sweep_begin(self):
        self.B.sweep(1)          # faces between the slab's own blocks, then the update
        self.pack_cut()          # the new state's cut faces
    def sweep_end(self):
        self.unpack_cut()
    def sweep(self, k):
        self.B.sweep(k)


for n, b, h, has_f in (((24, 20), (6, 4), 1, True), ((10, 8, 14), (5, 4, 2), 2, True), ((12, 9, 11), (4, 3, 3), 1, True), ((12, 12, 12), (4, 4, 4), 1, False)):
    rng = np.random.default_rng(51)                       # every rank draws the same global arrays
    shape = tuple(reversed(n))
    u0, f = rng.uniform(-1, 1, shape), rng.uniform(-1, 1, shape)
    bvals = [0.5, -1.0, 2.0, 3.0, -0.25, 1.5][: 2 * len(n)]
    n_slab, b_slab, flags, first = slab_of(n, b, rank, world)
    E = OracleEngine(n_slab, b_slab, h, has_f, flags)
    for face, v in enumerate(bvals):
        E.B.set_boundary(face, v)
    sl = slab_slice(n, b, rank, world)
    E.B.set_u(np.ascontiguousarray(u0[sl]))
    if has_f:
        E.B.set_f(np.ascontiguousarray(f[sl]))

    def sumsq():
        return torch.tensor([E.B.residual() ** 2], dtype=torch.float64)

    R = SlabRank(E, rank, world, dist, sumsq)
    assert (R.lo, R.hi) == (rank - 1 if rank > 0 else None, rank + 1 if rank + 1 < world else None)
    R.sweep(4)
    r4 = R.residual()
    R.sweep(2)
    mine = E.B.get_u()
    # gather the slabs on rank 0 and compare with the run of the whole domain
    parts = [None] * world
    dist.all_gather_object(parts, mine)
    mono = orc.mono_padded(n, bvals)
    mono[(slice(1, -1),) * len(n)] = u0
    m4 = orc.mono_sweep(mono, f if has_f else None, 4)
    want_r4 = orc.mono_residual(m4, f if has_f else None)
    m6 = orc.mono_sweep(m4, f if has_f else None, 2)
    assert np.array_equal(np.concatenate(parts, axis=0), m6[(slice(1, -1),) * len(n)]), n
    assert abs(r4 - want_r4) <= 1e-12 * want_r4, (r4, want_r4)
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


@pytest.mark.parametrize("world", [2, 3])
def test_slab_ranks_reproduce_the_unpartitioned_run(tmp_path, orc, world):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = str(31500 + (os.getpid() * 7 + world) % 2000)
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(world), OMP_NUM_THREADS="1")
        procs.append(subprocess.Popen([sys.executable, str(script), str(ROOT), port, str(world)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=300)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out
