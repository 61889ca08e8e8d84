"""Writes the stored expected values under tests/golden/ from the CPU oracle, and nothing else.

    python tests/golden/make_golden.py

Every value comes from ``oracle/`` (never from the GPU library).  Two small cases:

  heated_edge_256.txt   the 256 x 256 heated-edge problem (zero start, edge +y held at 1, no
                        right-hand side) after 100 sweeps: sampled grid values and the residual norm
  poisson3d_24.txt      a 24 x 18 x 12 box in 8 x 6 x 4 blocks, normal right-hand side (seed 3),
                        zero start, 20 sweeps: sampled grid values and the residual norm

The paper prints no worked numerical example of its Jacobi proxy (Section V-C gives only the
domain and the iteration structure), so these are regression fixtures of the oracle as pinned by
tests/test_oracle_*.py, not figures from the paper.  Values are hexadecimal floating-point
literals: the files fix bits, not decimals.
"""
from __future__ import annotations

import sys
from pathlib import Path

import numpy as np

HERE = Path(__file__).resolve().parent
ROOT = HERE.parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

from oracle import orc  # noqa: E402
from paper_2210_01238_b200 import inputs  # noqa: E402  (seeded generators, no Jacobi arithmetic)

CASES = {
    "heated_edge_256": inputs.HEATED_EDGE_256,
    "poisson3d_24": inputs.scaled(inputs.POISSON3D_1024, (24, 18, 12), (8, 6, 4), sweeps=20, name="poisson3d_24"),
}


def sample_points(w: inputs.Workload, count: int = 48):
    """A fixed, seeded choice of interior points plus the corners of the grid."""
    rng = np.random.default_rng(20221001)
    pts = {tuple(int(rng.integers(0, n)) for n in w.n) for _ in range(count)}
    pts |= {tuple(0 for _ in w.n), tuple(n - 1 for n in w.n)}
    if w.name.startswith("c1"):
        pts |= {(0, 255), (128, 255), (128, 254), (127, 200), (128, 200)}   # next to the heated edge
    return sorted(pts)


def run_case(w: inputs.Workload):
    B = orc.Blocked(w.n, w.b, w.halo, w.has_f)
    for face, v in enumerate(w.boundary()):
        B.set_boundary(face, v)
    B.set_u(inputs.initial_u(w))
    f = inputs.rhs(w)
    if f is not None:
        B.set_f(f)
    B.sweep(w.sweeps)
    u, r = B.get_u(), B.residual()
    B.close()
    return u, r


def write_case(name: str, w: inputs.Workload):
    u, r = run_case(w)
    lines = [f"# {name}: grid {'x'.join(map(str, w.n))}, blocks {'x'.join(map(str, w.b))}, halo {w.halo}, "
             f"{w.sweeps} sweeps; written by tests/golden/make_golden.py from the CPU oracle",
             f"residual {float(r).hex()}"]
    for p in sample_points(w):
        lines.append("u " + " ".join(map(str, p)) + " " + float(u[tuple(reversed(p))]).hex())
    (HERE / f"{name}.txt").write_text("\n".join(lines) + "\n")


def read_case(name: str):
    """(residual, [(point, value), ...]) of a stored case."""
    residual, values = None, []
    for line in (HERE / f"{name}.txt").read_text().splitlines():
        if line.startswith("#") or not line.strip():
            continue
        parts = line.split()
        if parts[0] == "residual":
            residual = float.fromhex(parts[1])
        else:
            values.append((tuple(int(x) for x in parts[1:-1]), float.fromhex(parts[-1])))
    return residual, values


if __name__ == "__main__":
    for name, w in CASES.items():
        write_case(name, w)
        print("wrote", HERE / f"{name}.txt")
