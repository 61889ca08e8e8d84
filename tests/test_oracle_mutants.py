"""The pins have teeth: each planted mistake in a copy of the oracle's source must make at
least one pin fail.  The mistakes are planted on the CPU, in the oracle, never in a kernel."""
import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
SRC = ROOT / "oracle" / "jacobi_oracle.c"

MUTANTS = {
    "wrong_2d_weight": ("out[p] = s * 0.25;", "out[p] = s * 0.2;", 1),
    "sign_of_east_neighbour": ("(u[p - 1] + u[p + 1])", "(u[p - 1] - u[p + 1])", 0),
    "sign_of_f": ("if (f) s = s + f[", "if (f) s = s - f[", 0),
    "transposed_f_2d": ("f[(j - 1) * nx + (i - 1)]", "f[(i - 1) * ny + (j - 1)]", 0),
    "one_sixth_off_by_an_ulp": ("const double c6 = 1.0 / 6.0;",
                                "const double c6 = 0.16666666666666669;", 0),
    "z_term_reads_one_side_twice": ("s = s + (u[p - pxy] + u[p + pxy]);",
                                    "s = s + (u[p - pxy] + u[p - pxy]);", 1),
    "blocked_update_drops_z": ("if (s->ndim == 3) sum = sum + (u[p - pxy] + u[p + pxy]);\n"
                               "                    if (f) sum = sum + f[(k * s->b[1] + j) * s->b[0] + i];\n"
                               "                    o[p]",
                               "if (f) sum = sum + f[(k * s->b[1] + j) * s->b[0] + i];\n"
                               "                    o[p]", 1),
    "pack_strip_shifted": ("lo[axis] = ghost ? -s->h : 0;", "lo[axis] = ghost ? -s->h : 1;", 1),
    "unpack_reads_same_side": ("blk_send(s, nb, face ^ 1)", "blk_send(s, nb, face)", 1),
    "residual_sign": ("const double r = s - t;", "const double r = s + t;", 1),
    "residual_centre_weight": ("t = 6.0 * u[p];", "t = 4.0 * u[p];", 1),
    "exchange_after_update": ("        orc_blocked_pack(s);\n        orc_blocked_unpack(s);\n"
                              "        orc_blocked_update(s);",
                              "        orc_blocked_update(s);\n        orc_blocked_pack(s);\n"
                              "        orc_blocked_unpack(s);", 1),
    "wide_strips_leave_out_the_ghost_extent": ("if (a != axis) { lo[a] = -s->h; hi[a] = hi[a] + s->h; }",
                                               "if (a != axis) { lo[a] = 0; }", 1),
    "group_updates_do_not_shrink": ("orc_blocked_update_ext(s, t - m);", "orc_blocked_update_ext(s, 0);", 1),
    "extended_update_moves_dirichlet_cells": ("                        o[p] = u[p];\n                        continue;\n",
                                              "", 1),
    "extended_update_reads_own_f": ("return s->f[owner * s->blk_elems +",
                                    "owner = (c[2] * s->g[1] + c[1]) * s->g[0] + c[0]; return s->f[owner * s->blk_elems +", 1),
    "wide_unpack_reads_same_side": ("wsend + (nb * 6 + (face ^ 1)) * wmax", "wsend + (nb * 6 + face) * wmax", 1),
    "wide_exchange_skips_last_axis": ("for (int axis = 0; axis < s->ndim; ++axis)\n        wide_phase",
                                      "for (int axis = 0; axis + 1 < s->ndim; ++axis)\n        wide_phase", 1),
    "dirichlet_of_remainder_block_at_full_size_position": (
        "if (face & 1) { lo[axis] = ext[axis]; hi[axis] = ext[axis] + s->h; }",
        "if (face & 1) { lo[axis] = s->b[axis]; hi[axis] = s->b[axis] + s->h; }", 1),
    "cut_pack_takes_the_ghost_layers": ("strip_range(s, blk0 + m, face, 0, lo, hi);", "strip_range(s, blk0 + m, face, 1, lo, hi);", 1),
    "cut_unpack_fills_the_interior_strip": ("strip_range(s, blk0 + m, face, 1, lo, hi);\n        const double *buf = in",
                                            "strip_range(s, blk0 + m, face, 0, lo, hi);\n        const double *buf = in", 1),
    "cut_plane_of_the_wrong_end": ("*blk0 = side ? (s->g[sa] - 1) * *count : 0;", "*blk0 = side ? 0 : (s->g[sa] - 1) * *count;", 1),
    "cut_slots_overlap": ("double *buf = out + m * s->face_elems[face];", "double *buf = out + m * (s->face_elems[face] - 1);", 1),
    "update_runs_over_the_full_block_size": (
        "        for (int64_t k = 0; k < ext[2]; ++k)\n            for (int64_t j = 0; j < ext[1]; ++j)\n"
        "                for (int64_t i = 0; i < ext[0]; ++i) {\n                    const int64_t p = pad_index(s, i, j, k);",
        "        for (int64_t k = 0; k < s->b[2]; ++k)\n            for (int64_t j = 0; j < s->b[1]; ++j)\n"
        "                for (int64_t i = 0; i < s->b[0]; ++i) {\n                    const int64_t p = pad_index(s, i, j, k);", 1),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(name, tmp_path):
    old, new, count = MUTANTS[name]
    text = SRC.read_text()
    assert old in text, f"mutation site for {name} not found"
    mutated = text.replace(old, new) if count == 0 else text.replace(old, new, count)
    assert mutated != text
    c = tmp_path / "mutant.c"
    so = tmp_path / "mutant.so"
    c.write_text(mutated)
    subprocess.run(["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
                    "-o", str(so), str(c), "-lm"], check=True)
    env = dict(os.environ, ORC_LIB=str(so))
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        str(ROOT / "tests" / "test_oracle_sweep.py"),
                        str(ROOT / "tests" / "test_oracle_blocks.py"),
                        str(ROOT / "tests" / "test_oracle_wide.py"),
                        str(ROOT / "tests" / "test_oracle_remainder.py"),
                        str(ROOT / "tests" / "test_oracle_slabs.py")],
                       cwd=ROOT, env=env, capture_output=True, text=True)
    assert r.returncode == 1, f"mutant {name} survived the pins:\n{r.stdout[-2000:]}"
    assert "failed" in r.stdout
