"""The stand-in for a memory sanitizer: a build of the library whose kernels compare every global
address with the array it belongs to (-DJAC_CHECK_BOUNDS), run through the small parity tests.  An
access outside its array would be skipped and recorded, and closing the context then raises."""
import ctypes as C
import os
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def checked_lib():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_01238_b200 import build
    return build.build_checked()


WORKER = r"""
import sys
sys.path.insert(0, sys.argv[1])
import numpy as np
from paper_2210_01238_b200 import jac
from oracle import orc
n, b = (96, 64), (32, 16)
u0 = np.random.default_rng(3).uniform(-1, 1, (64, 96))
# 1. an ordinary run: checked, nothing recorded, right answer
J = jac.Jacobi(n, b, 1, False, "exchange")
J.set_u(u0); J.sweep(3)
B = orc.Blocked(n, b, 1); B.set_u(u0); B.sweep(3)
assert np.array_equal(J.get_u(), B.get_u())
assert J.bounds_record() == (True, 0), J.bounds_record()
J.close()
# 2. the check at work: hold the kernels to a range that ends early; accesses that are in fact
#    legitimate are now "outside", get skipped, and the first one is on record -- no access left the workspace
for mode, array, cut, kid in (("fused", 0, 65536, 1), ("temporal", 0, 65536, 9), ("exchange", 1, 4096, 4)):
    J = jac.Jacobi(n, b, 1, False, mode)
    J.set_u(u0)
    assert jac.lib().jac_debug_shrink_bounds(J._ctx, array, cut) == 0
    if mode == "exchange":
        J.pack_halos()
    else:
        J.sweep(1)
    checked, rec = J.bounds_record()
    assert checked and rec != 0 and rec >> 56 == kid and (rec >> 52) & 15 == array, (mode, hex(rec))
    try:
        J.close()
        raise SystemExit("closing a context with a record must raise")
    except jac.JacError:
        pass
print("worker ok")
"""


def test_the_check_records_and_skips(checked_lib, tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, JAC_LIB=str(checked_lib))
    r = subprocess.run([sys.executable, str(script), str(ROOT)], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "worker ok" in r.stdout, r.stdout + r.stderr


def test_parity_tests_pass_under_the_checked_build(checked_lib):
    """Every schedule, 2D and 3D, remainder blocks, wide halos, slabs: the small shapes of the parity
    suites with all addresses checked.  A context that recorded a violation raises when it is closed."""
    env = dict(os.environ, JAC_LIB=str(checked_lib))
    sel = ("test_sweep_matches_oracle or test_pack_and_unpack or test_temporal_blocking or fused_residual or "
           "first_sweep or norms_every or solve_stops or remainder or wide or resident or slab_contexts or cut_planes")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-k", sel,
                        "tests/test_gpu_parity.py", "tests/test_gpu_remainder.py", "tests/test_gpu_wide.py",
                        "tests/test_gpu_resident.py", "tests/test_gpu_slabs.py", "tests/test_gpu_staging.py"],
                       cwd=str(ROOT), env=env, capture_output=True, text=True, timeout=3000)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout


def test_the_ordinary_build_makes_no_checks():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2210_01238_b200 import jac
    with jac.Jacobi((32, 32), (16, 16)) as J:
        J.sweep(2)
        assert J.bounds_record() == (False, 0)
        assert jac.lib().jac_debug_shrink_bounds(J._ctx, 3, 0) == jac.EINVAL
