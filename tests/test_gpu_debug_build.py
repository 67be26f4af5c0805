"""The index-check build of the library (librobe_debug.so: the same sources with -DROBE_DEBUG, every
computed index compared with its bound before use; it stands in for a memory checker, which cannot
be run on the machines this is tested on).  The small shape lists of the parity tests - every kernel
family, wrap-heavy arrays, ragged blocks, windows, long walks, kept block starts - are run against
it in a child process; each test there must match the oracle as usual AND leave the debug word at
zero (tests/conftest.py checks it after every test)."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu

SELFTEST = """
import paper_2108_02191_b200 as robe
assert robe.robe_debug_status() == 0
assert robe.robe_debug_selftest() == 0
assert robe.robe_debug_status() == robe.ROBE_DBG_SELFTEST   # the planted failure is reported ...
assert robe.robe_debug_status() == 0                        # ... once
print("selftest ok")
"""


def _debug_env():
    from paper_2108_02191_b200 import build
    return dict(os.environ, ROBE_LIBRARY=build.build_debug())


def test_release_build_has_no_checks():
    import paper_2108_02191_b200 as robe
    if os.environ.get("ROBE_LIBRARY"):
        pytest.skip("running on the index-check build")
    assert robe.robe_debug_status() == robe.ROBE_ERR_UNSUPPORTED
    assert robe.robe_debug_selftest() == robe.ROBE_ERR_UNSUPPORTED


def test_reporting_path_of_the_index_check_build():
    r = subprocess.run([sys.executable, "-c", SELFTEST], env=_debug_env(), cwd=ROOT, capture_output=True,
                       text=True, timeout=600)
    assert r.returncode == 0 and "selftest ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]


def test_shape_lists_run_clean_on_the_index_check_build():
    if os.environ.get("ROBE_LIBRARY"):
        pytest.skip("already inside the child run")
    pick = ("forward_shapes or backward_shapes or window_apply or step_sharing or vector_kernel or "
            "lane_hashed or adam or adagrad or merged_rows or table_major or int32 or cfg1 or hot_id or bit_reproducible")
    r = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "tests/test_zz_no_alloc.py",
                        "-m", "gpu", "-x", "-q", "-k", pick + " or two_calls or fused_sgd"],
                       env=_debug_env(), cwd=ROOT, capture_output=True, text=True, timeout=3000)
    assert r.returncode == 0, r.stdout[-4000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
