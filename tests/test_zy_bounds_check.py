"""The range-checking debug build of the library (-DST_BOUNDS_CHECK).

Every store whose index comes out of the packed-index arithmetic is checked on the device; a violation is
recorded, the store is skipped and st_check_status returns ST_ERR_DEV_BOUNDS.  The library is chosen when the
binding is first loaded, so the checks run in a child process: a part of the parity suite (every call, small
shapes and the named MTTKRP / TTM / third-moment sizes) against libstructtensor_check.so, whose per-test
fixture reads the status after each test.  The reporting path itself is tested with an index that is out of
range by construction and touches no memory.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CHECK_LIB = os.path.join(ROOT, "paper_2211_10482_b200", "libstructtensor_check.so")

pytestmark = pytest.mark.gpu

SELF_TEST = r"""
import paper_2211_10482_b200 as st
assert st.lib().st_bounds_checked_build() == 1
assert st.st_check_status() == st.ST_OK
assert st.lib().st_bounds_self_test(None) == st.ST_OK
assert st.st_check_status() == st.ST_ERR_DEV_BOUNDS      # recorded by the device-side check
assert st.st_check_status() == st.ST_OK                  # reading cleared the record
print("self test ok")
"""


def run(args):
    env = dict(os.environ, STRUCTTENSOR_LIB=CHECK_LIB)
    return subprocess.run([sys.executable, *args], cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)


def test_debug_build_reports_an_out_of_range_index_and_clears_it():
    if not os.path.exists(CHECK_LIB):
        from paper_2211_10482_b200 import _build
        _build.build(check=True)
    res = run(["-c", SELF_TEST])
    assert res.returncode == 0 and "self test ok" in res.stdout, res.stdout + res.stderr


def test_normal_build_has_no_self_test():
    import paper_2211_10482_b200 as st
    assert st.lib().st_bounds_checked_build() == 0
    assert st.lib().st_bounds_self_test(None) == st.ST_ERR_UNSUPPORTED


def test_parity_suite_under_the_range_checks():
    if not os.path.exists(CHECK_LIB):
        from paper_2211_10482_b200 import _build
        _build.build(check=True)
    select = ("pack_unpack or small or closed_form or mttkrp_config or ttm_config or moment3_config or moment4 or "
              "slice or structure or thp or chain or fixed_order or split or tf32")
    res = run(["-m", "pytest", "tests/test_gpu_parity.py", "-q", "-x", "-m", "gpu", "-k", select])
    tail = (res.stdout + res.stderr)[-3000:]
    assert res.returncode == 0, tail
    assert " passed" in res.stdout and "failed" not in res.stdout, tail
