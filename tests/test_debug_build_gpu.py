"""The checked build of the library (-DBM_DEBUG: every cache row index the kernels write with plain stores is tested
against the cache's capacity, a 256-byte guard sits behind every slab of the arena) runs the small lock-step parity
cases: same results, a clean status word, every guard intact.  It stands in for a memory checker on the device."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


def _debug_lib():
    from paper_2412_05693_b200.build import build
    return build(debug=True)


def test_small_parity_cases_pass_on_the_checked_build():
    env = dict(os.environ, BATCHMAX_LIB=_debug_lib())
    keys = ("small_shapes or random_shapes or random_cadences or unordered_cache_lockstep or short_blocks or "
            "window_pooled_rule_lockstep or average_std_rule_lockstep or left_padded or decode_with_one_cache")
    out = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_parity_gpu.py"), "-x", "-q",
                          "-m", "gpu", "-k", keys], capture_output=True, text=True, env=env, cwd=ROOT, timeout=1500)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-2000:]
    assert " passed" in out.stdout and "failed" not in out.stdout


CHECK = """
import sys
sys.path.insert(0, %r)
import paper_2412_05693_b200 as bm
from paper_2412_05693_b200.workloads import Workload, config_for
wl = Workload("dbg", b=2, Hq=4, Hkv=2, d=64, dtype="f32", s=64, B=16, K=16, steps=2)
cache = bm.BatchMaxCache(config_for(wl))
assert cache.status() == 0 and cache.check_canaries() == 0
cache.selftest_row_check()
print("debug", int(bm.debug_build()), "status", cache.status(), "canaries", cache.check_canaries())
cache.clear_status()
assert cache.status() == 0
"""


def test_row_test_reports_a_bad_index_without_faulting():
    # the self-test asks the row test about the first index past a cache: the checked build records BM_ERR_BOUNDS and
    # the context stays usable; the ordinary build has no such test and stays clean
    for lib, want in ((_debug_lib(), "debug 1 status 7 canaries 0"), (None, "debug 0 status 0 canaries 0")):
        env = dict(os.environ)
        env.pop("BATCHMAX_LIB", None)
        if lib is not None:
            env["BATCHMAX_LIB"] = lib
        out = subprocess.run([sys.executable, "-c", CHECK % ROOT], capture_output=True, text=True, env=env, timeout=300)
        assert out.returncode == 0, out.stderr[-2000:]
        assert want in out.stdout, out.stdout
