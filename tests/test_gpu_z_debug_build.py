"""The debug build of the library (-DQESGD_DEBUG): the codec kernels check every store index and
the indices of their code and scale loads against the buffer's extent and set QESGD_STATUS_RANGE
instead of touching memory outside it.  The small and ragged parity cases are run once more
against that build, in a process of its own: they compare with the oracle and with an expected
status word, so a range flag anywhere fails them."""
import os
import subprocess
import sys

import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_SELFTEST = r"""
import sys
sys.path.insert(0, sys.argv[1])
from paper_1901_03040_b200 import qesgd
assert qesgd.lib.qesgd_debug_build() == 1
c = qesgd.Context(0, None)
assert c.qesgd_status() == 0
assert qesgd.lib.qesgd_debug_range_selftest(c._h) == qesgd.OK
assert c.qesgd_status() == qesgd.STATUS_RANGE       # the flag, and no access was made
assert c.qesgd_status() == 0
c.close()
print("range selftest ok")
"""


def _debug_env():
    from paper_1901_03040_b200 import build
    try:
        build.build(debug=True)
    except Exception as exc:  # noqa: BLE001  (no nvcc on this machine and no library shipped with the tree)
        if not os.path.exists(build.LIB_DEBUG):
            pytest.skip(f"the debug library is not built and cannot be built here: {exc}")
    return dict(os.environ, QESGD_DEBUG="1")


def test_release_build_has_no_range_checks():
    from paper_1901_03040_b200 import qesgd
    if os.environ.get("QESGD_DEBUG") == "1":
        pytest.skip("this process already runs the debug build")
    assert qesgd.lib.qesgd_debug_build() == 0
    c = qesgd.Context(0, None)
    assert qesgd.lib.qesgd_debug_range_selftest(c._h) == qesgd.EINVAL
    c.close()


def test_range_check_reports_instead_of_faulting():
    out = subprocess.run([sys.executable, "-c", _SELFTEST, ROOT], env=_debug_env(), capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, (out.stdout + out.stderr)[-3000:]
    assert "range selftest ok" in out.stdout


def test_small_parity_cases_on_the_debug_build():
    if os.environ.get("QESGD_DEBUG") == "1":
        pytest.skip("already inside the debug run")
    pick = ("small_and_ragged or unaligned or encode_batch or nonfinite or subnormal or fixed_delta "
            "or decode_matches or small_sizes or k1_on_grid or requantize or axpy or fused_inner")
    out = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"),
                          "-x", "-q", "-m", "gpu", "-k", pick, "-p", "no:cacheprovider"],
                         env=_debug_env(), capture_output=True, text=True, timeout=1800, cwd=ROOT)
    assert out.returncode == 0, (out.stdout + out.stderr)[-4000:]
    assert " passed" in out.stdout
