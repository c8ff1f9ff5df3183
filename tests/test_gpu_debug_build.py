"""The bounds-checking build (-DTRA_DEBUG): every global index of the kernels is checked on the
device and a violation is recorded in the plan status instead of faulting.  The whole hot path
runs through it on the small, ragged and text shapes; the status must stay clean and every output
must equal the normal build's bit for bit."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


def _run(lib_path):
    env = dict(os.environ)
    if lib_path:
        env["TRA_B200_LIB"] = lib_path
    else:
        env.pop("TRA_B200_LIB", None)
    res = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "debug_build_case.py")], env=env, cwd=ROOT,
                         capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stderr[-2000:]
    return json.loads(res.stdout.strip().splitlines()[-1])


@pytest.mark.timeout(1800)
def test_bounds_checking_build_is_clean_and_bit_identical():
    import shutil
    from paper_2608_02504_b200 import build
    # compiled here, on the machine that runs it, whenever a compiler is at hand (else the shipped
    # library is used if its sources are unchanged)
    have_nvcc = os.path.exists(os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")) or shutil.which("nvcc")
    debug_lib = build.build(debug=True, force=bool(have_nvcc))
    checked = _run(debug_lib)
    normal = _run(None)
    assert checked["lib"] == "libtra_b200_debug.so" and normal["lib"] == "libtra_b200.so"
    for c, n in zip(checked["cases"], normal["cases"]):
        assert c["status"] == 0, c                       # no index out of range, consistent work lists
        assert c["status_overflow"] == -3, c             # the overflow is reported as such, nothing else
        assert c["status_wild"] == 0, c
        assert c["status_bad_list"] == -6 and n["status_bad_list"] == 0      # TRA_ERR_BOUNDS: the check is live
        assert c["digest"] == n["digest"]                # same bits from both builds
