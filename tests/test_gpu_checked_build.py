"""The -DPOT_CHECKED build (device-side index checks in front of stores, atomics and streamed shared-memory reads; a
failed check writes a code to the error words and skips the access) runs the small-shape parity tests in a child
process: every result must still match the oracle and the error words must stay zero.  It stands in for
compute-sanitizer, which these tests cannot use.  No test makes a kernel go out of range on purpose."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_shape_suite_against_the_checked_build():
    from paper_2507_11959_b200 import build
    lib = build.build(checked=True)
    env = dict(os.environ, POT_B200_LIB=str(lib))
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_gpu_gemv.py", "tests/test_gpu_prefill.py", "tests/test_gpu_dequant.py", "tests/test_gpu_bf16.py",
           "tests/test_gpu_dependent_launches.py", "tests/test_zz_no_alloc.py"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout, r.stdout[-1000:]
