"""The parity suites once more against the checked build of the library (-DAMOEBA_CHECK_ITEMS): every work item of
every kernel is tested on the device against the extent of the buffers it addresses before it is moved; an item that
would reach outside is skipped and reported as AMOEBA_ERR_INTERNAL.  Every test of those suites compares the status
word with the oracle's, so the run only passes if no item of any case ever left its buffer.  (compute-sanitizer is
not available on the GPU pool; this, the guard regions and the whole-buffer comparisons stand in for it.)"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_parity_suites_pass_with_per_item_extent_checks():
    import paper_2509_19729_b200.build as b

    b.build(checked=True)
    env = dict(os.environ, AMOEBA_BINDING_BUILD="checked")
    suites = ["tests/test_gpu_parity.py", "tests/test_gpu_reshape.py", "tests/test_gpu_merge.py"]
    r = subprocess.run([sys.executable, "-m", "pytest", *suites, "-m", "gpu", "-x", "-q", "-p", "no:cacheprovider"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    tail = "\n".join(r.stdout.splitlines()[-15:])
    assert r.returncode == 0, tail
    assert " passed" in tail and "libamoeba_checked.so" in subprocess.run(
        [sys.executable, "-c", "import paper_2509_19729_b200 as A; print(A.library_path())"], cwd=ROOT, env=env,
        capture_output=True, text=True).stdout
