"""The bounds-checking build of the library (-DTA_BOUNDS_CHECK: every global index the tensor-core and decode
kernels form is compared with its tensor's extent on the device; a failure sets TA_DEVERR_BAD_INDEX and skips the
access).  The small-shape parity tests are run once more in a child process that loads that build; each of them
asserts that the device error word stays zero, so a pass here means no kernel formed an out-of-range index on any
of those shapes, ragged tails and empty caches included."""
import os
import subprocess
import sys

import pytest

from paper_2603_30033_b200 import binding as Bd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CHILD = "TA_BOUNDS_CHECK_CHILD"


@pytest.mark.gpu
@pytest.mark.skipif(os.environ.get(CHILD) == "1", reason="already inside the bounds-checking run")
def test_small_shapes_under_the_bounds_checking_build():
    env = dict(os.environ, TUCKER_ATTN_LIB="checked")
    env[CHILD] = "1"
    sel = ("small_shapes_tensor_core_path or decode_tensor_core_path or writes_cache or shared or garbage or "
           "growing or checked_library or fused_and_unfused or bad_cache_len or latent_rope")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-v", "-m", "gpu", "-k", sel, "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests")], env=env, cwd=ROOT, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert "test_checked_library_is_the_one_loaded PASSED" in r.stdout


@pytest.mark.gpu
@pytest.mark.skipif(os.environ.get(CHILD) != "1", reason="runs only inside the bounds-checking run")
def test_checked_library_is_the_one_loaded():
    assert Bd.bounds_checked() and Bd.LIB_PATH.endswith("libtucker_attn_checked.so")


@pytest.mark.gpu
def test_normal_build_carries_no_checks():
    if os.environ.get(CHILD) != "1":
        assert not Bd.bounds_checked()
