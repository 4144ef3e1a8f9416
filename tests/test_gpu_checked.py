"""The bounds-checked build of the library (the same sources compiled with -DDYNAKV_CHECKED: every index a kernel takes
out of a table and turns into an address -- a cluster id, a page of a chain, a row of the gather list, a token slot --
is tested against the array it indexes) runs the parity and edge suites in a child process.  The suites' own
assertions check results as always; on top of that no index test may have failed (status bit BOUNDS, asserted by the
parity harness and the loop helper).  This stands in for a memory checker on the device code."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu


def test_parity_and_edge_suites_on_the_bounds_checked_build():
    from paper_2511_07427_b200.build import build
    build(checked=True)
    env = dict(os.environ, DYNAKV_LIBRARY="checked")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_gpu_parity.py"), os.path.join(ROOT, "tests", "test_gpu_edge.py")]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=800)
    tail = (r.stdout + r.stderr)[-4000:]
    assert r.returncode == 0, tail
    assert " passed" in tail and "failed" not in tail, tail
    print(tail.strip().splitlines()[-1])


def test_the_ordinary_build_has_no_index_tests():
    import paper_2511_07427_b200 as P
    if os.environ.get("DYNAKV_LIBRARY") == "checked":
        pytest.skip("this process runs the checked build")
    assert P.load_library().dynakv_checked_build() == 0
