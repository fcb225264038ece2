"""The bounded device-side waits really run out, in the permitted form: nothing faults, traps or spins without limit.

A second build of the library (short wait limits, plus a test hook that makes CTA 0's producer leave one pipeline
stage unissued: nothing armed, nothing in flight, no address touched) runs in a child process; the stage's barrier
never completes, the gate's wait expires after about a millisecond, the kernel raises NM_STATUS_TIMEOUT, drains and
returns, and the next call on the same stream matches the oracle.  One case per kernel family that this form has been
shown to be safe for (the 512-channel pair kernel's case is not run: see timeout_case.py), and one for the staged projection
kernel, where a warp leaves the bulk copies of one chunk unissued and its wait for the chunk expires."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _shortwait_lib():
    import importlib.util
    spec = importlib.util.spec_from_file_location("nm_build", os.path.join(ROOT, "paper_2206_15014_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod.build(variant="shortwait")


@pytest.mark.parametrize("family", ["one_cta", "one_cta_narrow", "pair", "pair_streamed", "pack_staged"])
def test_expired_wait_reports_timeout_and_leaves_the_context_usable(family):
    env = dict(os.environ, NMSPARSE_LIB=_shortwait_lib())
    r = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "timeout_case.py"), family], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and f"ok {family}" in r.stdout, r.stdout + r.stderr


def test_product_library_has_no_test_hook():
    import paper_2206_15014_b200 as nm
    with pytest.raises(nm.NmError) as e:
        nm.nm_debug_set_option("skip_stage", 1)
    assert e.value.code == nm.NM_ERR_UNSUPPORTED
