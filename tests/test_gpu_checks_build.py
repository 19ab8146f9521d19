"""The bounds-check build (libarb_checks.so, -DARB_CHECKS): the small parity cases of every kernel run once more in
a child process that loads it.  Every index the kernels derive on the device is tested there before it is used, and
the buffers of the context lie between guard zones; a clean run raises no ARB_DEV_CHECK_FAILED (the parity tests
assert a zero status word) and leaves every guard byte as it was.  This stands in for a memory checker."""
import os
import re
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent

SMALL_CASES = ["tests/test_gpu_decode_step.py", "tests/test_gpu_step_loop.py", "tests/test_gpu_route.py",
               "tests/test_gpu_attn.py"]


def test_small_parity_cases_under_the_bounds_check_build():
    from paper_2512_05033_b200 import build
    build.build(checks=True)
    env = dict(os.environ, ARB_LIB_VARIANT="checks")
    # the small cases: the long-sequence and full-size ones add nothing a range test could see
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-s", "-m", "gpu", "-k",
                        "not split and not full and not mixed_shapes and not 40000", *SMALL_CASES],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = r.stdout[-3000:] + r.stderr[-2000:]
    assert r.returncode == 0, tail
    m = re.search(r"guard zones: (\d+) bytes checked, (\d+) overwritten", r.stdout)
    assert m is not None, tail
    assert int(m.group(1)) > 0 and int(m.group(2)) == 0, tail


def test_a_planted_overrun_is_seen_by_the_guard_check():
    """The guard check itself: a byte written just past a context-owned buffer is counted (done from the host side
    by an entry point that exists in the bounds-check build only; the bytes belong to the context's own allocation)."""
    from paper_2512_05033_b200 import build
    build.build(checks=True)
    code = (
        "import ctypes\n"
        "from paper_2512_05033_b200 import binding\n"
        "c = binding.Context(0)\n"
        "bad, checked = c.guard_zones()\n"
        "assert bad == 0 and checked > 0, (bad, checked)\n"
        "poke = binding.lib.arb_debug_poke_guard\n"
        "poke.restype = ctypes.c_int; poke.argtypes = [ctypes.c_void_p, ctypes.c_int]\n"
        "assert poke(c._h, 3) == 0\n"          # three bytes just in front of the workspace
        "assert c.guard_zones()[0] == 3\n"
        "print('planted overrun seen')\n")
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=dict(os.environ, ARB_LIB_VARIANT="checks"),
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and "planted overrun seen" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]
