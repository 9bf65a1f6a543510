"""The debug build (-DCDGRAB_DEBUG): index checks in front of the decision routines' writes and
guard bytes around every handle-owned allocation, verified by cdgrab_status and cdgrab_destroy.
It stands in for a memory checker: a step on every code path leaves all guards intact, and a
guard byte overwritten FROM THE HOST is reported as CDGRAB_ERR_CORRUPT.  Nothing here writes out
of bounds on the device.  Runs in a child process, because a process loads one build of the library."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import ctypes as C, sys, torch
from paper_2302_00845_b200 import binding, build
build.build(variant="debug")
L = binding.lib()
L.cdgrab_debug_guard_count.argtypes = [C.c_void_p]
L.cdgrab_debug_poke_guard.argtypes = [C.c_void_p, C.c_int, C.c_int]
shapes = [(4, 8, 1024, "f32", "literal"), (8, 8, 4096, "f32", "fused"), (16, 8, 70000, "f32", "fma"),
          (5, 8, 1023, "f32", "fma"), (40, 8, 20000, "bf16", "umma"), (48, 8, 20004, "f32", "umma"),
          (70, 8, 3000, "bf16", "fma")]
for m, n, d, dtype, path in shapes:
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    h = binding.CdGrab(m, n, d, dtype)
    assert h.path == path, (h.path, path)
    guards = L.cdgrab_debug_guard_count(h._h)
    assert guards >= 10, guards
    h.begin_epoch()
    for k in range(n // 2):
        h.step((torch.randn(2, m, d, device="cuda") + 0.1).to(tdt))
    h.end_epoch()
    assert h.status() == binding.OK, (path, h.status())
    # one byte of a guard block overwritten from the host: in front of the first allocation, behind the last
    which, tail = (0, 0) if m % 2 == 0 else (guards - 1, 1)
    assert L.cdgrab_debug_poke_guard(h._h, which, tail) == binding.OK
    assert h.status() == binding.ERR_CORRUPT
    assert L.cdgrab_destroy(h._h) == binding.ERR_CORRUPT
    h._h = None
    print("ok", m, n, d, dtype, path, "guards", guards)
print("DEBUG-BUILD-OK")
"""


def test_steps_leave_guards_intact_and_a_poked_guard_is_reported():
    env = dict(os.environ, CDGRAB_LIB="libcdgrab_debug.so", PYTHONPATH=ROOT)
    env.pop("CDGRAB_FORCE_PATH", None)
    res = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0 and "DEBUG-BUILD-OK" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]


def test_release_build_has_no_guard_exports():
    from paper_2302_00845_b200 import binding
    assert not hasattr(binding.lib(), "cdgrab_debug_poke_guard")
