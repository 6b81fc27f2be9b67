"""The bounds-checking build (-DTRI_INV_DEBUG, libtri_inv_debug.so) stands in for a memory checker: every global store
and table read of the kernels is range-checked, swizzled shared-memory offsets are checked against their tile, and the
mbarrier phase each wait names is checked against the copies requested so far.  A violation raises
TRI_INV_ERR_DEBUG_CHECK in the device status word and skips the access; nothing traps.  This test runs the small
parity cases of the suite through that library in a child process (the library is chosen when the binding loads) and
requires them to pass with the status word clean."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_cases_pass_under_the_bounds_checking_build():
    sys.path.insert(0, ROOT)
    from paper_2605_21325_b200 import build as lib_build
    lib = lib_build.build(debug=True)
    env = dict(os.environ, TRI_INV_LIB=lib)
    sel = "small or ragged or short or raw or refinement or fp16 or shifted or per_channel_decay_through or static_entry_matches"
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-k", sel,
                        "tests/test_parity_gpu.py", "tests/test_decay_forms_gpu.py", "tests/test_zz_no_alloc.py"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (r.stdout + r.stderr)[-3000:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "failed" not in r.stdout, tail


CHILD = r"""
import ctypes, sys
import numpy as np, torch
from paper_2605_21325_b200 import binding as b, workloads as wl
for C, dtype, d in ((64, wl.BF16, 128), (128, wl.BF16, 128), (64, wl.F32, 64)):
    inp = wl.make("dbg", 1, 6 * C, 3, d, d, C, dtype, seed=5)
    dev = b.to_device(inp)
    ref = b.fused(dev["K"], dev["V"], dev["beta"], dev["g"], C)
    torch.cuda.synchronize()
    assert b.last_device_status() == 0
    out = (torch.full_like(ref[0], float("nan")), torch.full_like(ref[1], float("nan")), torch.full_like(ref[2], float("nan")))
    desc, _ = b.make_desc(1, inp.T, inp.H, d, d, C, b._dtype_code(dev["K"]))
    rc = b.load().tri_inv_selftest_bounds_check(b._p(dev["K"]), b._p(dev["V"]), b._p(dev["beta"]), b._p(dev["g"]),
                                                b._p(out[0]), b._p(out[1]), b._p(out[2]), ctypes.byref(desc), None)
    torch.cuda.synchronize()
    assert rc == 0
    st = b.last_device_status()
    assert st == int(sys.argv[1]), (C, st)
    last = slice(inp.T - C, inp.T)
    for r, o in zip(ref, out):
        assert torch.equal(r[:, :inp.T - C], o[:, :inp.T - C])                    # everything before the last chunk is right
        if st: assert bool(torch.isnan(o[:, last].float()).all())                  # the refused items wrote nothing
        else: assert torch.equal(r[:, last], o[:, last])
    assert b.last_device_status() == 0
print("ok")
"""


def test_a_violation_is_reported_and_the_access_skipped():
    """tri_inv_selftest_bounds_check understates the token bound by one chunk (the buffers keep their full size, so
    nothing is out of range either way): under the bounds-checking build the last chunk's items are refused -- status
    TRI_INV_ERR_DEBUG_CHECK, their rows unwritten, everything else right -- and under the ordinary build nothing happens."""
    sys.path.insert(0, ROOT)
    from paper_2605_21325_b200 import build as lib_build
    for lib, want in ((lib_build.build(debug=True), 6), (lib_build.build(), 0)):
        r = subprocess.run([sys.executable, "-c", CHILD, str(want)], cwd=ROOT, env=dict(os.environ, TRI_INV_LIB=lib),
                           capture_output=True, text=True, timeout=600)
        assert r.returncode == 0 and "ok" in r.stdout, (lib, (r.stdout + r.stderr)[-2000:])
