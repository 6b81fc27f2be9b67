"""C-ABI checks that need no GPU: the library loads, exports what the header declares,
and rejects bad arguments on the host before touching the device."""
import ctypes
import os
import re

import numpy as np
import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    from paper_2605_21325_b200 import binding
    return binding.load(), binding


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names += re.findall(r"\b(tri_inv_[a-z_0-9]+)\s*\(", src)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(lib):
    L, binding = lib
    names = declared_functions()
    assert len(names) >= 7
    for n in names:
        assert hasattr(L, n), "missing export %s" % n
    assert set(binding.EXPORTS) <= set(names)


def test_status_strings(lib):
    L, binding = lib
    assert binding.status_string(0) == "ok"
    assert len({binding.status_string(i) for i in range(5)}) == 5


def test_count_matrices_and_descriptor_validation(lib):
    L, binding = lib
    d, _ = binding.make_desc(4, 4096, 16, 128, 128, 64, binding.BF16)
    assert binding.count_matrices(d) == 4096
    d, _ = binding.make_desc(2, 100, 3, 64, 64, 64, binding.F32)         # partial last chunk
    assert binding.count_matrices(d) == 2 * 2 * 3
    cu = np.array([0, 1, 70, 134, 200], np.int32)
    d, keep = binding.make_desc(1, 200, 2, 64, 64, 64, binding.BF16, cu)
    assert binding.count_matrices(d) == (1 + 2 + 1 + 2) * 2
    for bad in (dict(C=48), dict(d_k=12), dict(H=0), dict(kv_dtype=7), dict(B=0)):
        kw = dict(B=1, T=64, H=1, d_k=64, d_v=64, C=64, kv_dtype=binding.F32)
        kw.update(bad)
        d, _ = binding.make_desc(**kw)
        with pytest.raises(binding.TriInvError) as e:
            binding.count_matrices(d)
        assert e.value.status == binding.ERR_INVALID_ARG
    for cu_bad in ([0, 10, 5, 200], [1, 200], [0, 100]):                 # decreasing, bad start, bad end
        d, keep = binding.make_desc(1, 200, 2, 64, 64, 64, binding.BF16, np.array(cu_bad, np.int32))
        with pytest.raises(binding.TriInvError):
            binding.count_matrices(d)


def test_null_and_misaligned_pointers_rejected_before_any_device_work(lib):
    L, binding = lib
    d, _ = binding.make_desc(1, 64, 1, 64, 64, 64, binding.F32)
    p = ctypes.byref(d)
    ok = ctypes.c_void_p(4096)
    assert L.tri_inv_build(None, ok, ok, ok, p, 0, None) == binding.ERR_INVALID_ARG
    assert L.tri_inv_build(ok, ok, ok, ctypes.c_void_p(4100), p, 0, None) == binding.ERR_INVALID_ARG
    assert L.tri_inv_build(ok, ok, ok, ok, None, 0, None) == binding.ERR_INVALID_ARG
    assert L.tri_inv_build(ok, ok, ok, ok, p, 7, None) == binding.ERR_UNSUPPORTED
    assert L.tri_inv_build(ok, ok, ok, ok, p, binding.PRODUCT_SERIES | binding.LEAF_SERIES, None) == binding.ERR_UNSUPPORTED
    assert L.tri_inv_wy(ok, ok, ok, ok, ok, None, p, None) == binding.ERR_INVALID_ARG   # V without U
    assert L.tri_inv_fused(ok, None, ok, ok, ok, ok, ok, p, 0, None) == binding.ERR_INVALID_ARG
    assert binding.launch_count() == 0 or binding.launch_count() > 0   # callable without a device


def test_newer_entry_points_validate_on_the_host(lib):
    L, binding = lib
    d, _ = binding.make_desc(1, 64, 1, 128, 128, 64, binding.BF16)
    p = ctypes.byref(d)
    ok = ctypes.c_void_p(4096)
    odd = ctypes.c_void_p(4100)
    # per-channel decay build
    assert L.tri_inv_build_kda(ok, None, ok, ok, p, 0, None) == binding.ERR_INVALID_ARG
    assert L.tri_inv_build_kda(ok, odd, ok, ok, p, 0, None) == binding.ERR_INVALID_ARG
    assert L.tri_inv_build_kda(ok, ok, ok, ok, p, binding.W_DECAY, None) == binding.ERR_UNSUPPORTED   # no W to weight
    # decay-weighted W is a fused-call option only
    assert L.tri_inv_build(ok, ok, ok, ok, p, binding.W_DECAY, None) == binding.ERR_UNSUPPORTED
    # chunk scan: Q, K, W, U, g, O are required; S0 and S_out are optional but must be aligned when given
    scale = ctypes.c_float(1.0)
    assert L.tri_inv_chunk_scan(None, ok, ok, ok, ok, None, ok, None, scale, p, None) == binding.ERR_INVALID_ARG
    assert L.tri_inv_chunk_scan(ok, ok, ok, ok, ok, None, None, None, scale, p, None) == binding.ERR_INVALID_ARG
    assert L.tri_inv_chunk_scan(ok, ok, ok, ok, ok, odd, ok, None, scale, p, None) == binding.ERR_INVALID_ARG
    assert L.tri_inv_chunk_scan(ok, ok, ok, ok, ok, None, ok, None, scale, None, None) == binding.ERR_INVALID_ARG
    wide, _ = binding.make_desc(1, 64, 1, 512, 64, 64, binding.F32)      # d_k beyond the CUDA-core scan's state slice
    assert L.tri_inv_chunk_scan(ok, ok, ok, ok, ok, None, ok, None, scale, ctypes.byref(wide), None) == binding.ERR_UNSUPPORTED
