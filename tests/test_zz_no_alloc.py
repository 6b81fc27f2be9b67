"""The allocation-free packed entry point gives what the ordinary one gives.

tri_inv_fused_packed_static exists for callers that cannot allocate device memory at call time;
its chunk table lives in a fixed array inside the library.  Two calls in a row on different packed
batches (the second smaller, so stale entries of the first stay behind it in the array) must each
reproduce tri_inv_fused on the same inputs.  This file is named to be collected last."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2605_21325_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bnd():
    import __graft_entry__ as entry
    entry.build()
    from paper_2605_21325_b200 import binding
    torch.cuda.set_device(0)
    return binding


def packed_case(n_seqs, seed):
    rng = np.random.default_rng(seed)
    cu = wl.ragged_lengths(n_seqs, 700, rng)
    return wl.make("packed", 1, int(cu[-1]), 4, 128, 128, 64, wl.BF16, seed, kind="gdn", cu_seqlens=cu, rng=rng)


def test_static_entry_matches_allocating_entry_twice_in_a_row(bnd):
    for n_seqs, seed in ((9, 301), (4, 302)):
        inp = packed_case(n_seqs, seed)
        dev = bnd.to_device(inp)
        ref = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], inp.C, cu_seqlens=inp.cu_seqlens)
        out = (torch.full_like(ref[0], float("nan")), torch.full_like(ref[1], float("nan")), torch.full_like(ref[2], float("nan")))
        got = bnd.fused_packed_static(dev["K"], dev["V"], dev["beta"], dev["g"], inp.C, inp.cu_seqlens, out=out)
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        for r, o in zip(ref, got):
            r32, o32 = r.float(), o.float()
            assert not torch.isnan(o32).any()
            # same kernel, same inputs: identical; the parity tolerances are the formal bar
            assert (r32 - o32).abs().max().item() <= 2e-3 * r32.abs().max().item()
            assert torch.equal(r, o)
        # and against the fp64 oracle, with the tolerances of the parity tests (A 2e-3, W and U 1e-2)
        A_ref = oracle.build_A(inp.K, inp.beta, inp.g, inp.C, cu_seqlens=inp.cu_seqlens)
        W_ref, U_ref = oracle.wy(A_ref, inp.K, inp.V, inp.beta, inp.C, cu_seqlens=inp.cu_seqlens)
        for o, r, tol in zip(got, (A_ref, W_ref, U_ref), (2e-3, 1e-2, 1e-2)):
            assert np.abs(bnd.to_numpy_f64(o) - r).max() <= tol * np.abs(r).max()


def test_static_entry_allocates_no_device_memory(bnd):
    """The property the entry point exists for: across a call (after the first one on the device) the free
    device memory the driver reports does not move, and torch's allocator is not touched either."""
    inp = packed_case(5, 303)
    dev = bnd.to_device(inp)
    out = (torch.empty((1, inp.T, inp.H, inp.C), dtype=torch.float32, device="cuda"), torch.empty_like(dev["K"]),
           torch.empty_like(dev["V"]))
    bnd.fused_packed_static(dev["K"], dev["V"], dev["beta"], dev["g"], inp.C, inp.cu_seqlens, out=out)   # first call: set-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    reserved0, allocs0 = torch.cuda.memory_reserved(), torch.cuda.memory_stats().get("allocation.all.allocated", 0)
    for _ in range(3):
        bnd.fused_packed_static(dev["K"], dev["V"], dev["beta"], dev["g"], inp.C, inp.cu_seqlens, out=out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.cuda.memory_reserved() == reserved0
    assert torch.cuda.memory_stats().get("allocation.all.allocated", 0) == allocs0
    assert bnd.last_device_status() == 0


def test_static_entry_rejects_what_it_cannot_hold(bnd):
    L = bnd.load()
    dummy = torch.zeros(64, device="cuda")
    p = bnd._p(dummy)
    # more chunks of tokens than the fixed table holds: clear error, nothing launched
    n = bnd.STATIC_MAX_CHUNKS + 1
    cu = np.arange(0, n + 1, dtype=np.int32)            # n sequences of one token = n chunks
    desc, keep = bnd.make_desc(1, n, 1, 128, 128, 64, bnd.BF16, cu)
    before = bnd.launch_count()
    rc = L.tri_inv_fused_packed_static(p, p, p, p, p, p, p, ctypes.byref(desc), 0, None)
    assert rc == bnd.ERR_TOO_LARGE and "static" in bnd.status_string(rc)
    # dense descriptors are refused: they never needed scratch
    desc, _ = bnd.make_desc(1, 128, 1, 128, 128, 64, bnd.BF16)
    assert L.tri_inv_fused_packed_static(p, p, p, p, p, p, p, ctypes.byref(desc), 0, None) == bnd.ERR_INVALID_ARG
    assert bnd.launch_count() == before
