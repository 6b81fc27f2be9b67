"""Failure handling and shared state of the tensor-core kernels, on the GPU, without faulting or hanging it.

* A bounded device-side wait that runs out: the kernel must return, raise the status word once, leave the work
  counters at zero, and the next ordinary call must be bit-exact.  The wait is made to run out by leaving out the
  product it waits for (tri_inv_selftest_wait_timeout) with a limit of microseconds; every wait stays bounded.
* Work-counter pairs are private to a launch: a captured graph replayed on one stream while more plain launches
  than there are pairs run on another stream must give every row right (compared with the fp64 oracle).
"""
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


def nan_outs(dev, inp):
    return (torch.full((inp.B, inp.T, inp.H, inp.C), float("nan"), dtype=torch.float32, device="cuda"),
            torch.full_like(dev["K"], float("nan")), torch.full_like(dev["V"], float("nan")))


@pytest.mark.parametrize("C", [64, 128])
def test_bounded_wait_gives_up_and_the_library_recovers(bnd, C):
    inp = wl.make("timeout", 2, 16 * C, 8, 128, 128, C, wl.BF16, seed=611)      # 256 matrices
    dev = bnd.to_device(inp)
    ref = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], C)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    out = nan_outs(dev, inp)
    idle = bnd.selftest_wait_timeout(dev["K"], dev["V"], dev["beta"], dev["g"], C, wait_limit_ns=20_000, out=out)
    assert idle, "a work-counter pair was left non-zero"
    assert bnd.last_device_status() == bnd.ERR_DEVICE_TIMEOUT     # raised ...
    assert bnd.last_device_status() == 0                          # ... and cleared by the read
    # every matrix but the one whose product was left out (thread block 0's first: chunk 0, head 0) is right
    for r, o in zip(ref, out):
        r2, o2 = r.clone(), o.clone()
        r2[0, :C, 0] = 0
        o2[0, :C, 0] = 0
        assert torch.equal(r2, o2)
    # the next ordinary call on the same stream is bit-exact
    again = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], C, out=nan_outs(dev, inp))
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    for r, o in zip(ref, again):
        assert torch.equal(r, o)


def test_graph_replays_overlapping_many_plain_launches(bnd):
    a = wl.make("graph_side", 2, 16 * 64, 16, 128, 128, 64, wl.BF16, seed=621)    # 512 matrices: several items per CTA
    b = wl.make("plain_side", 2, 16 * 64, 16, 128, 128, 64, wl.BF16, seed=622)
    da, db = bnd.to_device(a), bnd.to_device(b)
    oa, ob = nan_outs(da, a), nan_outs(db, b)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    bnd.fused(da["K"], da["V"], da["beta"], da["g"], 64, out=oa, stream=s1)      # per-device set-up outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s1):
        with torch.cuda.graph(graph, stream=s1):
            bnd.fused(da["K"], da["V"], da["beta"], da["g"], 64, out=oa, stream=s1)
    for t in oa:
        t.fill_(float("nan"))
    torch.cuda.synchronize()
    for rep in range(8):
        with torch.cuda.stream(s1):
            graph.replay()
        for _ in range(20):                                                       # 160 plain launches in all, unsynchronised
            bnd.fused(db["K"], db["V"], db["beta"], db["g"], 64, out=ob, stream=s2)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    for inp, out in ((a, oa), (b, ob)):
        A_ref = oracle.build_A(inp.K, inp.beta, inp.g, inp.C)
        W_ref, U_ref = oracle.wy(A_ref, inp.K, inp.V, inp.beta, inp.C)
        for o, r, tol in zip(out, (A_ref, W_ref, U_ref), (2e-3, 1e-2, 1e-2)):
            x = bnd.to_numpy_f64(o)
            assert not np.isnan(x).any(), "a row was not written: two launches shared a work counter"
            assert np.abs(x - r).max() <= tol * np.abs(r).max()


@pytest.mark.parametrize("B,H", [(1, 2), (4, 16)], ids=["narrow_slices", "wide_slices"])
def test_scan_waits_that_run_out(bnd, B, H):
    """The chunk-scan kernel's ten warps wait for one another through barriers only; with one product of the first thread
    block left out (tri_inv_selftest_scan_wait_timeout, limit 100 us) every one of that block's waits must give up in turn,
    the kernel must return with the status word raised once, the other blocks' output must be untouched by it, and the
    next ordinary call must give the bits of the call before."""
    inp = wl.make("scan_stall", B, 6 * 64, H, 128, 128, 64, wl.BF16, seed=631 + H)
    dev = bnd.to_device(inp)
    Q = bnd.kv_to_torch(wl.queries(inp, seed=632))
    _, W, U = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], 64, method=bnd.W_DECAY, want_A=False)
    ref, _ = bnd.chunk_scan(Q, dev["K"], W, U, dev["g"], 64, scale=1.0, want_state=False)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    O = torch.full_like(dev["V"], float("nan"))
    bnd.selftest_scan_wait_timeout(Q, dev["K"], W, U, dev["g"], 64, wait_limit_ns=100_000, out=O)
    assert bnd.last_device_status() == bnd.ERR_DEVICE_TIMEOUT     # raised ...
    assert bnd.last_device_status() == 0                          # ... and cleared by the read
    # the stalled block is (sequence 0, head 0, first slice of value columns: 32 or 64 wide); its first chunk was written
    # before the product was left out
    width = 32 if B * H * 4 <= torch.cuda.get_device_properties(0).multi_processor_count else 64
    r2, o2 = ref.clone(), O.clone()
    assert torch.equal(o2[0, :64, 0, :width].view(torch.int16), r2[0, :64, 0, :width].view(torch.int16))
    r2[0, 64:, 0, :width] = 0
    o2[0, 64:, 0, :width] = 0
    assert torch.equal(r2.view(torch.int16), o2.view(torch.int16))
    again, _ = bnd.chunk_scan(Q, dev["K"], W, U, dev["g"], 64, scale=1.0, want_state=False)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    assert torch.equal(again.view(torch.int16), ref.view(torch.int16))


@pytest.mark.parametrize("C,with_wy", [(64, True), (64, False), (128, True)], ids=["C64_one_kernel", "C64_build", "C128_two_launches"])
def test_per_channel_waits_that_run_out(bnd, C, with_wy):
    """The per-channel kernels' give-up path (tri_inv_selftest_kda_wait_timeout, limit 50 us): the first thread block leaves out
    the Gram product of its first matrix, its waits run out, it raises the status word, drains what it has in flight, frees
    its tensor memory and returns.  256 matrices, fewer than resident thread blocks, so every other matrix must come out
    bit for bit as in an ordinary call; the status word reads DEVICE_TIMEOUT once; the next ordinary call is exact."""
    inp = wl.make("kda_timeout", 2, 16 * C, 8, 128, 128, C, wl.BF16, seed=612)
    dev = bnd.to_device(inp)
    Gd = torch.from_numpy(wl.per_channel_gate(inp, seed=613)).cuda()

    def call(selftest):
        A = torch.full((inp.B, inp.T, inp.H, C), float("nan"), dtype=torch.float32, device="cuda")
        W, U = (torch.full_like(dev["K"], float("nan")), torch.full_like(dev["V"], float("nan"))) if with_wy else (None, None)
        if selftest:
            bnd.selftest_kda_wait_timeout(dev["K"], dev["V"] if with_wy else None, Gd, dev["beta"], C, wait_limit_ns=50_000, out=(A, W, U))
        elif with_wy:
            bnd.fused_kda(dev["K"], dev["V"], Gd, dev["beta"], C, out=(A, W, U))
        else:
            bnd.build_kda(dev["K"], Gd, dev["beta"], C, out=A)
        torch.cuda.synchronize()
        return [t for t in (A, W, U) if t is not None]

    ref = call(False)
    assert bnd.last_device_status() == 0
    out = call(True)
    assert bnd.last_device_status() == bnd.ERR_DEVICE_TIMEOUT     # raised ...
    assert bnd.last_device_status() == 0                          # ... and cleared by the read
    for r, o in zip(ref, out):
        r2, o2 = r.clone(), o.clone()
        r2[0, :C, 0] = 0
        o2[0, :C, 0] = 0
        assert torch.equal(r2.view(torch.int32 if r.dtype == torch.float32 else torch.int16),
                           o2.view(torch.int32 if o.dtype == torch.float32 else torch.int16))
    again = call(False)
    assert bnd.last_device_status() == 0
    for r, o in zip(ref, again):
        assert torch.equal(r.view(torch.int32 if r.dtype == torch.float32 else torch.int16),
                           o.view(torch.int32 if o.dtype == torch.float32 else torch.int16))
