"""tri_inv_fused_host: host buffers in, host buffers out, device workspace of the caller's.  Results must be those of
tri_inv_fused on the same inputs (bit for bit) and within tolerance of the oracle; dense (sliced), ragged last chunk and
packed batches (one slice); pinned and pageable host memory; a workspace that is too small is refused."""
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


def test_host_call_matches_device_call_and_oracle(bnd):
    rng = np.random.default_rng(3)
    cu = wl.ragged_lengths(6, 300, rng)
    cases = [(wl.make("h_dense", 3, 24 * 64, 4, 128, 128, 64, wl.BF16, seed=701), True),
             (wl.make("h_tail", 2, 5 * 64 + 17, 2, 128, 128, 64, wl.BF16, seed=702), True),
             (wl.make("h_packed", 1, int(cu[-1]), 2, 128, 128, 64, wl.BF16, seed=703, cu_seqlens=cu, rng=rng), False),
             (wl.make("h_f32", 2, 4 * 64, 2, 64, 64, 64, wl.F32, seed=704), True)]
    for inp, pin in cases:
        dev = bnd.to_device(inp)
        ref = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], inp.C, cu_seqlens=inp.cu_seqlens)
        hK, hV = bnd.kv_to_torch(inp.K, "cpu", pin=pin), bnd.kv_to_torch(inp.V, "cpu", pin=pin)
        hb, hg = torch.from_numpy(inp.beta), torch.from_numpy(inp.g)
        outs = [torch.full(ref[0].shape, float("nan"), dtype=torch.float32), torch.full(ref[1].shape, float("nan"), dtype=ref[1].dtype),
                torch.full(ref[2].shape, float("nan"), dtype=ref[2].dtype)]
        if pin:
            hb, hg = hb.pin_memory(), hg.pin_memory()
            outs = [t.pin_memory() for t in outs]
        n = bnd.fused_host_workspace_bytes(inp.B, inp.T, inp.H, inp.d_k, inp.d_v, inp.C, bnd._dtype_code(dev["K"]), inp.cu_seqlens)
        ws = torch.empty(n, dtype=torch.uint8, device="cuda")
        bnd.fused_host(hK, hV, hb, hg, inp.C, outs[0], outs[1], outs[2], ws, cu_seqlens=inp.cu_seqlens)
        torch.cuda.current_stream().synchronize()        # the caller's stream covers the whole call
        assert bnd.last_device_status() == 0
        mask = torch.zeros(inp.B * inp.T, dtype=torch.bool)
        for t0, r in inp.chunk_list():
            mask[t0:t0 + r] = True
        for r, o in zip(ref, outs):
            rr, oo = r.cpu().reshape(inp.B * inp.T, -1)[mask], o.reshape(inp.B * inp.T, -1)[mask]
            assert torch.equal(rr, oo)
        A_ref = oracle.build_A(inp.K, inp.beta, inp.g, inp.C, cu_seqlens=inp.cu_seqlens)
        a = outs[0].numpy().astype(np.float64).reshape(inp.B * inp.T, -1)[mask.numpy()]
        assert np.abs(a - A_ref.reshape(inp.B * inp.T, -1)[mask.numpy()]).max() <= (2e-3 if inp.kv_dtype == wl.BF16 else 1e-5)
        # too small a workspace: refused, nothing enqueued
        before = bnd.launch_count()
        with pytest.raises(bnd.TriInvError) as e:
            bnd.fused_host(hK, hV, hb, hg, inp.C, outs[0], outs[1], outs[2], ws[:n - 256], cu_seqlens=inp.cu_seqlens)
        assert e.value.status == bnd.ERR_INVALID_ARG and bnd.launch_count() == before
