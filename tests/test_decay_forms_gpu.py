"""GPU parity for the other decay forms of Table 1: the Comba row (decay matrix from j to i-1, TRI_INV_GATE_SHIFTED) and the
KDA row through the whole layer (per-channel decay: tri_inv_fused_kda, tri_inv_chunk_scan_kda), against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_21325_b200 import workloads as wl
from parity_util import max_ratio, max_residual, structure_errors

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bnd():
    import __graft_entry__ as entry
    entry.build()
    from paper_2605_21325_b200 import binding
    torch.cuda.set_device(0)
    return binding


def cases(C, dtype, d):
    rng = np.random.default_rng(500 + C + d)
    cu = wl.ragged_lengths(5, 4 * C, rng)
    return [wl.make("dense", 2, 5 * C, 3, d, d, C, dtype, seed=1200 + C + d),
            wl.make("packed", 1, int(cu[-1]), 2, d, d, C, dtype, seed=1300 + C + d, cu_seqlens=cu, rng=rng)]


@pytest.mark.parametrize("C,dtype,d", [(64, wl.BF16, 128), (128, wl.BF16, 128), (64, wl.F32, 64), (32, wl.BF16, 64)])
def test_shifted_gate_build_and_wy(bnd, C, dtype, d):
    """N_ij = beta_i (k_i . k_j) exp(g_{i-1} - g_j): A for every scheme, and the decay-weighted W (row i weighted by
    exp(g_{i-1})) and U, on the tensor-core kernel (bf16, d = 128) and the CUDA-core kernel (other shapes, fp32)."""
    tol_a, tol_r, tol_w = (2e-3, 5e-3, 1e-2) if dtype == wl.BF16 else (1e-5, 5e-5, 1e-5)
    for inp in cases(C, dtype, d):
        cu = inp.cu_seqlens
        A_ref, N_ref = oracle.build_A_shifted(inp.K, inp.beta, inp.g, C, cu_seqlens=cu, return_N=True)
        gs = oracle.shifted_gate(inp.g, C, cu_seqlens=cu)
        Kd = inp.kv_as_f32("K").astype(np.float64)
        W_ref, _ = oracle.wy(A_ref, Kd * np.exp(gs)[..., None], None, inp.beta, C, cu_seqlens=cu)
        _, U_ref = oracle.wy(A_ref, inp.K, inp.V, inp.beta, C, cu_seqlens=cu)
        dev = bnd.to_device(inp)
        for m in (bnd.BLOCK_RECURSIVE, bnd.BLOCK_RECURSIVE | bnd.LEAF_SERIES, bnd.PRODUCT_SERIES):
            A, W, U = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], C, method=m | bnd.GATE_SHIFTED | bnd.W_DECAY, cu_seqlens=cu)
            torch.cuda.synchronize()
            assert bnd.last_device_status() == 0
            a = A.cpu().numpy()
            assert structure_errors(a, inp) == (0, 0)
            assert max_ratio(a, A_ref) <= tol_a and max_residual(a, N_ref, inp) <= tol_r
            assert max_ratio(bnd.to_numpy_f64(W), W_ref) <= tol_w and max_ratio(bnd.to_numpy_f64(U), U_ref) <= tol_w
        A = bnd.build(dev["K"], dev["beta"], dev["g"], C, method=bnd.GATE_SHIFTED, cu_seqlens=cu)
        torch.cuda.synchronize()
        assert max_ratio(A.cpu().numpy(), A_ref) <= tol_a
        # the flag matters: without it the matrix differs visibly
        A0 = bnd.build(dev["K"], dev["beta"], dev["g"], C, cu_seqlens=cu)
        torch.cuda.synchronize()
        assert max_ratio(A0.cpu().numpy(), A_ref) > 10 * tol_a


def test_comba_layer_two_launches_against_its_recurrence(bnd):
    """Fused call with the shifted gate and the decay-weighted W, then the unchanged chunk scan, against
    S_t = (alpha_t I - beta_t k_t k_t^T) S_{t-1} + beta_t k_t v_t^T token by token."""
    for inp in cases(64, wl.BF16, 128):
        cu = inp.cu_seqlens
        Q = wl.queries(inp, seed=77)
        S0 = wl.initial_state(inp, seed=78)
        dev = bnd.to_device(inp)
        _, W, U = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], 64, method=bnd.GATE_SHIFTED | bnd.W_DECAY, cu_seqlens=cu, want_A=False)
        O, S = bnd.chunk_scan(bnd.kv_to_torch(Q), dev["K"], W, U, dev["g"], 64, scale=0.5, S0=torch.from_numpy(S0).cuda(), cu_seqlens=cu)
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        O_ref, S_ref = oracle.recurrence_ex(Q, inp.K, inp.V, inp.beta, inp.g, 64, read_before_decay=True, scale=0.5, S0=S0, cu_seqlens=cu)
        assert max_ratio(bnd.to_numpy_f64(O), O_ref) <= 2e-2 and max_ratio(bnd.to_numpy_f64(S), S_ref) <= 2e-2


@pytest.mark.parametrize("C,dtype,d", [(64, wl.BF16, 128), (64, wl.F32, 64), (32, wl.BF16, 64), (128, wl.BF16, 128)])
def test_per_channel_decay_through_wy_and_scan(bnd, C, dtype, d):
    """tri_inv_fused_kda (tensor-core route at bf16 / d = 128 / C = 64, CUDA cores elsewhere) against the oracle's A, W, U;
    then tri_inv_chunk_scan_kda on them against the token-by-token recurrence with one decay per key feature."""
    tol_a, tol_r, tol_w, tol_o = (2e-3, 5e-3, 1e-2, 2e-2) if dtype == wl.BF16 else (1e-5, 5e-5, 1e-5, 1e-4)
    for inp in cases(C, dtype, d):
        cu = inp.cu_seqlens
        G = wl.per_channel_gate(inp, seed=61)
        A_ref, N_ref = oracle.build_A_kda(inp.K, G, inp.beta, C, cu_seqlens=cu, return_N=True)
        Kd = inp.kv_as_f32("K").astype(np.float64)
        W_ref, _ = oracle.wy(A_ref, Kd * np.exp(G.astype(np.float64)), None, inp.beta, C, cu_seqlens=cu)
        _, U_ref = oracle.wy(A_ref, inp.K, inp.V, inp.beta, C, cu_seqlens=cu)
        dev = bnd.to_device(inp)
        Gd = torch.from_numpy(G).cuda()
        nan = lambda t: torch.full_like(t, float("nan"))
        out = (torch.full((inp.B, inp.T, inp.H, C), float("nan"), dtype=torch.float32, device="cuda"), nan(dev["K"]), nan(dev["V"]))
        A, W, U = bnd.fused_kda(dev["K"], dev["V"], Gd, dev["beta"], C, cu_seqlens=cu, out=out)
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        a = A.cpu().numpy()
        assert not np.isnan(a).any() and structure_errors(a, inp) == (0, 0)
        assert max_ratio(a, A_ref) <= tol_a and max_residual(a, N_ref, inp) <= tol_r
        w, u = bnd.to_numpy_f64(W), bnd.to_numpy_f64(U)
        assert not np.isnan(w).any() and not np.isnan(u).any()
        assert max_ratio(w, W_ref) <= tol_w and max_ratio(u, U_ref) <= tol_w
        Q = wl.queries(inp, seed=62)
        S0 = wl.initial_state(inp, seed=63)
        O, S = bnd.chunk_scan_kda(bnd.kv_to_torch(Q), dev["K"], W, U, Gd, C, scale=0.5, S0=torch.from_numpy(S0).cuda(), cu_seqlens=cu)
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        O_ref, S_ref = oracle.recurrence_ex(Q, inp.K, inp.V, inp.beta, None, C, G=G, scale=0.5, S0=S0, cu_seqlens=cu)
        assert max_ratio(bnd.to_numpy_f64(O), O_ref) <= tol_o and max_ratio(bnd.to_numpy_f64(S), S_ref) <= tol_o
        # the scan alone, fed the oracle's own W and U (rounded to the storage type), against its definition
        if dtype == wl.F32:
            Wt, Ut = torch.from_numpy(W_ref.astype(np.float32)).cuda(), torch.from_numpy(U_ref.astype(np.float32)).cuda()
            O2, S2 = bnd.chunk_scan_kda(bnd.kv_to_torch(Q), dev["K"], Wt, Ut, Gd, C, scale=0.5, S0=torch.from_numpy(S0).cuda(), cu_seqlens=cu)
            O3, S3 = oracle.chunk_scan_kda(Q, inp.K, W_ref.astype(np.float32), U_ref.astype(np.float32), G, C, scale=0.5, S0=S0, cu_seqlens=cu)
            torch.cuda.synchronize()
            assert max_ratio(bnd.to_numpy_f64(O2), O3) <= 1e-5 and max_ratio(bnd.to_numpy_f64(S2), S3) <= 1e-5


def test_flags_the_per_channel_calls_refuse(bnd):
    import ctypes
    d = torch.zeros(64, device="cuda")
    desc, _ = bnd.make_desc(1, 64, 1, 128, 128, 64, bnd.BF16)
    L = bnd.load()
    p = bnd._p(d)
    assert L.tri_inv_build_kda(p, p, p, p, ctypes.byref(desc), bnd.GATE_SHIFTED, None) == bnd.ERR_UNSUPPORTED
    assert L.tri_inv_fused_kda(p, p, p, p, p, p, p, ctypes.byref(desc), bnd.W_DECAY, None) == bnd.ERR_UNSUPPORTED
    assert L.tri_inv_fused_kda(p, p, p, p, None, p, p, ctypes.byref(desc), 0, None) == bnd.ERR_INVALID_ARG


def test_per_channel_scan_on_the_tensor_cores_full_size_ragged(bnd):
    """tri_inv_chunk_scan_kda at bf16 / d = 128 / C = 64 (operand preparation + the tensor-core scan) on the packed, ragged
    shape of config 5: EVERY token of O and every final state against the token-by-token recurrence with one decay per
    key feature; the same launch twice gives the same bits; and a sequence resumed from a returned state reproduces the
    continuous run bit for bit."""
    inp = wl.config(5)
    cu = inp.cu_seqlens
    G = wl.per_channel_gate(inp, seed=3005)
    Q = wl.queries(inp, seed=64)
    S0 = wl.initial_state(inp, seed=65)
    dev = bnd.to_device(inp)
    Gd, Qd, S0d = torch.from_numpy(G).cuda(), bnd.kv_to_torch(Q), torch.from_numpy(S0).cuda()
    _, W, U = bnd.fused_kda(dev["K"], dev["V"], Gd, dev["beta"], 64, cu_seqlens=cu)
    O = torch.full_like(dev["V"], float("nan"))
    O, S = bnd.chunk_scan_kda(Qd, dev["K"], W, U, Gd, 64, scale=0.25, S0=S0d, cu_seqlens=cu, out=O)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    O_ref, S_ref = oracle.recurrence_ex(Q, inp.K, inp.V, inp.beta, None, 64, G=G, scale=0.25, S0=S0, cu_seqlens=cu)
    o = bnd.to_numpy_f64(O)
    assert not np.isnan(o).any(), "a row of O was not written"
    assert max_ratio(o, O_ref) <= 2e-2 and max_ratio(bnd.to_numpy_f64(S), S_ref) <= 2e-2
    O2, S2 = bnd.chunk_scan_kda(Qd, dev["K"], W, U, Gd, 64, scale=0.25, S0=S0d, cu_seqlens=cu)
    torch.cuda.synchronize()
    assert torch.equal(O2.view(torch.int16), O.view(torch.int16)) and torch.equal(S2, S)


def test_per_channel_scan_resumes_bit_for_bit(bnd):
    """Dense batch cut at a chunk boundary: the second part, started from the first part's returned state, gives the very
    bits of the uncut run (few (sequence, head) pairs: the 32-column instance; many: the 64-column one)."""
    for B, H in ((1, 2), (3, 20)):
        T, cut = 6 * 64 + 23, 4 * 64
        inp = wl.make("resume", B, T, H, 128, 128, 64, wl.BF16, seed=1400 + H)
        G = wl.per_channel_gate(inp, seed=66)
        Q = wl.queries(inp, seed=67)
        dev = bnd.to_device(inp)
        Gd, Qd = torch.from_numpy(G).cuda(), bnd.kv_to_torch(Q)
        _, W, U = bnd.fused_kda(dev["K"], dev["V"], Gd, dev["beta"], 64)
        O, S = bnd.chunk_scan_kda(Qd, dev["K"], W, U, Gd, 64, scale=0.5)
        part = lambda t, a, b: t[:, a:b].contiguous()
        O1, S1 = bnd.chunk_scan_kda(part(Qd, 0, cut), part(dev["K"], 0, cut), part(W, 0, cut), part(U, 0, cut), part(Gd, 0, cut), 64, scale=0.5)
        O2, S2 = bnd.chunk_scan_kda(part(Qd, cut, T), part(dev["K"], cut, T), part(W, cut, T), part(U, cut, T), part(Gd, cut, T), 64, scale=0.5, S0=S1)
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        assert torch.equal(torch.cat([O1, O2], dim=1).view(torch.int16), O.view(torch.int16)) and torch.equal(S2, S)


def test_per_channel_layer_captured_in_a_cuda_graph(bnd):
    """The four launches of the per-channel layer forward (build, WY, operand preparation, scan) and the scan's scratch
    memory (stream-ordered allocation and release) can be captured once and replayed on new inputs in the same buffers."""
    inp = wl.make("kda_graph", 2, 4 * 64, 4, 128, 128, 64, wl.BF16, seed=1500)
    G = wl.per_channel_gate(inp, seed=68)
    Q = wl.queries(inp, seed=69)
    dev = bnd.to_device(inp)
    Gd, Qd = torch.from_numpy(G).cuda(), bnd.kv_to_torch(Q)
    A = torch.empty((2, 4 * 64, 4, 64), dtype=torch.float32, device="cuda")
    W, U, O = torch.empty_like(dev["K"]), torch.empty_like(dev["V"]), torch.empty_like(dev["V"])

    def forward():
        bnd.fused_kda(dev["K"], dev["V"], Gd, dev["beta"], 64, out=(A, W, U))
        bnd.chunk_scan_kda(Qd, dev["K"], W, U, Gd, 64, scale=0.125, out=O, want_state=False)

    forward()                       # first use: per-device set-up happens outside the capture
    torch.cuda.synchronize()
    O_eager = O.clone()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            forward()
    torch.cuda.synchronize()
    O.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    assert torch.equal(O.view(torch.int16), O_eager.view(torch.int16))
    inp2 = wl.make("kda_graph2", 2, 4 * 64, 4, 128, 128, 64, wl.BF16, seed=1501)
    G2 = wl.per_channel_gate(inp2, seed=70)
    dev2 = bnd.to_device(inp2)
    for k in ("K", "V", "beta"):
        dev[k].copy_(dev2[k])
    Gd.copy_(torch.from_numpy(G2).cuda())
    graph.replay()
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    O_ref, _ = oracle.recurrence_ex(Q, inp2.K, inp2.V, inp2.beta, None, 64, G=G2, scale=0.125)
    assert max_ratio(bnd.to_numpy_f64(O), O_ref) <= 2e-2


@pytest.mark.parametrize("C", [64, 128])
def test_per_channel_forms_under_strong_decay(bnd, C):
    """A gate that falls by about one (natural-log unit) per token and channel: G reaches -60 .. -75 at the end of a chunk of
    64 and twice that at 128, so that exp(G_i - G_j) spans the whole fp32 range and exp(-G) alone would overflow.  The
    tensor-core kernels scale rows against a reference row in the middle of the chunk (of each half at C = 128), which keeps
    every factor within exp(+-|G over 32 tokens|): A, W, U must still match the fp64 oracle, and at C = 64 the scan on the
    prepared operands must still match the token-by-token recurrence."""
    inp = wl.make("strong", 2, 3 * C + 11, 3, 128, 128, C, wl.BF16, seed=1600 + C)
    G = wl.per_channel_gate(inp, seed=71, mean=-0.5)
    assert G.min() < (-100.0 if C == 128 else -50.0)
    A_ref, N_ref = oracle.build_A_kda(inp.K, G, inp.beta, C, return_N=True)
    Kd = inp.kv_as_f32("K").astype(np.float64)
    W_ref, _ = oracle.wy(A_ref, Kd * np.exp(G.astype(np.float64)), None, inp.beta, C)
    _, U_ref = oracle.wy(A_ref, inp.K, inp.V, inp.beta, C)
    dev = bnd.to_device(inp)
    Gd = torch.from_numpy(G).cuda()
    A, W, U = bnd.fused_kda(dev["K"], dev["V"], Gd, dev["beta"], C)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    a = A.cpu().numpy()
    assert np.isfinite(a).all() and structure_errors(a, inp) == (0, 0)
    assert max_ratio(a, A_ref) <= 2e-3 and max_residual(a, N_ref, inp) <= 5e-3
    assert max_ratio(bnd.to_numpy_f64(W), W_ref) <= 1e-2 and max_ratio(bnd.to_numpy_f64(U), U_ref) <= 1e-2
    if C == 64:
        Q = wl.queries(inp, seed=72)
        S0 = wl.initial_state(inp, seed=73)
        O, S = bnd.chunk_scan_kda(bnd.kv_to_torch(Q), dev["K"], W, U, Gd, C, scale=0.5, S0=torch.from_numpy(S0).cuda())
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        O_ref, S_ref = oracle.recurrence_ex(Q, inp.K, inp.V, inp.beta, None, C, G=G, scale=0.5, S0=S0)
        o, s_ = bnd.to_numpy_f64(O), bnd.to_numpy_f64(S)
        assert np.isfinite(o).all() and np.isfinite(s_).all()
        assert max_ratio(o, O_ref) <= 2e-2 and max_ratio(s_, S_ref) <= 2e-2
