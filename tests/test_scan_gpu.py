"""GPU parity of the chunk scan (consumer of W and U) and of the two-launch layer forward.

Tolerances (every product operand is bf16 -- 2^-9 relative each -- with fp32 accumulation, and the state forgets
with the gate's decay, so a chunk's rounding does not pile up; a few times 2^-9 of max|O| at the tail):
  chunk scan alone, given the oracle's W and U rounded to bf16:
      max|O_gpu - O_ref| / max|O_ref| <= 1e-2,   max|S_gpu - S_ref| / max|S_ref| <= 1e-2
  whole layer (fused kernel with decay-weighted W, then scan) against the token-by-token recurrence: <= 2e-2.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_21325_b200 import workloads as wl
from parity_util import max_ratio

pytestmark = pytest.mark.gpu

TOL_SCAN, TOL_LAYER = 1e-2, 2e-2


@pytest.fixture(scope="module")
def bnd():
    import __graft_entry__ as entry
    entry.build()
    from paper_2605_21325_b200 import binding
    torch.cuda.set_device(0)
    return binding


def to_bf16_bits(x64):
    return wl._store(x64.astype(np.float32), wl.BF16)


def exact_wu(inp, cu_seqlens):
    """The oracle's decay-weighted W and U, rounded once to bf16 storage."""
    A = oracle.build_A(inp.K, inp.beta, inp.g, inp.C, cu_seqlens=cu_seqlens)
    Kd = oracle._widen(inp.K) * np.exp(inp.g.astype(np.float64))[..., None]
    W, _ = oracle.wy(A, Kd, None, inp.beta, inp.C, cu_seqlens=cu_seqlens)
    _, U = oracle.wy(A, inp.K, inp.V, inp.beta, inp.C, cu_seqlens=cu_seqlens)
    return to_bf16_bits(W), to_bf16_bits(U)


CASES = [
    ("dense", 2, 5 * 64, 3, None, False),
    ("dense_partial_s0", 1, 3 * 64 + 17, 2, None, True),
    ("ragged_s0", 1, 0, 2, np.array([0, 64, 65, 65, 300, 531], np.int32), True),
    ("many_heads", 5, 2 * 64, 64, None, True),   # 640 CTAs: several per SM in turn
    # few (sequence, head) pairs run as four CTAs of 32 value columns per pair, more as two of 64: both sides of the switch
    ("pairs_36", 2, 3 * 64 + 9, 18, None, True),
    ("pairs_40", 2, 3 * 64 + 9, 20, None, True),
]


@pytest.mark.parametrize("name,B,T,H,cu,with_s0", CASES, ids=[c[0] for c in CASES])
def test_chunk_scan_matches_its_definition(bnd, name, B, T, H, cu, with_s0):
    if cu is not None:
        T = int(cu[-1])
    inp = wl.make(name, B, T, H, 128, 128, 64, wl.BF16, seed=300 + H, cu_seqlens=cu)
    Q = wl.queries(inp, seed=301)
    S0 = wl.initial_state(inp, seed=302) if with_s0 else None
    Wb, Ub = exact_wu(inp, cu)
    scale = 128 ** -0.5
    O_ref, S_ref = oracle.chunk_scan(Q, inp.K, Wb, Ub, inp.g, 64, scale=scale, S0=S0, cu_seqlens=cu)
    dev = bnd.to_device(inp)
    Qd, Wd, Ud = (bnd.kv_to_torch(x) for x in (Q, Wb, Ub))
    S0d = None if S0 is None else torch.from_numpy(S0).cuda()
    O = torch.full((B, T, H, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    O, S = bnd.chunk_scan(Qd, dev["K"], Wd, Ud, dev["g"], 64, scale=scale, S0=S0d, cu_seqlens=cu, out=O)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    o, s = bnd.to_numpy_f64(O), bnd.to_numpy_f64(S)
    assert not np.isnan(o).any(), "a row of O was not written"
    assert max_ratio(o, O_ref) <= TOL_SCAN
    assert max_ratio(s, S_ref) <= TOL_SCAN
    # the same inputs through the recurrence itself: the scan is the layer
    O_rec, S_rec = oracle.gdn_recurrence(Q, inp.K, inp.V, inp.beta, inp.g, 64, scale=scale, S0=S0, cu_seqlens=cu)
    assert max_ratio(o, O_rec) <= TOL_LAYER and max_ratio(s, S_rec) <= TOL_LAYER


def test_layer_forward_two_launches_against_the_recurrence(bnd):
    cu = np.array([0, 200, 264, 777], np.int32)
    for cu_seqlens, B, T in ((None, 2, 6 * 64), (cu, 1, 777)):
        inp = wl.make("layer", B, T, 4, 128, 128, 64, wl.BF16, seed=310, cu_seqlens=cu_seqlens)
        Q = wl.queries(inp, seed=311)
        S0 = wl.initial_state(inp, seed=312)
        O_ref, S_ref = oracle.gdn_recurrence(Q, inp.K, inp.V, inp.beta, inp.g, 64, scale=0.125, S0=S0, cu_seqlens=cu_seqlens)
        dev = bnd.to_device(inp)
        O, S = bnd.gdn_forward(bnd.kv_to_torch(Q), dev["K"], dev["V"], dev["beta"], dev["g"], 64, scale=0.125,
                               S0=torch.from_numpy(S0).cuda(), cu_seqlens=cu_seqlens)
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        assert max_ratio(bnd.to_numpy_f64(O), O_ref) <= TOL_LAYER
        assert max_ratio(bnd.to_numpy_f64(S), S_ref) <= TOL_LAYER


def test_chunk_scan_edge_cases(bnd):
    # an empty sequence keeps its initial state; unsupported shapes are refused, not approximated
    cu = np.array([0, 0, 70], np.int32)
    inp = wl.make("edge", 1, 70, 1, 128, 128, 64, wl.BF16, seed=320, cu_seqlens=cu)
    Q = wl.queries(inp, seed=321)
    S0 = wl.initial_state(inp, seed=322)
    Wb, Ub = exact_wu(inp, cu)
    dev = bnd.to_device(inp)
    O, S = bnd.chunk_scan(bnd.kv_to_torch(Q), dev["K"], bnd.kv_to_torch(Wb), bnd.kv_to_torch(Ub), dev["g"], 64,
                          S0=torch.from_numpy(S0).cuda(), cu_seqlens=cu)
    torch.cuda.synchronize()
    assert np.array_equal(S[0].cpu().numpy(), S0[0])
    _, S_ref = oracle.chunk_scan(Q, inp.K, Wb, Ub, inp.g, 64, S0=S0, cu_seqlens=cu)
    assert max_ratio(bnd.to_numpy_f64(S), S_ref) <= TOL_SCAN


SIMT_CASES = [
    ("cfg1_shape_fp32", 1, 256, 2, 64, 64, 64, wl.F32, None),
    ("fp32_c128_partial", 2, 300, 2, 32, 96, 128, wl.F32, None),
    ("fp32_c16_ragged", 1, 0, 3, 16, 40, 16, wl.F32, np.array([0, 5, 5, 37, 100], np.int32)),
    ("bf16_d64_c32", 2, 100, 2, 64, 64, 32, wl.BF16, None),
]


@pytest.mark.parametrize("name,B,T,H,d_k,d_v,C,dtype,cu", SIMT_CASES, ids=[c[0] for c in SIMT_CASES])
def test_chunk_scan_cuda_core_kernel_other_shapes(bnd, name, B, T, H, d_k, d_v, C, dtype, cu):
    """fp32 storage and shapes outside the tensor-core kernel: fp32 arithmetic throughout, so the scan is held to
    1e-5 of max|O| against its fp64 definition (bf16 storage: the output's own rounding, 2^-8)."""
    if cu is not None:
        T = int(cu[-1])
    inp = wl.make(name, B, T, H, d_k, d_v, C, dtype, seed=330 + C, cu_seqlens=cu)
    Q = wl.queries(inp, seed=331)
    S0 = wl.initial_state(inp, seed=332)
    A = oracle.build_A(inp.K, inp.beta, inp.g, C, cu_seqlens=cu)
    Kg = oracle._widen(inp.K) * np.exp(inp.g.astype(np.float64))[..., None]
    W64, _ = oracle.wy(A, Kg, None, inp.beta, C, cu_seqlens=cu)
    _, U64 = oracle.wy(A, inp.K, inp.V, inp.beta, C, cu_seqlens=cu)
    Ws, Us = wl._store(W64.astype(np.float32), dtype), wl._store(U64.astype(np.float32), dtype)
    O_ref, S_ref = oracle.chunk_scan(Q, inp.K, Ws, Us, inp.g, C, scale=0.5, S0=S0, cu_seqlens=cu)
    dev = bnd.to_device(inp)
    O = torch.full((B, T, H, d_v), float("nan"), dtype=dev["V"].dtype, device="cuda")
    O, S = bnd.chunk_scan(bnd.kv_to_torch(Q), dev["K"], bnd.kv_to_torch(Ws), bnd.kv_to_torch(Us), dev["g"], C, scale=0.5,
                          S0=torch.from_numpy(S0).cuda(), cu_seqlens=cu, out=O)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    o = bnd.to_numpy_f64(O)
    assert not np.isnan(o).any()
    tol = 1e-5 if dtype == wl.F32 else 2.0 ** -8
    assert max_ratio(o, O_ref) <= tol
    assert max_ratio(bnd.to_numpy_f64(S), S_ref) <= 1e-5
    if dtype == wl.F32:   # and the whole layer in fp32 through the CUDA-core kernels against the recurrence
        O2, S2 = bnd.gdn_forward(bnd.kv_to_torch(Q), dev["K"], dev["V"], dev["beta"], dev["g"], C, scale=0.5,
                                 S0=torch.from_numpy(S0).cuda(), cu_seqlens=cu)
        torch.cuda.synchronize()
        O_rec, S_rec = oracle.gdn_recurrence(Q, inp.K, inp.V, inp.beta, inp.g, C, scale=0.5, S0=S0, cu_seqlens=cu)
        assert max_ratio(bnd.to_numpy_f64(O2), O_rec) <= 1e-5 and max_ratio(bnd.to_numpy_f64(S2), S_rec) <= 1e-5


# ---------------------------------------------------------------- full sizes, in the launch configuration bench.py times

def test_layer_full_size_config2_sampled_and_restart(bnd):
    inp = wl.config(2)
    Q = wl.queries(inp, seed=4002)
    dev = bnd.to_device(inp)
    Qd = bnd.kv_to_torch(Q)
    scale = 128 ** -0.5
    O, S = bnd.gdn_forward(Qd, dev["K"], dev["V"], dev["beta"], dev["g"], 64, scale=scale)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    assert not bool(torch.isnan(O.float()).any())
    # (a) the first 8 chunks of every sequence and head against the token-by-token recurrence
    Ts = 512
    O_ref, _ = oracle.gdn_recurrence(Q[:, :Ts], inp.K[:, :Ts], inp.V[:, :Ts], inp.beta[:, :Ts], inp.g[:, :Ts], 64, scale=scale)
    assert max_ratio(bnd.to_numpy_f64(O[:, :Ts]), O_ref) <= TOL_LAYER
    # (b) at any size: stopping after half the chunks and resuming from the returned state reproduces the
    # second half of the outputs and the final state bit for bit (same arithmetic, same order)
    half = inp.T // 2
    first = [x[:, :half].contiguous() for x in (Qd, dev["K"], dev["V"], dev["beta"], dev["g"])]
    second = [x[:, half:].contiguous() for x in (Qd, dev["K"], dev["V"], dev["beta"], dev["g"])]
    O1, S1 = bnd.gdn_forward(*first, 64, scale=scale)
    O2, S2 = bnd.gdn_forward(*second, 64, scale=scale, S0=S1)
    torch.cuda.synchronize()
    assert torch.equal(O1, O[:, :half]) and torch.equal(O2, O[:, half:]) and torch.equal(S2, S)
    # (c) the last chunk of one sequence and head from the carried state, in fp64: one step of the chunk form
    t0 = inp.T - 64
    Wd, Ud = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], 64, method=bnd.W_DECAY, want_A=False)[1:]
    _, S_prev = bnd.chunk_scan(Qd[:, :t0].contiguous(), dev["K"][:, :t0].contiguous(), Wd[:, :t0].contiguous(),
                               Ud[:, :t0].contiguous(), dev["g"][:, :t0].contiguous(), 64, scale=scale)
    torch.cuda.synchronize()
    sl = slice(t0, inp.T)
    O_last, S_last = oracle.chunk_scan(Q[:, sl], inp.K[:, sl], wl._store(Wd[:, sl].float().cpu().numpy(), wl.BF16),
                                       wl._store(Ud[:, sl].float().cpu().numpy(), wl.BF16), inp.g[:, sl], 64, scale=scale,
                                       S0=S_prev.cpu().numpy())
    assert max_ratio(bnd.to_numpy_f64(O[:, sl]), O_last) <= TOL_SCAN
    assert max_ratio(bnd.to_numpy_f64(S), S_last) <= TOL_SCAN


def test_layer_full_size_config5_ragged(bnd):
    inp = wl.config(5)
    Q = wl.queries(inp, seed=4005)
    dev = bnd.to_device(inp)
    O, S = bnd.gdn_forward(bnd.kv_to_torch(Q), dev["K"], dev["V"], dev["beta"], dev["g"], 64, scale=128 ** -0.5,
                           cu_seqlens=inp.cu_seqlens)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    O_ref, S_ref = oracle.gdn_recurrence(Q, inp.K, inp.V, inp.beta, inp.g, 64, scale=128 ** -0.5, cu_seqlens=inp.cu_seqlens)
    assert max_ratio(bnd.to_numpy_f64(O), O_ref) <= TOL_LAYER
    assert max_ratio(bnd.to_numpy_f64(S), S_ref) <= TOL_LAYER


def test_layer_forward_captured_in_a_cuda_graph(bnd):
    """Dense calls allocate nothing after their first use on a device: the two launches of the layer forward can be
    captured once and replayed on new inputs written into the same buffers."""
    inp = wl.make("graph", 2, 4 * 64, 4, 128, 128, 64, wl.BF16, seed=340)
    Q = wl.queries(inp, seed=341)
    dev = bnd.to_device(inp)
    Qd = bnd.kv_to_torch(Q)
    W, U, O = torch.empty_like(dev["K"]), torch.empty_like(dev["V"]), torch.empty_like(dev["V"])
    S = torch.empty((2, 4, 128, 128), dtype=torch.float32, device="cuda")

    def forward():
        bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], 64, method=bnd.W_DECAY, out=(None, W, U))
        bnd.chunk_scan(Qd, dev["K"], W, U, dev["g"], 64, scale=0.125, out=O, state_out=S)

    forward()                       # first use: per-device set-up happens outside the capture
    torch.cuda.synchronize()
    O_eager, S_eager = O.clone(), S.clone()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            forward()
    torch.cuda.synchronize()
    O.zero_(); S.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    assert torch.equal(O, O_eager) and torch.equal(S, S_eager)
    # new inputs in the same buffers: the replay computes the new result
    inp2 = wl.make("graph2", 2, 4 * 64, 4, 128, 128, 64, wl.BF16, seed=342)
    dev2 = bnd.to_device(inp2)
    for k in ("K", "V", "beta", "g"):
        dev[k].copy_(dev2[k])
    graph.replay()
    torch.cuda.synchronize()
    O_ref, S_ref = oracle.gdn_recurrence(Q, inp2.K, inp2.V, inp2.beta, inp2.g, 64, scale=0.125)
    assert max_ratio(bnd.to_numpy_f64(O), O_ref) <= TOL_LAYER and max_ratio(bnd.to_numpy_f64(S), S_ref) <= TOL_LAYER


def test_chunk_scan_with_a_gate_that_is_not_monotone(bnd):
    """g is taken as given: nothing in the scan assumes that it decreases along the chunk."""
    inp = wl.make("anyg", 2, 3 * 64 + 5, 2, 128, 128, 64, wl.BF16, seed=350)
    rng = np.random.default_rng(351)
    g = (0.5 * rng.standard_normal(inp.g.shape)).astype(np.float32)          # rises and falls, |differences| of a few units
    Q = wl.queries(inp, seed=352)
    A = oracle.build_A(inp.K, inp.beta, g, 64)
    Kg = oracle._widen(inp.K) * np.exp(g.astype(np.float64))[..., None]
    W64, _ = oracle.wy(A, Kg, None, inp.beta, 64)
    _, U64 = oracle.wy(A, inp.K, inp.V, inp.beta, 64)
    Wb, Ub = to_bf16_bits(W64), to_bf16_bits(U64)
    O_ref, S_ref = oracle.chunk_scan(Q, inp.K, Wb, Ub, g, 64, scale=0.3)
    dev = bnd.to_device(inp)
    O, S = bnd.chunk_scan(bnd.kv_to_torch(Q), dev["K"], bnd.kv_to_torch(Wb), bnd.kv_to_torch(Ub), torch.from_numpy(g).cuda(), 64, scale=0.3)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    assert max_ratio(bnd.to_numpy_f64(O), O_ref) <= TOL_SCAN and max_ratio(bnd.to_numpy_f64(S), S_ref) <= TOL_SCAN
    # and the fused call with the same gate feeds it consistently (decay-weighted W from the kernel)
    gd = torch.from_numpy(g).cuda()
    O2, S2 = bnd.gdn_forward(bnd.kv_to_torch(Q), dev["K"], dev["V"], dev["beta"], gd, 64, scale=0.3)
    torch.cuda.synchronize()
    O_rec, S_rec = oracle.gdn_recurrence(Q, inp.K, inp.V, inp.beta, g, 64, scale=0.3)
    assert max_ratio(bnd.to_numpy_f64(O2), O_rec) <= TOL_LAYER and max_ratio(bnd.to_numpy_f64(S2), S_rec) <= TOL_LAYER


def random_layout(rng, C, max_chunks):
    """A dense or packed layout with ragged ends, empty sequences included."""
    if rng.random() < 0.5:
        n = int(rng.integers(1, 6))
        lens = rng.integers(0, max_chunks * C, size=n)
        lens[rng.integers(0, n)] += 1
        cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        return 1, int(cu[-1]), cu
    return int(rng.integers(1, 4)), int(rng.integers(1, max_chunks * C)), None


@pytest.mark.parametrize("seed", [11, 12])
def test_random_layouts_layer_forward(bnd, seed):
    """Seeded random batch layouts through both launches: within tolerance of the recurrence and bit-identical
    from run to run (a race between the kernel's warps would show up as a difference)."""
    rng = np.random.default_rng(seed)
    for it in range(12):
        H = int(rng.integers(1, 9))
        B, T, cu = random_layout(rng, 64, 7)
        inp = wl.make("rand", B, T, H, 128, 128, 64, wl.BF16, seed=int(rng.integers(1 << 30)), cu_seqlens=cu)
        Q = wl.queries(inp, seed=it)
        S0 = wl.initial_state(inp, seed=it + 1000) if rng.random() < 0.7 else None
        dev = bnd.to_device(inp)
        O_ref, S_ref = oracle.gdn_recurrence(Q, inp.K, inp.V, inp.beta, inp.g, 64, scale=0.2, S0=S0, cu_seqlens=cu)
        runs = []
        for _ in range(2):
            O, S = bnd.gdn_forward(bnd.kv_to_torch(Q), dev["K"], dev["V"], dev["beta"], dev["g"], 64, scale=0.2,
                                   S0=None if S0 is None else torch.from_numpy(S0).cuda(), cu_seqlens=cu)
            torch.cuda.synchronize()
            runs.append((O.clone(), S.clone()))
        assert bnd.last_device_status() == 0
        assert torch.equal(runs[0][0], runs[1][0]) and torch.equal(runs[0][1], runs[1][1])
        assert max_ratio(bnd.to_numpy_f64(O), O_ref) <= TOL_LAYER and max_ratio(bnd.to_numpy_f64(S), S_ref) <= TOL_LAYER, (it, B, T, H, cu)


@pytest.mark.parametrize("n_seqs,H", [(9, 3), (26, 8)], ids=["narrow_slices", "wide_slices"])
def test_chunk_scan_repeats_bit_for_bit(bnd, n_seqs, H):
    """The hand-offs inside a CTA (copies, products, operand writes of ten warps) are all ordered by barriers: the same
    launch on the same inputs gives the same bits every time.  A missing ordering would show as a difference between runs.
    Ragged packed sequences; both slice widths (27 and 208 (sequence, head) pairs)."""
    rng = np.random.default_rng(60 + H)
    cu = np.concatenate([[0], np.cumsum(rng.integers(1, 500, size=n_seqs))]).astype(np.int32)
    inp = wl.make("repeat", 1, int(cu[-1]), H, 128, 128, 64, wl.BF16, seed=360 + H, cu_seqlens=cu)
    Q = wl.queries(inp, seed=361)
    S0 = wl.initial_state(inp, seed=362)
    Wb, Ub = exact_wu(inp, cu)
    dev = bnd.to_device(inp)
    Qd, Wd, Ud = (bnd.kv_to_torch(x) for x in (Q, Wb, Ub))
    S0d = torch.from_numpy(S0).cuda()
    first = None
    for _ in range(12):
        O = torch.full((1, int(cu[-1]), H, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
        O, S = bnd.chunk_scan(Qd, dev["K"], Wd, Ud, dev["g"], 64, scale=128 ** -0.5, S0=S0d, cu_seqlens=cu, out=O)
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        if first is None:
            first = (O.clone(), S.clone())
            O_ref, S_ref = oracle.chunk_scan(Q, inp.K, Wb, Ub, inp.g, 64, scale=128 ** -0.5, S0=S0, cu_seqlens=cu)
            assert max_ratio(bnd.to_numpy_f64(O), O_ref) <= TOL_SCAN and max_ratio(bnd.to_numpy_f64(S), S_ref) <= TOL_SCAN
        else:
            assert torch.equal(O.view(torch.int16), first[0].view(torch.int16)) and torch.equal(S, first[1])
