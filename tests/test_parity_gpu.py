"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle, element by element.

Tolerances (A's are the stated targets of this library; W/U's follow from bf16 storage and bf16 A' operands,
2^-8 + 2^-9 sqrt(C) rms/max, about 5e-3, rounded up):
  fp32 inputs:  max|A_gpu - A_ref| / max|A_ref| <= 1e-5
  bf16 inputs:  the same ratio <= 2e-3 and ||(I+N) A_gpu - I||_max <= 5e-3
  both:         upper triangle all-bits-zero, diagonal exactly 1.0f
  W, U:         max|W_gpu - W_ref| / max|W_ref| <= 1e-2 (bf16 storage), <= 1e-5 (fp32)
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_21325_b200 import workloads as wl
from parity_util import max_ratio, max_residual, structure_errors

pytestmark = pytest.mark.gpu

TOL_A = {wl.F32: 1e-5, wl.BF16: 2e-3}
TOL_RES = {wl.F32: 5e-5, wl.BF16: 5e-3}
TOL_WY = {wl.F32: 1e-5, wl.BF16: 1e-2}


@pytest.fixture(scope="module")
def bnd():
    import __graft_entry__ as entry
    entry.build()
    from paper_2605_21325_b200 import binding
    torch.cuda.set_device(0)
    return binding


_oracle_cache = {}


def oracle_all(inp, key=None):
    if key is not None and key in _oracle_cache:
        return _oracle_cache[key]
    A, N = oracle.build_A(inp.K, inp.beta, inp.g, inp.C, cu_seqlens=inp.cu_seqlens, return_N=True)
    W, U = oracle.wy(A, inp.K, inp.V, inp.beta, inp.C, cu_seqlens=inp.cu_seqlens)
    if key is not None:
        _oracle_cache[key] = (A, N, W, U)
    return A, N, W, U


def nan_like(shape, dtype, device="cuda"):
    """Output buffers pre-filled with NaN: an unwritten real row shows up, and rows of no token must stay NaN."""
    return torch.full(shape, float("nan"), dtype=dtype, device=device)


def token_mask(inp):
    m = np.zeros(inp.B * inp.T, dtype=bool)
    for t0, r in inp.chunk_list():
        m[t0:t0 + r] = True
    return m.reshape(inp.B, inp.T)


def check_A(A_t, inp, A_ref, N_ref, tol=None, tol_res=None):
    A = A_t.detach().cpu().numpy()
    assert not np.isnan(A).any(), "a row of A was not written"
    bad_upper, bad_diag = structure_errors(A, inp)
    assert bad_upper == 0, "upper triangle is not bit-exact +0.0"
    assert bad_diag == 0, "diagonal is not exactly 1.0f"
    r = max_ratio(A, A_ref)
    assert r <= (TOL_A[inp.kv_dtype] if tol is None else tol), "A ratio %.3e" % r
    res = max_residual(A, N_ref, inp, max_chunks=64)
    assert res <= (TOL_RES[inp.kv_dtype] if tol_res is None else tol_res), "residual %.3e" % res
    return r, res


def check_WU(W_t, U_t, inp, W_ref, U_ref, bnd, tol=None):
    tol = TOL_WY[inp.kv_dtype] if tol is None else tol
    W, U = bnd.to_numpy_f64(W_t), bnd.to_numpy_f64(U_t)
    assert not np.isnan(W).any() and not np.isnan(U).any()
    rw, ru = max_ratio(W, W_ref), max_ratio(U, U_ref)
    assert rw <= tol and ru <= tol, "W ratio %.3e, U ratio %.3e" % (rw, ru)
    return rw, ru


def run_fused(bnd, inp, method, want_A=True):
    dev = bnd.to_device(inp)
    A = nan_like((inp.B, inp.T, inp.H, inp.C), torch.float32) if want_A else None
    W = nan_like(dev["K"].shape, dev["K"].dtype)
    U = nan_like(dev["V"].shape, dev["V"].dtype)
    bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], inp.C, method=method, cu_seqlens=inp.cu_seqlens, out=(A, W, U))
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    return A, W, U


def methods(bnd):
    return [bnd.BLOCK_RECURSIVE, bnd.BLOCK_RECURSIVE | bnd.LEAF_SERIES, bnd.PRODUCT_SERIES]


# ---------------------------------------------------------------- config 1: fp32 throughout

@pytest.mark.parametrize("mi", [0, 1, 2])
def test_cfg1_fp32_build(bnd, mi):
    inp = wl.config(1)
    A_ref, N_ref, _, _ = oracle_all(inp, "cfg1")
    dev = bnd.to_device(inp)
    A = nan_like((inp.B, inp.T, inp.H, inp.C), torch.float32)
    bnd.build(dev["K"], dev["beta"], dev["g"], inp.C, method=methods(bnd)[mi], out=A)
    torch.cuda.synchronize()
    check_A(A, inp, A_ref, N_ref)


@pytest.mark.parametrize("mi", [0, 2])
def test_cfg1_fp32_fused_and_wy(bnd, mi):
    inp = wl.config(1)
    A_ref, N_ref, W_ref, U_ref = oracle_all(inp, "cfg1")
    A, W, U = run_fused(bnd, inp, methods(bnd)[mi])
    check_A(A, inp, A_ref, N_ref)
    check_WU(W, U, inp, W_ref, U_ref, bnd)
    # tri_inv_wy on the oracle's A rounded to fp32
    dev = bnd.to_device(inp)
    W2, U2 = bnd.wy(torch.from_numpy(A_ref.astype(np.float32)).cuda(), dev["K"], dev["V"], dev["beta"])
    torch.cuda.synchronize()
    check_WU(W2, U2, inp, W_ref, U_ref, bnd)


# ---------------------------------------------------------------- small bf16 cases, every method, both kernels

@pytest.mark.parametrize("force_simt", [False, True])
@pytest.mark.parametrize("mi", [0, 1, 2])
def test_small_bf16_c64(bnd, mi, force_simt):
    inp = wl.config(2, shrink=16)                      # B=4, T=256, H=16, d=128: 256 matrices, several waves of tiles
    A_ref, N_ref, W_ref, U_ref = oracle_all(inp, "cfg2s")
    m = methods(bnd)[mi] | (bnd.FORCE_SIMT if force_simt else 0)
    A, W, U = run_fused(bnd, inp, m)
    check_A(A, inp, A_ref, N_ref)
    check_WU(W, U, inp, W_ref, U_ref, bnd)


@pytest.mark.parametrize("force_simt", [False, True])
@pytest.mark.parametrize("mi", [0, 1, 2])
def test_small_bf16_c128(bnd, mi, force_simt):
    inp = wl.config(4, shrink=16)                      # B=2, T=512, H=16, d=128, C=128: 128 matrices
    A_ref, N_ref, W_ref, U_ref = oracle_all(inp, "cfg4s")
    m = methods(bnd)[mi] | (bnd.FORCE_SIMT if force_simt else 0)
    A, W, U = run_fused(bnd, inp, m)
    check_A(A, inp, A_ref, N_ref)
    check_WU(W, U, inp, W_ref, U_ref, bnd)


@pytest.mark.parametrize("C", [16, 32, 64, 128])
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_chunk_sizes_and_odd_shapes(bnd, C, dtype):
    # T not a multiple of C (partial last chunk per sequence), d_k != d_v, 3 heads
    inp = wl.make("odd", 2, 3 * C + 5, 3, 64, 32, C, dtype, seed=40 + C)
    A_ref, N_ref, W_ref, U_ref = oracle_all(inp)
    for m in methods(bnd):
        A, W, U = run_fused(bnd, inp, m)
        check_A(A, inp, A_ref, N_ref)
        check_WU(W, U, inp, W_ref, U_ref, bnd)


# ---------------------------------------------------------------- entry points agree with each other

def test_build_then_wy_equals_fused(bnd):
    inp = wl.config(2, shrink=32)
    dev = bnd.to_device(inp)
    for m in (bnd.BLOCK_RECURSIVE, bnd.PRODUCT_SERIES):
        A1 = bnd.build(dev["K"], dev["beta"], dev["g"], inp.C, method=m)
        W1, U1 = bnd.wy(A1, dev["K"], dev["V"], dev["beta"])
        A2, W2, U2 = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], inp.C, method=m)
        _, W3, U3 = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], inp.C, method=m, want_A=False)
        torch.cuda.synchronize()
        assert torch.equal(A1, A2)
        assert torch.equal(W2, W3) and torch.equal(U2, U3)
        # build+wy re-reads A from memory in fp32, the fused kernel keeps it on chip: same values
        assert (W1.float() - W2.float()).abs().max().item() <= 2 ** -7 * W2.float().abs().max().item()
        assert (U1.float() - U2.float()).abs().max().item() <= 2 ** -7 * U2.float().abs().max().item()


def test_wy_only_w(bnd):
    inp = wl.config(2, shrink=32)
    A_ref, _, W_ref, _ = oracle_all(inp, "cfg2ss")
    dev = bnd.to_device(inp)
    W, U = bnd.wy(torch.from_numpy(A_ref.astype(np.float32)).cuda(), dev["K"], None, dev["beta"])
    torch.cuda.synchronize()
    assert U is None
    assert max_ratio(bnd.to_numpy_f64(W), W_ref) <= 1e-2


# ---------------------------------------------------------------- exact case: first-difference matrix

@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("C", [64, 128])
def test_first_difference_is_exact(bnd, dtype, C):
    # N = all-ones strictly lower: every intermediate of the block recursion is 0 or +-1, so the
    # result must equal the first-difference matrix exactly in any arithmetic.
    inp = wl.first_difference_case(2, 2 * C, 2, 128, C, dtype)
    A, W, U = run_fused(bnd, inp, bnd.BLOCK_RECURSIVE)
    exp = (np.eye(C) - np.eye(C, k=-1)).astype(np.float32)
    A = A.cpu().numpy()
    for b in range(2):
        for c in range(2):
            for h in range(2):
                assert np.array_equal(A[b, c * C:(c + 1) * C, h, :], exp)
    # W = A K with identical keys e_0: row 0 is e_0, every other row is 0; U = A * ones likewise
    Wn = bnd.to_numpy_f64(W)
    assert np.array_equal(Wn[:, 0::C, :, 0], np.ones_like(Wn[:, 0::C, :, 0]))
    assert np.count_nonzero(Wn) == Wn[:, 0::C, :, 0].size


# ---------------------------------------------------------------- ragged packing, partial chunks, untouched rows

@pytest.mark.parametrize("force_simt", [False, True])
def test_ragged_cfg5_small(bnd, force_simt):
    inp = wl.config(5, shrink=8)                       # 8 packed sequences, lengths in [1, 2048]
    A_ref, N_ref, W_ref, U_ref = oracle_all(inp, "cfg5s")
    for m in methods(bnd):
        A, W, U = run_fused(bnd, inp, m | (bnd.FORCE_SIMT if force_simt else 0))
        check_A(A, inp, A_ref, N_ref)
        check_WU(W, U, inp, W_ref, U_ref, bnd)


def test_short_sequences_and_neighbour_isolation(bnd):
    # lengths 1, 69, 64, 66, 3: partial chunks sit directly before other sequences' rows, whose keys
    # are set to huge values; nothing of them may leak into the short chunk's result.
    cu = np.array([0, 1, 70, 134, 200, 203], np.int32)
    rng = np.random.default_rng(9)
    inp = wl.make("iso", 1, int(cu[-1]), 4, 128, 128, 64, wl.BF16, seed=9, kind="stress", cu_seqlens=cu, rng=rng)
    A_ref, N_ref, W_ref, U_ref = oracle_all(inp)
    for m in methods(bnd):
        A, W, U = run_fused(bnd, inp, m)
        check_A(A, inp, A_ref, N_ref)
        check_WU(W, U, inp, W_ref, U_ref, bnd)
    # same inputs with every other sequence's keys replaced by infinities: sequence 1 must not change
    K2 = wl.bf16_bits_to_f32(inp.K).copy()
    K2[:, 70:] = np.inf
    K2[:, :1] = np.inf
    inp2 = wl.Inputs("iso2", 1, inp.T, 4, 128, 128, 64, wl.BF16, wl.f32_to_bf16_bits(K2), inp.V, inp.beta, inp.g, cu)
    A2, W2, U2 = run_fused(bnd, inp2, bnd.BLOCK_RECURSIVE)
    A1, W1, U1 = run_fused(bnd, inp, bnd.BLOCK_RECURSIVE)
    assert torch.equal(A1[:, 1:70], A2[:, 1:70]) and torch.equal(W1[:, 1:70], W2[:, 1:70])


def test_dense_partial_tail_rows_beyond_T_untouched(bnd):
    # allocate T+C rows, describe only T: the extra rows must keep their NaN sentinel
    T, C, H, d = 100, 64, 2, 128
    inp = wl.make("tail", 1, T, H, d, d, C, wl.BF16, seed=77)
    dev = bnd.to_device(inp)
    A = nan_like((1, T + C, H, C), torch.float32)
    W = nan_like((1, T + C, H, d), torch.bfloat16)
    U = nan_like((1, T + C, H, d), torch.bfloat16)
    desc, keep = bnd.make_desc(1, T, H, d, d, C, bnd.BF16)
    import ctypes
    rc = bnd.load().tri_inv_fused(bnd._p(dev["K"]), bnd._p(dev["V"]), bnd._p(dev["beta"]), bnd._p(dev["g"]),
                                  bnd._p(A), bnd._p(W), bnd._p(U), ctypes.byref(desc), 0, bnd._stream(None))
    assert rc == 0
    torch.cuda.synchronize()
    assert torch.isnan(A[:, T:]).all() and torch.isnan(W[:, T:].float()).all() and torch.isnan(U[:, T:].float()).all()
    assert not torch.isnan(A[:, :T]).any()
    A_ref, N_ref, _, _ = oracle_all(inp)
    assert max_ratio(A[:, :T].cpu().numpy(), A_ref) <= 2e-3


def test_empty_inputs(bnd):
    K = torch.zeros((1, 0, 2, 128), dtype=torch.bfloat16, device="cuda")
    b = torch.zeros((1, 0, 2), dtype=torch.float32, device="cuda")
    # zero tokens: nothing to do, no launch, no error (pointers of empty tensors may be null: pass a dummy)
    dummy = torch.zeros(16, device="cuda")
    desc, _ = bnd.make_desc(1, 0, 2, 128, 128, 64, bnd.BF16)
    import ctypes
    rc = bnd.load().tri_inv_build(bnd._p(dummy), bnd._p(dummy), bnd._p(dummy), bnd._p(dummy), ctypes.byref(desc), 0, None)
    assert rc == 0
    desc, keep = bnd.make_desc(1, 0, 2, 128, 128, 64, bnd.BF16, np.array([0, 0, 0], np.int32))
    rc = bnd.load().tri_inv_build(bnd._p(dummy), bnd._p(dummy), bnd._p(dummy), bnd._p(dummy), ctypes.byref(desc), 0, None)
    assert rc == 0
    torch.cuda.synchronize()


def test_launch_counter_and_device_status(bnd):
    inp = wl.config(2, shrink=32)
    dev = bnd.to_device(inp)
    n0 = bnd.launch_count()
    bnd.build(dev["K"], dev["beta"], dev["g"], inp.C)
    bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], inp.C)
    torch.cuda.synchronize()
    assert bnd.launch_count() == n0 + 2
    assert bnd.last_device_status() == 0


def test_runs_on_a_side_stream(bnd):
    inp = wl.config(2, shrink=32)
    A_ref, _, _, _ = oracle_all(inp, "cfg2ss")
    dev = bnd.to_device(inp)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        A = bnd.build(dev["K"], dev["beta"], dev["g"], inp.C, stream=s)
    s.synchronize()
    assert max_ratio(A.cpu().numpy(), A_ref) <= 2e-3


# ---------------------------------------------------------------- Newton-Schulz (Alg. 3) and refinement (Alg. 6)

@pytest.mark.parametrize("cfg,shrink", [(1, 1), (2, 32)])
def test_newton_schulz_and_refinement(bnd, cfg, shrink):
    inp = wl.config(cfg, shrink=shrink)
    A_ref, N_ref, W_ref, U_ref = oracle_all(inp)
    # default iteration count (2 log2 C) reaches fp32 accuracy
    A, W, U = run_fused(bnd, inp, bnd.NEWTON_SCHULZ)
    r_full, _ = check_A(A, inp, A_ref, N_ref, tol=1e-5, tol_res=5e-5)
    check_WU(W, U, inp, W_ref, U_ref, bnd)
    # too few iterations leave a visible error; one refinement step equals one more round
    errs = {}
    for name, m in (("ns6", bnd.NEWTON_SCHULZ | bnd.ns_iters(6)), ("ns8", bnd.NEWTON_SCHULZ | bnd.ns_iters(8)),
                    ("ns8+ir", bnd.NEWTON_SCHULZ | bnd.ns_iters(8) | bnd.REFINE), ("ns9", bnd.NEWTON_SCHULZ | bnd.ns_iters(9))):
        A, _, _ = run_fused(bnd, inp, m)
        errs[name] = max_ratio(A.cpu().numpy(), A_ref)
    assert errs["ns6"] > errs["ns8"] > errs["ns8+ir"] and errs["ns6"] > 1e-3
    assert abs(errs["ns8+ir"] - errs["ns9"]) <= 1e-5 + 0.05 * errs["ns9"]
    # refinement after the block recursion keeps the result within the fp32 bound
    A, W, U = run_fused(bnd, inp, bnd.BLOCK_RECURSIVE | bnd.REFINE)
    check_A(A, inp, A_ref, N_ref, tol=1e-5, tol_res=5e-5)
    A, _, _ = run_fused(bnd, inp, bnd.BLOCK_RECURSIVE | bnd.LEAF_SERIES | bnd.REFINE)
    check_A(A, inp, A_ref, N_ref, tol=1e-5, tol_res=5e-5)


@pytest.mark.parametrize("C", [64, 128])
def test_refinement_step_on_the_tensor_cores(bnd, C):
    """Alg. 6 after the block recursion, bf16 keys (tensor-core kernel): one step brings the forward error from
    the TF32 level of the merges (about 1e-4) down to a few 1e-6 or better -- Sec. 4.1's remark that one step gives
    the mixed recursion its lost digits back.  Dense and packed (short chunks), fused, build-only and raw calls."""
    rng = np.random.default_rng(77 + C)
    cu = wl.ragged_lengths(5, 5 * C, rng)
    cases = [wl.make("ref_dense", 2, 6 * C, 4, 128, 128, C, wl.BF16, seed=910 + C),
             wl.make("ref_packed", 1, int(cu[-1]), 3, 128, 128, C, wl.BF16, seed=920 + C, cu_seqlens=cu, rng=rng)]
    for inp in cases:
        A_ref, N_ref, W_ref, U_ref = oracle_all(inp)
        A0, _, _ = run_fused(bnd, inp, bnd.BLOCK_RECURSIVE)
        e_plain = max_ratio(A0.cpu().numpy(), A_ref)
        for m in (bnd.BLOCK_RECURSIVE | bnd.REFINE, bnd.BLOCK_RECURSIVE | bnd.LEAF_SERIES | bnd.REFINE):
            A, W, U = run_fused(bnd, inp, m)
            e_ref, _ = check_A(A, inp, A_ref, N_ref, tol=2e-5, tol_res=5e-5)
            check_WU(W, U, inp, W_ref, U_ref, bnd)
            assert e_ref < 0.2 * e_plain, (e_plain, e_ref)
        dev = bnd.to_device(inp)
        A = bnd.build(dev["K"], dev["beta"], dev["g"], C, method=bnd.BLOCK_RECURSIVE | bnd.REFINE, cu_seqlens=inp.cu_seqlens,
                      out=nan_like((inp.B, inp.T, inp.H, C), torch.float32))
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        check_A(A, inp, A_ref, N_ref, tol=2e-5, tol_res=5e-5)
    # the raw front end with the refinement step
    raw = wl.make_raw("ref_raw", 2, 4 * C, 2, 128, C, wl.BF16, seed=930 + C)
    Kh, bh, gh = oracle.raw_front_end(raw.K, raw.beta, raw.g, C)
    A_ref = oracle.build_A(Kh, bh, gh, C)
    dev = bnd.to_device(raw)
    A, W, U, _, _ = bnd.fused_raw(dev["K"], dev["V"], dev["beta"], dev["g"], C, method=bnd.BLOCK_RECURSIVE | bnd.REFINE)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    assert max_ratio(A.cpu().numpy(), A_ref) <= 2e-5


@pytest.mark.parametrize("C", [64, 128])
def test_product_series_with_fp16_operands(bnd, C):
    """Alg. 5 with fp16 operands (TRI_INV_OPERANDS_F16; Sec. 4.1 ranks fp16 above bf16): same tolerances as the TF32
    series on the configurations' value distributions; dense, packed with short chunks, build-only and raw calls."""
    rng = np.random.default_rng(177 + C)
    cu = wl.ragged_lengths(6, 4 * C, rng)
    m = bnd.PRODUCT_SERIES | bnd.OPERANDS_F16
    for inp in (wl.make("h16_dense", 2, 5 * C, 4, 128, 128, C, wl.BF16, seed=940 + C),
                wl.make("h16_packed", 1, int(cu[-1]), 3, 128, 128, C, wl.BF16, seed=950 + C, cu_seqlens=cu, rng=rng)):
        A_ref, N_ref, W_ref, U_ref = oracle_all(inp)
        A, W, U = run_fused(bnd, inp, m)
        check_A(A, inp, A_ref, N_ref)
        check_WU(W, U, inp, W_ref, U_ref, bnd)
        dev = bnd.to_device(inp)
        A = bnd.build(dev["K"], dev["beta"], dev["g"], C, method=m, cu_seqlens=inp.cu_seqlens, out=nan_like((inp.B, inp.T, inp.H, C), torch.float32))
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        check_A(A, inp, A_ref, N_ref)
    raw = wl.make_raw("h16_raw", 2, 4 * C, 2, 128, C, wl.BF16, seed=960 + C)
    Kh, bh, gh = oracle.raw_front_end(raw.K, raw.beta, raw.g, C)
    A_ref = oracle.build_A(Kh, bh, gh, C)
    dev = bnd.to_device(raw)
    A, W, U, _, _ = bnd.fused_raw(dev["K"], dev["V"], dev["beta"], dev["g"], C, method=m)
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    assert max_ratio(A.cpu().numpy(), A_ref) <= 2e-3
    # (the first-difference example of Sec. 3.2 is no case for this variant: its powers of N are binomials up to
    # about 2^C / sqrt(C), far outside fp16's range -- the overflow the header warns of)
    # fp32 storage has no fp16-operand kernel: a clear refusal, no launch
    f32 = wl.config(1)
    d32 = bnd.to_device(f32)
    with pytest.raises(bnd.TriInvError) as e:
        bnd.build(d32["K"], d32["beta"], d32["g"], 64, method=m)
    assert e.value.status == bnd.ERR_UNSUPPORTED


def test_method_flag_combinations_rejected(bnd):
    import ctypes
    d = torch.zeros(64, device="cuda")
    desc, _ = bnd.make_desc(1, 64, 1, 128, 128, 64, bnd.BF16)
    L = bnd.load()
    for bad in (bnd.PRODUCT_SERIES | bnd.REFINE, bnd.BLOCK_RECURSIVE | bnd.ns_iters(4), bnd.NEWTON_SCHULZ | bnd.LEAF_SERIES, 3,
                bnd.BLOCK_RECURSIVE | bnd.OPERANDS_F16, bnd.PRODUCT_SERIES | bnd.OPERANDS_F16 | bnd.FORCE_SIMT):
        rc = L.tri_inv_build(bnd._p(d), bnd._p(d), bnd._p(d), bnd._p(d), ctypes.byref(desc), bad, None)
        assert rc == bnd.ERR_UNSUPPORTED, bad


# ---------------------------------------------------------------- fused front end (raw keys and logits)

def oracle_raw(raw):
    Kh, b, g = oracle.raw_front_end(raw.K, raw.beta, raw.g, raw.C, cu_seqlens=raw.cu_seqlens)
    A, N = oracle.build_A(Kh, b, g, raw.C, cu_seqlens=raw.cu_seqlens, return_N=True)
    W, U = oracle.wy(A, Kh, raw.V, b, raw.C, cu_seqlens=raw.cu_seqlens)
    return A, N, W, U, b, g


@pytest.mark.parametrize("C,dtype,d", [(64, wl.BF16, 128), (128, wl.BF16, 128), (64, wl.F32, 64), (32, wl.BF16, 64)])
def test_fused_raw_front_end(bnd, C, dtype, d):
    cu = np.array([0, 3 * C + 7, 5 * C + 7, 5 * C + 8], np.int32)          # partial chunks and a one-token sequence
    for cu_seqlens, B, T in ((None, 2, 4 * C), (cu, 1, int(cu[-1]))):
        raw = wl.make_raw("raw", B, T, 3, d, C, dtype, seed=60 + C, cu_seqlens=cu_seqlens)
        A_ref, N_ref, W_ref, U_ref, b_ref, g_ref = oracle_raw(raw)
        dev = bnd.to_device(raw)
        for m in methods(bnd):
            out = (nan_like((B, T, 3, C), torch.float32), nan_like(dev["K"].shape, dev["K"].dtype), nan_like(dev["V"].shape, dev["V"].dtype),
                   nan_like((B, T, 3), torch.float32), nan_like((B, T, 3), torch.float32))
            A, W, U, bo, go = bnd.fused_raw(dev["K"], dev["V"], dev["beta"], dev["g"], C, method=m, cu_seqlens=cu_seqlens, out=out)
            torch.cuda.synchronize()
            assert bnd.last_device_status() == 0
            check_A(A, raw, A_ref, N_ref)
            check_WU(W, U, raw, W_ref, U_ref, bnd)
            assert np.abs(bo.cpu().numpy() - b_ref).max() <= 1e-6
            assert np.abs(go.cpu().numpy() - g_ref).max() <= 1e-5 * max(1.0, np.abs(g_ref).max())
        # gates are optional
        A2, W2, U2, bo2, go2 = bnd.fused_raw(dev["K"], dev["V"], dev["beta"], dev["g"], C, cu_seqlens=cu_seqlens)
        torch.cuda.synchronize()
        assert bo2 is None and go2 is None
        check_A(A2, raw, A_ref, N_ref)


def test_fused_raw_equals_fused_on_prepared_inputs(bnd):
    # the same layer step done in two passes (front end on the host in fp32, then tri_inv_fused) and in one
    raw = wl.make_raw("raw", 2, 256, 4, 128, 64, wl.BF16, seed=71)
    Kh, b, g = oracle.raw_front_end(raw.K, raw.beta, raw.g, 64)
    prep = wl.Inputs("prep", 2, 256, 4, 128, 128, 64, wl.BF16, wl.f32_to_bf16_bits(Kh.astype(np.float32)), raw.V,
                     b.astype(np.float32), g.astype(np.float32))
    d_raw, d_prep = bnd.to_device(raw), bnd.to_device(prep)
    A1, W1, U1, _, _ = bnd.fused_raw(d_raw["K"], d_raw["V"], d_raw["beta"], d_raw["g"], 64)
    A2, W2, U2 = bnd.fused(d_prep["K"], d_prep["V"], d_prep["beta"], d_prep["g"], 64)
    torch.cuda.synchronize()
    # two-pass keys are rounded to bf16 after normalising, the fused path normalises the Gram in fp32: close, not equal
    assert (A1 - A2).abs().max().item() <= 2e-3
    assert (W1.float() - W2.float()).abs().max().item() <= 1e-2 * W2.float().abs().max().item()
    assert (U1.float() - U2.float()).abs().max().item() <= 1e-2 * U2.float().abs().max().item()


# ---------------------------------------------------------------- host-to-host pipeline

@pytest.mark.parametrize("B,T", [(4, 512), (1, 2048), (2, 192)])
def test_host_pipeline_matches_single_call(bnd, B, T):
    inp = wl.make("pipe", B, T, 4, 128, 128, 64, wl.BF16, seed=83)
    dev = bnd.to_device(inp)
    A, W, U = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], 64)
    pipe = bnd.HostPipeline(B, T, 4, 128, 128, 64)
    hK, hV = bnd.kv_to_torch(inp.K, "cpu", pin=True), bnd.kv_to_torch(inp.V, "cpu", pin=True)
    hb, hg = torch.from_numpy(inp.beta).pin_memory(), torch.from_numpy(inp.g).pin_memory()
    hA = torch.full(A.shape, float("nan")).pin_memory()
    hW, hU = torch.zeros(W.shape, dtype=W.dtype).pin_memory(), torch.zeros(U.shape, dtype=U.dtype).pin_memory()
    for _ in range(2):
        pipe.run(hK, hV, hb, hg, hA, hW, hU)
    torch.cuda.synchronize()
    assert torch.equal(hA, A.cpu()) and torch.equal(hW, W.cpu()) and torch.equal(hU, U.cpu())


def test_concurrent_launches_on_two_streams(bnd):
    # launches that overlap on the GPU use different work counters and their own tensor memory
    inp1, inp2 = wl.config(2, shrink=4), wl.config(4, shrink=4)
    d1, d2 = bnd.to_device(inp1), bnd.to_device(inp2)
    ref1 = bnd.fused(d1["K"], d1["V"], d1["beta"], d1["g"], inp1.C)
    ref2 = bnd.fused(d2["K"], d2["V"], d2["beta"], d2["g"], inp2.C, method=bnd.PRODUCT_SERIES)
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    outs1, outs2 = [], []
    for _ in range(6):
        with torch.cuda.stream(s1):
            outs1.append(bnd.fused(d1["K"], d1["V"], d1["beta"], d1["g"], inp1.C, stream=s1))
        with torch.cuda.stream(s2):
            outs2.append(bnd.fused(d2["K"], d2["V"], d2["beta"], d2["g"], inp2.C, method=bnd.PRODUCT_SERIES, stream=s2))
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    for o in outs1:
        assert all(torch.equal(a, b) for a, b in zip(o, ref1))
    for o in outs2:
        assert all(torch.equal(a, b) for a, b in zip(o, ref2))


# ---------------------------------------------------------------- per-channel decay (KDA row of Table 1)

@pytest.mark.parametrize("C,dtype,d", [(64, wl.BF16, 128), (64, wl.F32, 64), (32, wl.BF16, 64), (128, wl.BF16, 128)])
def test_build_kda(bnd, C, dtype, d):
    cu = np.array([0, 2 * C + 9, 3 * C + 9, 3 * C + 10], np.int32)
    for cu_seqlens, B, T in ((None, 2, 3 * C), (cu, 1, int(cu[-1]))):
        inp = wl.make("kda", B, T, 3, d, d, C, dtype, seed=90 + C, cu_seqlens=cu_seqlens)
        G = wl.per_channel_gate(inp, seed=91)
        A_ref, N_ref = oracle.build_A_kda(inp.K, G, inp.beta, C, cu_seqlens=cu_seqlens, return_N=True)
        dev = bnd.to_device(inp)
        Gd = torch.from_numpy(G).cuda()
        for m in (bnd.BLOCK_RECURSIVE, bnd.BLOCK_RECURSIVE | bnd.LEAF_SERIES, bnd.PRODUCT_SERIES):
            A = nan_like((B, T, 3, C), torch.float32)
            bnd.build_kda(dev["K"], Gd, dev["beta"], C, method=m, cu_seqlens=cu_seqlens, out=A)
            torch.cuda.synchronize()
            assert bnd.last_device_status() == 0
            # bf16 operands K * exp(+-(G - G_mid)) carry 2^-9 relative rounding each: same bound as the bf16 configs
            check_A(A, inp, A_ref, N_ref)


def test_build_kda_with_a_channel_constant_gate_equals_build(bnd):
    inp = wl.config(2, shrink=16)
    dev = bnd.to_device(inp)
    G = torch.from_numpy(np.repeat(inp.g[..., None], 128, axis=-1).copy()).cuda()
    A1 = bnd.build_kda(dev["K"], G, dev["beta"], 64)
    A2 = bnd.build(dev["K"], dev["beta"], dev["g"], 64)
    torch.cuda.synchronize()
    assert (A1 - A2).abs().max().item() <= 2e-3


# ---------------------------------------------------------------- decay-weighted W (input of the chunk scan)

@pytest.mark.parametrize("C,dtype,d", [(64, wl.BF16, 128), (128, wl.BF16, 128), (64, wl.F32, 64)])
def test_fused_decay_weighted_w(bnd, C, dtype, d):
    cu = np.array([0, 2 * C + 9, 3 * C + 9, 3 * C + 10], np.int32)
    for cu_seqlens, B, T in ((None, 2, 3 * C), (cu, 1, int(cu[-1]))):
        inp = wl.make("wd", B, T, 2, d, d, C, dtype, seed=70 + C, cu_seqlens=cu_seqlens)
        A_ref = oracle.build_A(inp.K, inp.beta, inp.g, C, cu_seqlens=cu_seqlens)
        Kg = bnd.to_numpy_f64(bnd.kv_to_torch(inp.K, "cpu")) * np.exp(inp.g.astype(np.float64))[..., None]
        W_ref, _ = oracle.wy(A_ref, Kg, None, inp.beta, C, cu_seqlens=cu_seqlens)
        _, U_ref = oracle.wy(A_ref, inp.K, inp.V, inp.beta, C, cu_seqlens=cu_seqlens)
        dev = bnd.to_device(inp)
        for m in (bnd.BLOCK_RECURSIVE, bnd.PRODUCT_SERIES):
            A, W, U = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], C, method=m | bnd.W_DECAY, cu_seqlens=cu_seqlens)
            torch.cuda.synchronize()
            assert bnd.last_device_status() == 0
            assert max_ratio(bnd.to_numpy_f64(W), W_ref) <= TOL_WY[dtype]
            assert max_ratio(bnd.to_numpy_f64(U), U_ref) <= TOL_WY[dtype]


def test_w_decay_is_refused_where_there_is_no_w(bnd):
    inp = wl.config(1)
    dev = bnd.to_device(inp)
    with pytest.raises(bnd.TriInvError):
        bnd.build(dev["K"], dev["beta"], dev["g"], inp.C, method=bnd.BLOCK_RECURSIVE | bnd.W_DECAY)


# ---------------------------------------------------------------- re-entrancy
def test_concurrent_calls_from_two_host_threads_on_two_streams(bnd):
    """The library is re-entrant: launches that overlap on different streams, issued by different host threads,
    neither share a work counter nor disturb each other's results (bit-exact against the serial runs)."""
    import threading
    cases = []
    for seed, cu in ((501, None), (502, np.array([0, 300, 301, 900], np.int32))):
        B, T = (2, 8 * 64) if cu is None else (1, int(cu[-1]))
        inp = wl.make("mt", B, T, 8, 128, 128, 64, wl.BF16, seed=seed, cu_seqlens=cu)
        dev = bnd.to_device(inp)
        ref = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], 64, cu_seqlens=cu)
        cases.append((inp, dev, cu, ref))
    torch.cuda.synchronize()
    errors = []

    def worker(k):
        try:
            inp, dev, cu, ref = cases[k]
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                for _ in range(25):
                    A, W, U = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], 64, cu_seqlens=cu, stream=st)
            st.synchronize()
            if not (torch.equal(A, ref[0]) and torch.equal(W, ref[1]) and torch.equal(U, ref[2])):
                errors.append("thread %d: results differ from the serial run" % k)
        except Exception as e:  # noqa: BLE001
            errors.append(repr(e))

    threads = [threading.Thread(target=worker, args=(k,)) for k in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    assert bnd.last_device_status() == 0


@pytest.mark.parametrize("seed", [21, 22])
def test_random_layouts_fused_all_methods(bnd, seed):
    """Seeded random batch layouts (dense and packed, ragged ends, empty sequences), both chunk sizes, every scheme:
    within tolerance of the oracle and bit-identical from run to run."""
    rng = np.random.default_rng(seed)
    for it in range(10):
        C = int(rng.choice([64, 128]))
        H = int(rng.integers(1, 7))
        if rng.random() < 0.5:
            n = int(rng.integers(1, 6))
            lens = rng.integers(0, 5 * C, size=n)
            lens[rng.integers(0, n)] += 1
            cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
            B, T = 1, int(cu[-1])
        else:
            cu, B, T = None, int(rng.integers(1, 4)), int(rng.integers(1, 6 * C))
        inp = wl.make("rand", B, T, H, 128, 128, C, wl.BF16, seed=int(rng.integers(1 << 30)), cu_seqlens=cu)
        dev = bnd.to_device(inp)
        A_ref, N_ref = oracle.build_A(inp.K, inp.beta, inp.g, C, cu_seqlens=cu, return_N=True)
        W_ref, U_ref = oracle.wy(A_ref, inp.K, inp.V, inp.beta, C, cu_seqlens=cu)
        for m in (bnd.BLOCK_RECURSIVE, bnd.BLOCK_RECURSIVE | bnd.LEAF_SERIES, bnd.PRODUCT_SERIES):
            runs = []
            for _ in range(2):
                A = nan_like((B, T, H, C), torch.float32)
                W, U = nan_like(dev["K"].shape, dev["K"].dtype), nan_like(dev["V"].shape, dev["V"].dtype)
                bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], C, method=m, cu_seqlens=cu, out=(A, W, U))
                torch.cuda.synchronize()
                runs.append((A, W, U))
            assert bnd.last_device_status() == 0
            assert all(torch.equal(x, y) for x, y in zip(runs[0], runs[1]))
            check_A(runs[0][0], inp, A_ref, N_ref)
            assert max_ratio(bnd.to_numpy_f64(runs[0][1]), W_ref) <= TOL_WY[wl.BF16]
            assert max_ratio(bnd.to_numpy_f64(runs[0][2]), U_ref) <= TOL_WY[wl.BF16]


def test_head_dimension_64_on_the_tensor_cores(bnd):
    """bf16 keys and values with d_k = d_v = 64 at C = 64: tri_inv_build, tri_inv_fused (block recursion and series
    leaves) and tri_inv_wy take the tensor-core kernel's one-box instances.  Dense and packed ragged layouts, every
    matrix against the fp64 oracle; sentinels show that every row of real tokens is written and no other."""
    rng = np.random.default_rng(77)
    cu = wl.ragged_lengths(7, 5 * 64, rng)
    cases = [wl.make("d64_dense", 3, 6 * 64, 5, 64, 64, 64, wl.BF16, seed=1700),
             wl.make("d64_packed", 1, int(cu[-1]), 4, 64, 64, 64, wl.BF16, seed=1701, cu_seqlens=cu, rng=rng)]
    for inp in cases:
        cuq = inp.cu_seqlens
        A_ref, N_ref = oracle.build_A(inp.K, inp.beta, inp.g, 64, cu_seqlens=cuq, return_N=True)
        W_ref, U_ref = oracle.wy(A_ref, inp.K, inp.V, inp.beta, 64, cu_seqlens=cuq)
        dev = bnd.to_device(inp)
        nan = lambda t: torch.full_like(t, float("nan"))
        for m in (bnd.BLOCK_RECURSIVE, bnd.BLOCK_RECURSIVE | bnd.LEAF_SERIES):
            out = (torch.full((inp.B, inp.T, inp.H, 64), float("nan"), dtype=torch.float32, device="cuda"), nan(dev["K"]), nan(dev["V"]))
            A, W, U = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], 64, method=m, cu_seqlens=cuq, out=out)
            torch.cuda.synchronize()
            assert bnd.last_device_status() == 0
            a = A.cpu().numpy()
            assert not np.isnan(a).any() and structure_errors(a, inp) == (0, 0)
            assert max_ratio(a, A_ref) <= TOL_A[wl.BF16] and max_residual(a, N_ref, inp) <= TOL_RES[wl.BF16]
            w, u = bnd.to_numpy_f64(W), bnd.to_numpy_f64(U)
            assert not np.isnan(w).any() and not np.isnan(u).any()
            assert max_ratio(w, W_ref) <= 1e-2 and max_ratio(u, U_ref) <= 1e-2
        A_only = bnd.build(dev["K"], dev["beta"], dev["g"], 64, cu_seqlens=cuq)
        W2, U2 = bnd.wy(A_only, dev["K"], dev["V"], dev["beta"], cu_seqlens=cuq)
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        assert max_ratio(A_only.cpu().numpy(), A_ref) <= TOL_A[wl.BF16]
        assert max_ratio(bnd.to_numpy_f64(W2), W_ref) <= 1e-2 and max_ratio(bnd.to_numpy_f64(U2), U_ref) <= 1e-2
        # the CUDA-core kernel, which served this shape before, agrees within the two paths' rounding
        A_simt, W_simt, U_simt = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], 64, method=bnd.FORCE_SIMT, cu_seqlens=cuq)
        torch.cuda.synchronize()
        assert float((A_simt - A).abs().max()) <= 4e-3 * float(A_simt.abs().max())
