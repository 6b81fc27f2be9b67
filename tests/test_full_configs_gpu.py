"""Parity at the full sizes of the five configurations, in the launch configuration bench.py times
(one fused call over the whole batch).  The structure of A is checked on every element on the
device; values of EVERY chunk matrix of every configuration are compared with the fp64 oracle, for each
of the three schemes (the oracle runs slab by slab along the tokens to bound host memory).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_21325_b200 import workloads as wl
from parity_util import max_ratio, max_residual, paper_metrics

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


def device_structure_check(A, inp):
    """Upper triangle all-bits-zero and diagonal exactly 1.0f over the whole tensor, on the device."""
    B, T, H, C = A.shape
    loc = torch.zeros(B * T, dtype=torch.int64)
    for t0, r in inp.chunk_list():
        loc[t0:t0 + r] = torch.arange(r)
    loc = loc.cuda().view(B, T, 1, 1)
    cols = torch.arange(C, device="cuda").view(1, 1, 1, C)
    bits = A.view(torch.int32)
    assert int(torch.count_nonzero(bits * (cols > loc))) == 0, "upper triangle is not bit-exact +0.0"
    diag = torch.gather(A, 3, loc.expand(B, T, H, 1))
    assert bool((diag == 1.0).all()), "diagonal is not exactly 1.0f"
    assert not bool(torch.isnan(A).any())


def sample_ranges(inp, n=6):
    """Token ranges made of whole chunks: first, last and a few in between (dense configs)."""
    chunks = inp.T // inp.C
    picks = sorted(set([0, chunks - 1] + [int(x) for x in np.linspace(0, chunks - 1, n)]))
    return [(c * inp.C, (c + 1) * inp.C) for c in picks]


def run_full(bnd, inp, method):
    dev = bnd.to_device(inp)
    A = torch.full((inp.B, inp.T, inp.H, inp.C), float("nan"), dtype=torch.float32, device="cuda")
    W = torch.full(dev["K"].shape, float("nan"), dtype=dev["K"].dtype, device="cuda")
    U = torch.full(dev["V"].shape, float("nan"), dtype=dev["V"].dtype, device="cuda")
    bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], inp.C, method=method, cu_seqlens=inp.cu_seqlens, out=(A, W, U))
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    return A, W, U


SLAB = 4096   # tokens per oracle call: bounds the fp64 host copies at the 32k-token configuration

_ref_cache = {}


def oracle_slabs(inp):
    """fp64 oracle results for EVERY chunk matrix of a dense configuration, slab by slab along the
    tokens (whole chunks per slab).  Cached per workload so that the schemes share one oracle run."""
    if inp.name not in _ref_cache:
        out = []
        for t0 in range(0, inp.T, SLAB):
            sl = slice(t0, min(t0 + SLAB, inp.T))
            A_ref, N_ref = oracle.build_A(inp.K[:, sl], inp.beta[:, sl], inp.g[:, sl], inp.C, return_N=True)
            W_ref, U_ref = oracle.wy(A_ref, inp.K[:, sl], inp.V[:, sl], inp.beta[:, sl], inp.C)
            out.append((sl, A_ref, N_ref, W_ref, U_ref))
        _ref_cache.clear()       # one workload's references at a time (config 3's are gigabytes)
        _ref_cache[inp.name] = out
    return _ref_cache[inp.name]


def compare_everything(bnd, inp, A, W, U):
    """Every chunk matrix of the batch against the oracle: the ratios are max |x - ref| / max |ref| over the
    WHOLE tensor (numerators and denominators accumulated over the slabs), the residual is the worst chunk's."""
    num = {"A": 0.0, "W": 0.0, "U": 0.0}
    den = {"A": 0.0, "W": 0.0, "U": 0.0}
    res, n_mat = 0.0, 0
    for sl, A_ref, N_ref, W_ref, U_ref in oracle_slabs(inp):
        a = A[:, sl].cpu().numpy()
        sub = wl.Inputs("s", inp.B, sl.stop - sl.start, inp.H, inp.d_k, inp.d_v, inp.C, inp.kv_dtype, inp.K[:, sl], inp.V[:, sl],
                        inp.beta[:, sl], inp.g[:, sl])
        n_mat += sub.n_matrices
        res = max(res, max_residual(a, N_ref, sub))
        for key, x, ref in (("A", a.astype(np.float64), A_ref), ("W", bnd.to_numpy_f64(W[:, sl]), W_ref),
                            ("U", bnd.to_numpy_f64(U[:, sl]), U_ref)):
            num[key] = max(num[key], float(np.abs(x - ref).max()))
            den[key] = max(den[key], float(np.abs(ref).max()))
    assert n_mat == inp.n_matrices
    return {"A": num["A"] / den["A"], "W": num["W"] / den["W"], "U": num["U"] / den["U"], "res": res, "matrices": n_mat}


SCHEMES = (("block_recursive", 0), ("mixed_recursion", 0x100), ("product_series", 1))


@pytest.mark.parametrize("cfg", [1, 2, 3, 4])
def test_dense_config_full_size_every_matrix_every_scheme(bnd, cfg):
    """All chunk matrices of the configuration (not a sample), for the block recursion, the mixed recursion
    and the product series, in the one-launch shape bench.py times."""
    inp = wl.config(cfg)
    report = {}
    schemes = SCHEMES + ((("product_series_f16", 1 | 0x400),) if inp.kv_dtype == wl.BF16 else ())   # fp16 operands: tensor-core kernel only
    for name, m in schemes:
        A, W, U = run_full(bnd, inp, m)
        device_structure_check(A, inp)
        assert not bool(torch.isnan(W.float()).any()) and not bool(torch.isnan(U.float()).any())
        worst = compare_everything(bnd, inp, A, W, U)
        report[name] = worst
        assert worst["matrices"] == inp.n_matrices
        assert worst["A"] <= TOL_A[inp.kv_dtype], (name, worst)
        assert worst["res"] <= TOL_RES[inp.kv_dtype], (name, worst)
        assert worst["W"] <= TOL_WY[inp.kv_dtype] and worst["U"] <= TOL_WY[inp.kv_dtype], (name, worst)
    print("config %d, every matrix, errors per scheme:" % cfg, report)


def test_split_calls_full_size_every_matrix(bnd):
    """tri_inv_build and tri_inv_wy as separate launches on configuration 2: every matrix against the oracle."""
    inp = wl.config(2)
    dev = bnd.to_device(inp)
    A = torch.full((inp.B, inp.T, inp.H, inp.C), float("nan"), dtype=torch.float32, device="cuda")
    bnd.build(dev["K"], dev["beta"], dev["g"], inp.C, out=A)
    W = torch.full(dev["K"].shape, float("nan"), dtype=dev["K"].dtype, device="cuda")
    U = torch.full(dev["V"].shape, float("nan"), dtype=dev["V"].dtype, device="cuda")
    bnd.wy(A, dev["K"], dev["V"], dev["beta"], out=(W, U))
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    device_structure_check(A, inp)
    worst = compare_everything(bnd, inp, A, W, U)
    assert worst["A"] <= 2e-3 and worst["res"] <= 5e-3 and worst["W"] <= 1e-2 and worst["U"] <= 1e-2, worst


def test_config5_ragged_full_size_per_method(bnd):
    """64 packed sequences, un-normalised keys, beta near 1, no decay: error against the oracle per method."""
    inp = wl.config(5)
    A_ref, N_ref = oracle.build_A(inp.K, inp.beta, inp.g, inp.C, cu_seqlens=inp.cu_seqlens, return_N=True)
    W_ref, U_ref = oracle.wy(A_ref, inp.K, inp.V, inp.beta, inp.C, cu_seqlens=inp.cu_seqlens)
    report = {}
    for name, m in (("block_recursive", bnd.BLOCK_RECURSIVE), ("mixed_recursion", bnd.BLOCK_RECURSIVE | bnd.LEAF_SERIES),
                    ("product_series", bnd.PRODUCT_SERIES)):
        A, W, U = run_full(bnd, inp, m)
        device_structure_check(A, inp)
        a = A.cpu().numpy()
        report[name] = dict(paper_metrics(a, A_ref), ratio=max_ratio(a, A_ref), residual=max_residual(a, N_ref, inp),
                            W=max_ratio(bnd.to_numpy_f64(W), W_ref), U=max_ratio(bnd.to_numpy_f64(U), U_ref))
        assert report[name]["ratio"] <= 2e-3 and report[name]["residual"] <= 5e-3, (name, report[name])
        assert report[name]["W"] <= 1e-2 and report[name]["U"] <= 1e-2, (name, report[name])
    print("config 5 errors per method:", report)


def test_adversarial_keys_report(bnd):
    """Correlated keys make ||N|| large: the block recursion stays within tolerance, the product series
    loses accuracy (Sec. 3.2).  Only the stable scheme is gated; the series' error is reported."""
    report = {}
    for rho, d_eff in ((0.5, None), (0.9, None), (0.0, 4)):
        inp = wl.correlated_keys_case(1, 4096, 4, 128, 64, wl.BF16, rho, seed=55, d_eff=d_eff)
        A_ref = oracle.build_A(inp.K, inp.beta, inp.g, inp.C)
        for name, m in (("block_recursive", bnd.BLOCK_RECURSIVE), ("product_series", bnd.PRODUCT_SERIES)):
            A, _, _ = run_full(bnd, inp, m)
            report[(inp.name, name)] = max_ratio(A.cpu().numpy(), A_ref)
        assert report[(inp.name, "block_recursive")] <= 2e-3, report
    print("adversarial keys, max ratio per method:", report)


@pytest.mark.parametrize("cfg", [2, 3, 5])
def test_wy_alone_reproduces_the_fused_call_at_full_size(bnd, cfg):
    """tri_inv_wy on the A that tri_inv_build stored gives, bit for bit, the W and U of the fused call (the same kernel
    with the matrix loaded instead of built), on every token of the large configurations -- also in place, with the keys
    in the buffer that receives W (the form tri_inv_fused_kda uses).  The matrix is loaded into the space that the output
    staging tiles of the item before live in: the stores that read them must be through first."""
    inp = wl.config(cfg)
    dev = bnd.to_device(inp)
    cu = inp.cu_seqlens
    _, W_ref, U_ref = bnd.fused(dev["K"], dev["V"], dev["beta"], dev["g"], inp.C, cu_seqlens=cu, want_A=False)
    A = bnd.build(dev["K"], dev["beta"], dev["g"], inp.C, cu_seqlens=cu)
    for in_place in (False, True):
        for _ in range(3):
            W = dev["K"].clone() if in_place else torch.full_like(dev["K"], float("nan"))
            U = torch.full_like(dev["V"], float("nan"))
            bnd.wy(A, W if in_place else dev["K"], dev["V"], dev["beta"], cu_seqlens=cu, out=(W, U))
            torch.cuda.synchronize()
            assert bnd.last_device_status() == 0
            assert torch.equal(W.view(torch.int16), W_ref.view(torch.int16)) and torch.equal(U.view(torch.int16), U_ref.view(torch.int16))


@pytest.mark.parametrize("cfg", [2, 3, 4], ids=["config2_C64", "config3_C64", "config4_C128"])
def test_per_channel_decay_full_size(bnd, cfg):
    """tri_inv_fused_kda on the shapes of config 2 (4096 matrices of 64 tokens) and config 4 (2048 of 128), the launches
    bench.py --call kda_fused times: structure on every element, EVERY matrix's A, W and U against the fp64 oracle, and -- at
    any size -- a gate that is the same on every channel must reproduce tri_inv_build's matrices within the rounding of the
    two bf16 operand copies."""
    inp = wl.config(cfg)
    G = wl.per_channel_gate(inp, seed=3000 + cfg)
    dev = bnd.to_device(inp)
    Gd = torch.from_numpy(G).cuda()
    A = torch.full((inp.B, inp.T, inp.H, inp.C), float("nan"), dtype=torch.float32, device="cuda")
    W, U = torch.full_like(dev["K"], float("nan")), torch.full_like(dev["V"], float("nan"))
    bnd.fused_kda(dev["K"], dev["V"], Gd, dev["beta"], inp.C, out=(A, W, U))
    torch.cuda.synchronize()
    assert bnd.last_device_status() == 0
    device_structure_check(A, inp)
    A_ref, N_ref = oracle.build_A_kda(inp.K, G, inp.beta, inp.C, return_N=True)
    a = A.cpu().numpy()
    assert max_ratio(a, A_ref) <= TOL_A[wl.BF16] and max_residual(a, N_ref, inp) <= TOL_RES[wl.BF16]
    Kg = wl.bf16_bits_to_f32(inp.K).astype(np.float64) * np.exp(G.astype(np.float64))
    W_ref, _ = oracle.wy(A_ref, Kg, None, inp.beta, inp.C)
    _, U_ref = oracle.wy(A_ref, inp.K, inp.V, inp.beta, inp.C)
    assert max_ratio(bnd.to_numpy_f64(W), W_ref) <= 1e-2 and max_ratio(bnd.to_numpy_f64(U), U_ref) <= 1e-2
    Gc = dev["g"].unsqueeze(-1).expand(-1, -1, -1, inp.d_k).contiguous()
    A_same = bnd.build_kda(dev["K"], Gc, dev["beta"], inp.C)
    A_scalar = bnd.build(dev["K"], dev["beta"], dev["g"], inp.C)
    torch.cuda.synchronize()
    assert float((A_same - A_scalar).abs().max()) <= 2e-3 * float(A_scalar.abs().max())


def test_per_channel_fused_call_on_the_ragged_configuration_repeats_bit_for_bit(bnd):
    """tri_inv_fused_kda (one kernel at C = 64) on config 5, whose 160 sequences end inside chunks: EVERY matrix's A, W and U
    against the fp64 oracle, nothing written past a sequence's end, and three calls into fresh buffers give the same bits
    (the kernel's staging tiles share their space with the operand tiles of the item before and after)."""
    inp = wl.config(5)
    cu = inp.cu_seqlens
    G = wl.per_channel_gate(inp, seed=3005)
    dev = bnd.to_device(inp)
    Gd = torch.from_numpy(G).cuda()
    outs = []
    for _ in range(3):
        A = torch.full((inp.B, inp.T, inp.H, inp.C), float("nan"), dtype=torch.float32, device="cuda")
        W, U = torch.full_like(dev["K"], float("nan")), torch.full_like(dev["V"], float("nan"))
        bnd.fused_kda(dev["K"], dev["V"], Gd, dev["beta"], inp.C, cu_seqlens=cu, out=(A, W, U))
        torch.cuda.synchronize()
        assert bnd.last_device_status() == 0
        outs.append((A, W, U))
    for A, W, U in outs[1:]:
        assert torch.equal(A.view(torch.int32), outs[0][0].view(torch.int32))
        assert torch.equal(W.view(torch.int16), outs[0][1].view(torch.int16)) and torch.equal(U.view(torch.int16), outs[0][2].view(torch.int16))
    A, W, U = outs[0]
    assert not torch.isnan(A).any() and not torch.isnan(W).any() and not torch.isnan(U).any()
    A_ref, N_ref = oracle.build_A_kda(inp.K, G, inp.beta, inp.C, cu_seqlens=cu, return_N=True)
    device_structure_check(A, inp)
    a = A.cpu().numpy()
    assert max_ratio(a, A_ref) <= TOL_A[wl.BF16] and max_residual(a, N_ref, inp) <= TOL_RES[wl.BF16]
    Kg = wl.bf16_bits_to_f32(inp.K).astype(np.float64) * np.exp(G.astype(np.float64))
    W_ref, _ = oracle.wy(A_ref, Kg, None, inp.beta, inp.C, cu_seqlens=cu)
    _, U_ref = oracle.wy(A_ref, inp.K, inp.V, inp.beta, inp.C, cu_seqlens=cu)
    assert max_ratio(bnd.to_numpy_f64(W), W_ref) <= 1e-2 and max_ratio(bnd.to_numpy_f64(U), U_ref) <= 1e-2
