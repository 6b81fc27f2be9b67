"""Pins for the fp64 oracle: it is checked against things other than itself.

Closed forms worked by hand, the paper's own examples (Sec. 3.2), exact
rational arithmetic, LAPACK, the defining identities, the |A_ij| <= 1
invariant of DeltaNet matrices (Sec. 2.2) and the sequential delta-rule
recurrence the chunk form was derived from.
"""
import os
from fractions import Fraction
from math import comb

import numpy as np
import pytest

import oracle
from oracle import algorithms as alg
from paper_2605_21325_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def load(name):
    return np.loadtxt(os.path.join(GOLD, name), comments="#")


def keys_for_integer_N(N):
    """Integer keys k_i (d = n) with k_i . k_j = N_ij for j < i: row i solves a unit
    lower-triangular integer system against the earlier rows, so it stays integral."""
    n = N.shape[0]
    K = np.zeros((n, n))
    for i in range(n):
        K[i, i] = 1.0
        for j in range(i):
            K[i, j] = N[i, j] - sum(K[i, m] * K[j, m] for m in range(j))
    return K


def run_single(K, beta=None, g=None, C=None, dtype=np.float32):
    """Oracle on one sequence, one head; returns (A, N) as [T, C] arrays."""
    T, d = K.shape
    C = T if C is None else C
    beta = np.ones(T) if beta is None else beta
    g = np.zeros(T) if g is None else g
    A, N = oracle.build_A(K.reshape(1, T, 1, d).astype(dtype), np.asarray(beta, np.float32).reshape(1, T, 1),
                          np.asarray(g, np.float32).reshape(1, T, 1), C, return_N=True)
    return A[0, :, 0, :], N[0, :, 0, :]


# ---------------------------------------------------------------- closed forms (hand-worked)

def test_closed_form_2x2_and_3x3():
    # k0=(1,0), k1=(1,1): k1.k0 = 1; beta1 = 0.5; g1-g0 = -ln 2  =>  n21 = 0.25, A21 = -0.25
    K = np.array([[1.0, 0.0], [1.0, 1.0]])
    A, N = run_single(K, beta=[1.0, 0.5], g=[0.0, -np.log(2.0)])
    assert abs(N[1, 0] - 0.25) < 1e-7          # g is stored in fp32
    assert A[0, 0] == 1.0 and A[1, 1] == 1.0 and A[0, 1] == 0.0
    assert abs(A[1, 0] + 0.25) < 1e-7
    # 3x3 with integer N: n21=2, n31=-1, n32=3  =>  A21=-2, A32=-3, A31 = n32 n21 - n31 = 7
    N3 = np.array([[0, 0, 0], [2, 0, 0], [-1, 3, 0]], float)
    A, N = run_single(keys_for_integer_N(N3))
    assert np.array_equal(N, N3)
    assert np.array_equal(A, np.array([[1, 0, 0], [-2, 1, 0], [7, -3, 1]], float))


def test_closed_form_4x4_golden():
    G = load("closed_form_4x4.txt")
    N4, A4 = G[:4], G[4:]
    A, N = run_single(keys_for_integer_N(N4))
    assert np.array_equal(N, N4)
    assert np.array_equal(A, A4)


def test_first_difference_matrix():
    # all keys equal one unit vector, beta = 1, g = 0: N = ones strictly lower
    K = np.zeros((5, 3)); K[:, 1] = 1.0
    A, N = run_single(K)
    assert np.array_equal(N, np.tril(np.ones((5, 5)), -1))
    assert np.array_equal(A, load("first_difference_n5.txt"))
    inp = wl.first_difference_case(2, 128, 2, 16, 64, wl.BF16)
    A = oracle.build_A(inp.K, inp.beta, inp.g, 64)
    exp = np.eye(64) - np.eye(64, k=-1)
    for b in range(2):
        for c in range(2):
            assert np.array_equal(A[b, c * 64:(c + 1) * 64, 1, :], exp)


def test_growth_example_powers_of_two():
    # Sec. 3.2: N = -(ones strictly lower)  =>  A_ij = sum_k binom(i-j-1, k-1) = 2^(i-j-1)
    K = np.zeros((6, 2)); K[:, 0] = 1.0
    A, N = run_single(K, beta=-np.ones(6))
    assert np.array_equal(A, load("growth_example_n6.txt"))
    n = 128
    K = np.zeros((n, 2)); K[:, 0] = 1.0
    A, _ = run_single(K, beta=-np.ones(n))
    i, j = np.tril_indices(n, -1)
    assert np.array_equal(A[i, j], 2.0 ** (i - j - 1))      # exact in fp64 up to 2^126


def test_series_terms_are_binomials():
    # pins the series/product code used below, against the paper's closed form
    n = 6
    Lm = np.tril(np.ones((n, n)), -1)
    assert np.array_equal(np.linalg.matrix_power(Lm, 3), load("ones_power3_n6.txt"))
    n = 16
    Lm = np.tril(np.ones((n, n)), -1)
    for k in (1, 2, 5, 8):
        P = np.linalg.matrix_power(Lm, k)
        for i in range(n):
            for j in range(n):
                expect = comb(i - j - 1, k - 1) if i > j else 0
                assert P[i, j] == expect
    # repeated squaring on the same matrix (negated) gives the growth example
    X = alg.mch(-Lm)
    i, j = np.tril_indices(n, -1)
    assert np.array_equal(X[i, j], 2.0 ** (i - j - 1))


# ---------------------------------------------------------------- exact rational brute force

def exact_inverse(N):
    n = len(N)
    M = [[Fraction(int(i == j)) + Fraction(N[i][j]) for j in range(n)] for i in range(n)]
    X = [[Fraction(int(i == j)) for j in range(n)] for i in range(n)]
    for i in range(n):                      # Gauss-Jordan, no pivoting needed (unit diagonal)
        for r in range(n):
            if r != i and M[r][i] != 0:
                f = M[r][i]
                M[r] = [a - f * b for a, b in zip(M[r], M[i])]
                X[r] = [a - f * b for a, b in zip(X[r], X[i])]
    return X


@pytest.mark.parametrize("n,seed", [(2, 0), (3, 1), (5, 2), (8, 3)])
def test_exact_rational_brute_force(n, seed):
    rng = np.random.default_rng(seed)
    K = rng.integers(-2, 3, size=(n, 4)).astype(np.float64)
    beta = rng.choice([0.5, 1.0, -1.0, 2.0], size=n)
    A, N = run_single(K, beta=beta)
    S = K @ K.T
    Nx = [[Fraction(beta[i]) * Fraction(int(S[i, j])) if j < i else Fraction(0) for j in range(n)] for i in range(n)]
    X = exact_inverse(Nx)
    for i in range(n):
        for j in range(n):
            assert float(Nx[i][j]) == N[i, j]
            ref = float(X[i][j])
            assert abs(A[i, j] - ref) <= 1e-12 * max(1.0, abs(ref))


# ---------------------------------------------------------------- identities on model-like inputs

@pytest.fixture(scope="module")
def small_gdn():
    inp = wl.make("t", 2, 192, 3, 32, 48, 64, wl.BF16, seed=7)
    A, N = oracle.build_A(inp.K, inp.beta, inp.g, inp.C, return_N=True)
    W, U = oracle.wy(A, inp.K, inp.V, inp.beta, inp.C)
    return inp, A, N, W, U


def chunks_of(inp):
    for t0, r in inp.chunk_list():
        b, t = divmod(t0, inp.T)
        for h in range(inp.H):
            yield b, t, h, r


def test_residual_unit_diagonal_zero_upper(small_gdn):
    inp, A, N, _, _ = small_gdn
    C = inp.C
    for b, t, h, r in chunks_of(inp):
        a, n = A[b, t:t + r, h, :r], N[b, t:t + r, h, :r]
        I = np.eye(r)
        assert np.abs((I + n) @ a - I).max() <= 1e-12
        assert np.abs(a @ (I + n) - I).max() <= 1e-12
        assert np.array_equal(np.diag(a), np.ones(r))
        iu = np.triu_indices(r, 1)
        assert not a[iu].any() and not np.signbit(a[iu]).any()
        assert not n[np.triu_indices(r, 0)].any()


def test_N_matches_definition_and_lapack(small_gdn):
    inp, A, N, _, _ = small_gdn
    Kf = inp.kv_as_f32("K").astype(np.float64)
    for b, t, h, r in chunks_of(inp):
        n = alg.chunk_N(Kf[b, t:t + r, h], inp.beta[b, t:t + r, h], inp.g[b, t:t + r, h])
        assert np.abs(n - N[b, t:t + r, h, :r]).max() <= 1e-15
        ref = np.linalg.inv(np.eye(r) + n)
        assert np.abs(ref - A[b, t:t + r, h, :r]).max() <= 1e-12


def test_entries_bounded_by_one_and_condition_number(small_gdn):
    # Sec. 2.2: inverse of a DeltaNet matrix has entries in [-1,1]; kappa_2 <= n^2 (Cor. 2.1).
    # bf16 storage rounding moves |k| off 1 by <= 2^-9, so allow that slack.
    inp, A, N, _, _ = small_gdn
    assert np.abs(A).max() <= 1.0 + 1e-2
    for b, t, h, r in chunks_of(inp):
        assert np.linalg.cond(np.eye(r) + N[b, t:t + r, h, :r], 2) <= r * r
    for seed in range(3):
        x = wl.make("u", 1, 128, 2, 128, 128, 128, wl.F32, seed=100 + seed)
        x.g[:] = 0                                      # ungated DeltaNet, unit keys, beta in (0,1)
        a = oracle.build_A(x.K, x.beta, x.g, 128)
        assert np.abs(a).max() <= 1.0 + 1e-5


def test_wy_solve_identities(small_gdn):
    inp, A, N, W, U = small_gdn
    Kf = inp.kv_as_f32("K").astype(np.float64)
    Vf = inp.kv_as_f32("V").astype(np.float64)
    for b, t, h, r in chunks_of(inp):
        n = N[b, t:t + r, h, :r]
        bt = inp.beta[b, t:t + r, h].astype(np.float64)[:, None]
        assert np.abs((np.eye(r) + n) @ W[b, t:t + r, h] - bt * Kf[b, t:t + r, h]).max() <= 1e-12
        assert np.abs((np.eye(r) + n) @ U[b, t:t + r, h] - bt * Vf[b, t:t + r, h]).max() <= 1e-12
        # row recurrence w_i = beta_i k_i - sum_{j<i} N_ij w_j
        w = np.zeros((r, inp.d_k))
        for i in range(r):
            w[i] = bt[i] * Kf[b, t + i, h] - n[i, :i] @ w[:i]
        assert np.abs(w - W[b, t:t + r, h]).max() <= 1e-12


def test_delta_rule_recurrence(small_gdn):
    """Sequential gated delta rule, token by token (O(C d^2), no matrix inverse):
         S_t = a_t S_{t-1} (I - beta_t k_t k_t^T) + beta_t v_t k_t^T,   a_t = exp(g_t - g_{t-1}), S_0 = 0
       equals sum_t exp(g_last - g_t) u_t k_t^T with U from the oracle; and, without decay,
       prod_t (I - beta_t k_t k_t^T) = I - W^T K.  This ties N's conventions (beta on rows,
       exp(g_i - g_j), + sign) to the model the chunk form came from."""
    inp, A, N, W, U = small_gdn
    Kf = inp.kv_as_f32("K").astype(np.float64)
    Vf = inp.kv_as_f32("V").astype(np.float64)
    for b, t, h, r in list(chunks_of(inp))[:6]:
        k, v = Kf[b, t:t + r, h], Vf[b, t:t + r, h]
        bt = inp.beta[b, t:t + r, h].astype(np.float64)
        g = inp.g[b, t:t + r, h].astype(np.float64)
        S = np.zeros((inp.d_v, inp.d_k))
        P = np.eye(inp.d_k)
        for i in range(r):
            a = np.exp(g[i] - (g[i - 1] if i else g[0]))     # first token's own decay cancels from S_0 = 0
            S = a * (S - bt[i] * np.outer(S @ k[i], k[i])) + bt[i] * np.outer(v[i], k[i])
            P = a * (P - bt[i] * np.outer(P @ k[i], k[i]))
        u = U[b, t:t + r, h]
        S_chunk = sum(np.exp(g[r - 1] - g[i]) * np.outer(u[i], k[i]) for i in range(r))
        assert np.abs(S - S_chunk).max() <= 1e-12
        # decayed transition: P = e^{g_last - g_0}... written with omega = A diag(beta e^{g}) K
        a_mat = A[b, t:t + r, h, :r]
        omega = a_mat @ ((bt * np.exp(g - g[0]))[:, None] * k)
        P_chunk = np.exp(g[r - 1] - g[0]) * np.eye(inp.d_k) - sum(np.exp(g[r - 1] - g[i]) * np.outer(omega[i], k[i]) for i in range(r))
        assert np.abs(P - P_chunk).max() <= 1e-12
    # ungated: ordered product of Householder-like factors equals I - W^T K
    x = wl.make("v", 1, 64, 1, 16, 16, 64, wl.F32, seed=11)
    x.g[:] = 0
    a = oracle.build_A(x.K, x.beta, x.g, 64)
    w, _ = oracle.wy(a, x.K, x.V, x.beta, 64)
    k = x.K[0, :, 0].astype(np.float64)
    P = np.eye(16)
    for i in range(64):
        P = P - float(x.beta[0, i, 0]) * np.outer(P @ k[i], k[i])
    assert np.abs(P - (np.eye(16) - w[0, :, 0].T @ k)).max() <= 1e-12


# ---------------------------------------------------------------- the paper's algorithms reach the same matrix

@pytest.mark.parametrize("n", [2, 4, 8, 16, 64, 128])
def test_algorithms_agree_with_substitution(n):
    x = wl.make("w", 1, n, 1, 128, 8, n, wl.F32, seed=20 + n)
    A, N = oracle.build_A(x.K, x.beta, x.g, n, return_N=True)
    a, L = A[0, :, 0], N[0, :, 0]
    assert np.abs(alg.forward_substitution(L) - a).max() <= 1e-14
    if n <= 16:
        assert np.abs(alg.neumann_series(L) - a).max() <= 1e-13
    assert np.abs(alg.mch(L) - a).max() <= 1e-13           # Alg. 5
    assert np.abs(alg.product_form(L) - a).max() <= 1e-13  # factorised series
    assert np.abs(alg.mbh(L) - a).max() <= 1e-13           # Alg. 4 from b0 = 1
    assert np.abs(alg.mxr(L, 16) - a).max() <= 1e-13       # Alg. 2
    assert np.abs(alg.block_recursive(L, 16) - a).max() <= 1e-13
    if n >= 4:
        h = n // 2                                         # 2x2 block formula from two half-size oracle inverses
        X11 = oracle.build_A(x.K[:, :h], x.beta[:, :h], x.g[:, :h], h)[0, :, 0]
        X22 = oracle.build_A(x.K[:, h:], x.beta[:, h:], x.g[:, h:], h)[0, :, 0]
        assert np.abs(a[:h, :h] - X11).max() <= 1e-14 and np.abs(a[h:, h:] - X22).max() <= 1e-14
        assert np.abs(a[h:, :h] + X22 @ L[h:, :h] @ X11).max() <= 1e-13


# ---------------------------------------------------------------- layout: ragged packing, partial chunks, heads

def test_ragged_and_partial_chunks_match_per_sequence_runs():
    rng = np.random.default_rng(5)
    cu = np.array([0, 1, 70, 134, 200], np.int32)          # lengths 1, 69, 64, 66
    x = wl.make("r", 1, int(cu[-1]), 2, 16, 8, 64, wl.BF16, seed=31, kind="stress", cu_seqlens=cu, rng=rng)
    x.g[:] = (rng.standard_normal(x.g.shape) * 0.1).astype(np.float32)
    A = oracle.build_A(x.K, x.beta, x.g, 64, cu_seqlens=cu)
    W, U = oracle.wy(A, x.K, x.V, x.beta, 64, cu_seqlens=cu)
    for s in range(4):
        b, e = int(cu[s]), int(cu[s + 1])
        As = oracle.build_A(x.K[:, b:e], x.beta[:, b:e], x.g[:, b:e], 64)
        Ws, Us = oracle.wy(As, x.K[:, b:e], x.V[:, b:e], x.beta[:, b:e], 64)
        assert np.array_equal(As, A[:, b:e]) and np.array_equal(Ws, W[:, b:e]) and np.array_equal(Us, U[:, b:e])
    # the 69-token sequence: second chunk has 5 real rows; columns >= 5 of those rows are zero
    assert not A[0, 65:70, :, 5:].any()
    assert np.array_equal(A[0, 65, 0, :1], [1.0])
    # heads are independent: permuting heads permutes outputs
    A2 = oracle.build_A(x.K[:, :, ::-1], x.beta[:, :, ::-1], x.g[:, :, ::-1], 64, cu_seqlens=cu)
    assert np.array_equal(A2[:, :, ::-1], A)


def test_threads_do_not_change_results():
    x = wl.config(2, shrink=32)
    a1 = oracle.build_A(x.K, x.beta, x.g, x.C, n_threads=1)
    a4 = oracle.build_A(x.K, x.beta, x.g, x.C, n_threads=4)
    assert np.array_equal(a1, a4)


# ---------------------------------------------------------------- iterative schemes (Alg. 3, Alg. 6)

def test_newton_schulz_and_refinement_converge_to_substitution():
    x = wl.make("ns", 1, 64, 1, 128, 8, 64, wl.F32, seed=91)
    A, N = oracle.build_A(x.K, x.beta, x.g, 64, return_N=True)
    a, L = A[0, :, 0], N[0, :, 0]
    err = {m: np.linalg.norm(alg.newton_schulz(L, m) - a) / np.linalg.norm(a) for m in (6, 8, 10, 12, 14)}
    # Sec. 4.2: six iterations are not enough at C = 64, twelve are, more add nothing
    assert err[6] > 1e-2 and err[10] < 1e-4 and err[12] < 1e-12 and err[14] < 1e-12
    assert err[6] > err[8] > err[10] > err[12]
    # the default count is 2 log2(n)
    assert np.abs(alg.newton_schulz(L) - a).max() < 1e-12
    # one refinement step squares the residual: it equals one more Newton-Schulz round
    x8 = alg.newton_schulz(L, 8)
    assert np.abs(alg.iterative_refinement(x8, L) - alg.newton_schulz(L, 9)).max() < 1e-12
    r0 = np.abs(np.eye(64) - x8 @ (np.eye(64) + L)).max()
    r1 = np.abs(np.eye(64) - alg.iterative_refinement(x8, L) @ (np.eye(64) + L)).max()
    assert r1 < 64 * r0 * r0
    # refinement leaves an exact inverse unchanged
    assert np.abs(alg.iterative_refinement(a, L) - a).max() < 1e-14


# ---------------------------------------------------------------- raw front end (sigmoid, log-sigmoid + chunk cumsum, key norm)

def test_raw_front_end_hand_values_and_generator_recipe():
    # hand values: sigmoid(0) = 1/2, log sigmoid(0) = -ln 2, (3,4) / 5 = (0.6, 0.8)
    K = np.array([[3.0, 4.0], [0.0, 2.0], [0.0, 0.0]], np.float32).reshape(1, 3, 1, 2)
    Kh, b, g = oracle.raw_front_end(K, np.zeros((1, 3, 1)), np.zeros((1, 3, 1)), 2)
    assert np.allclose(Kh[0, :, 0], [[0.6, 0.8], [0.0, 1.0], [0.0, 0.0]], atol=1e-15)   # a zero key stays zero
    assert np.array_equal(b[0, :, 0], [0.5, 0.5, 0.5])
    assert np.allclose(g[0, :, 0], [-np.log(2), -2 * np.log(2), -np.log(2)], atol=1e-15)  # the sum restarts at the chunk (C = 2)
    # large |logit|: no overflow, log sigmoid(-50) = -50 - log1p(e^-50), log sigmoid(50) = -e^-50
    _, b, g = oracle.raw_front_end(K, np.array([50.0, -50.0, 0.0]).reshape(1, 3, 1), np.array([-50.0, 50.0, 0.0]).reshape(1, 3, 1), 4)
    assert abs(b[0, 0, 0] - 1.0) < 1e-15 and 0 < b[0, 1, 0] < 1e-20
    assert abs(g[0, 0, 0] + 50.0) < 1e-12 and abs(g[0, 1, 0] + 50.0) < 1e-12
    # the generator of the configurations applies the same recipe (in fp32): same A up to fp32 rounding
    raw = wl.make_raw("raw", 2, 160, 2, 32, 64, wl.F32, seed=17)
    Kh, b, g = oracle.raw_front_end(raw.K, raw.beta, raw.g, 64)
    assert np.abs(np.linalg.norm(Kh, axis=-1) - 1).max() < 1e-12
    assert (np.diff(g.reshape(2, 160, 2)[:, :64], axis=1) <= 0).all()       # log-decays are negative inside a chunk
    rng = np.random.default_rng(17)                                          # wl.make draws K, V, beta, g noise in this order
    ref = wl.make("prep", 2, 160, 2, 32, 32, 64, wl.F32, seed=17, rng=rng)
    assert np.abs(oracle.build_A(Kh, b, g, 64) - oracle.build_A(ref.K, ref.beta, ref.g, 64)).max() < 5e-6
    # ragged: the sum restarts at every sequence and chunk
    cu = np.array([0, 70, 160], np.int32)
    raw1 = wl.make_raw("raw", 1, 160, 2, 32, 64, wl.F32, seed=18, cu_seqlens=cu)
    _, _, g = oracle.raw_front_end(raw1.K, raw1.beta, raw1.g, 64, cu_seqlens=cu)
    z = raw1.g.astype(np.float64)
    ls = np.minimum(z, 0) - np.log1p(np.exp(-np.abs(z)))
    for t in (0, 64, 70, 134):
        assert np.allclose(g[0, t], ls[0, t], atol=1e-15)
    assert np.allclose(g[0, 69], ls[0, 64:70].sum(axis=0), atol=1e-13)


# ---------------------------------------------------------------- per-channel decay (KDA row of Table 1)

def test_per_channel_decay_reduces_to_the_scalar_gate_and_to_deltanet():
    # (the numpy + LAPACK statement, which takes G in fp64; the C statement, which reads G in fp32 as the library does, is
    # held against it in test_per_channel_chunk_form_equals_its_recurrence)
    x = wl.make("kda", 2, 150, 2, 16, 16, 64, wl.BF16, seed=33)
    # Gamma = 1: plain DeltaNet matrix (g = 0)
    A0 = oracle.build_A_kda_numpy(x.K, np.zeros((2, 150, 2, 16)), x.beta, 64)
    assert np.abs(A0 - oracle.build_A(x.K, x.beta, np.zeros_like(x.g), 64)).max() < 1e-13
    # the same log-decay on every channel: the GDN scalar gate exp(g_i - g_j)
    G = np.repeat(x.g[..., None].astype(np.float64), 16, axis=-1)
    A1, N1 = oracle.build_A_kda_numpy(x.K, G, x.beta, 64, return_N=True)
    A_ref, N_ref = oracle.build_A(x.K, x.beta, x.g, 64, return_N=True)
    assert np.abs(N1 - N_ref).max() < 1e-14 and np.abs(A1 - A_ref).max() < 1e-13
    # a hand value: k_0 = (1, 2), k_1 = (3, 1), G_0 = (0, 0), G_1 = (-ln 2, -ln 4), beta_1 = 2:
    # N_10 = 2 * (3 * 1 / 2 + 1 * 2 / 4) = 4
    K = np.array([[1.0, 2.0], [3.0, 1.0]], np.float32).reshape(1, 2, 1, 2)
    Gh = np.array([[0.0, 0.0], [-np.log(2.0), -np.log(4.0)]]).reshape(1, 2, 1, 2)
    A, N = oracle.build_A_kda_numpy(K, Gh, np.array([1.0, 2.0]).reshape(1, 2, 1), 2, return_N=True)
    assert abs(N[0, 1, 0, 0] - 4.0) < 1e-14 and abs(A[0, 1, 0, 0] + 4.0) < 1e-14
    # defining identities with a genuinely per-channel gate, ragged chunks included
    Gp = wl.per_channel_gate(x, seed=5)
    A2, N2 = oracle.build_A_kda_numpy(x.K, Gp, x.beta, 64, return_N=True)
    for b in range(2):
        for t0, r in ((0, 64), (64, 64), (128, 22)):
            n, a = N2[b, t0:t0 + r, 1, :r], A2[b, t0:t0 + r, 1, :r]
            assert np.abs((np.eye(r) + n) @ a - np.eye(r)).max() < 1e-12
            assert np.array_equal(np.diag(a), np.ones(r)) and not a[np.triu_indices(r, 1)].any()
    assert np.abs(A2 - A_ref).max() > 1e-3      # and it is a different matrix from the scalar-gate one
    # only differences inside a chunk enter: a per-(chunk, head, channel) offset of G changes nothing
    off = np.random.default_rng(6).standard_normal((2, 3, 2, 16)).repeat(64, axis=1)[:, :150]
    N3 = oracle.build_A_kda_numpy(x.K, Gp + off, x.beta, 64, return_N=True)[1]
    assert np.abs(N3 - N2).max() < 1e-12


# ---------------------------------------------------------------- the layer's recurrence and its chunk form

def test_recurrence_hand_worked_scalar_state():
    # d_k = d_v = 1.  Token 1: k=1, v=2, beta=1/2, no decay: S = 1.  Token 2: decay 1/2 (g_2 - g_1 = -ln 2),
    # k=2, v=3, beta=1/8: decayed S = 1/2, v - k S = 2, S = 1/2 + (1/8)(2)(2) = 1; read with q=4, scale 1/2: o = 2.
    K = np.array([1.0, 2.0]).reshape(1, 2, 1, 1)
    V = np.array([2.0, 3.0]).reshape(1, 2, 1, 1)
    Q = np.array([1.0, 4.0]).reshape(1, 2, 1, 1)
    beta = np.array([0.5, 0.125], np.float32).reshape(1, 2, 1)
    g = np.array([0.0, -np.log(2.0)], np.float32).reshape(1, 2, 1)
    O, S = oracle.gdn_recurrence(Q, K, V, beta, g, C=64, scale=0.5)
    assert abs(O[0, 0, 0, 0] - 0.5) < 1e-12 and abs(O[0, 1, 0, 0] - 2.0) < 1e-7 and abs(S[0, 0, 0, 0] - 1.0) < 1e-7
    # (a write-then-decay order would give S = (1 + (1/8)(2)(3 - 2)) / 2 = 5/8 instead)
    # the same tokens as two chunks of one token, g = 0: the cumulative sum restarts, token 2 sees no decay:
    # v - k S = 1, S = 1 + (1/8)(2)(1) = 5/4, o = (1/2)(4)(5/4) = 5/2
    g0 = np.zeros((1, 2, 1), np.float32)
    O2, S2 = oracle.gdn_recurrence(Q, K, V, beta, g0, C=1, scale=0.5)
    assert abs(S2[0, 0, 0, 0] - 1.25) < 1e-12 and abs(O2[0, 1, 0, 0] - 2.5) < 1e-12
    # g = (-ln 2, -ln 2) as two chunks of one token: token 2's own value is its decay (not the difference, 0)
    gr = np.full((1, 2, 1), -np.log(2.0), np.float32)
    _, S3 = oracle.gdn_recurrence(Q, K, V, beta, gr, C=1)
    assert abs(S3[0, 0, 0, 0] - 1.0) < 1e-7
    _, S4 = oracle.gdn_recurrence(Q, K, V, beta, gr, C=2)      # one chunk: difference 0, no decay
    assert abs(S4[0, 0, 0, 0] - 1.25) < 1e-7


def test_recurrence_writes_are_exact_reads_and_orthonormal_keys_give_linear_attention():
    rng = np.random.default_rng(7)
    d, T = 8, 8
    Kq, _ = np.linalg.qr(rng.standard_normal((d, d)))          # orthonormal rows
    K = Kq.reshape(1, T, 1, d)
    V = rng.standard_normal((1, T, 1, 5))
    ones, zeros = np.ones((1, T, 1), np.float32), np.zeros((1, T, 1), np.float32)
    # beta = 1, no decay, unit keys: right after writing (k_t, v_t) the memory returns v_t for the query k_t
    O, S = oracle.gdn_recurrence(K, K, V, ones, zeros, C=4)
    assert np.abs(O - V).max() < 1e-12
    # with mutually orthogonal keys nothing is ever overwritten: S = sum_t k_t v_t^T and the output is the
    # causal linear attention (Q K^T * M) V of Sec. 1
    Q = rng.standard_normal((1, T, 1, d))
    O, S = oracle.gdn_recurrence(Q, K, V, ones, zeros, C=4, scale=0.7)
    assert np.abs(S[0, 0] - K[0, :, 0].T @ V[0, :, 0]).max() < 1e-12
    M = np.tril(np.ones((T, T)))
    assert np.abs(O[0, :, 0] - 0.7 * ((Q[0, :, 0] @ K[0, :, 0].T) * M) @ V[0, :, 0]).max() < 1e-12
    # a general (non-orthogonal) unit key still reads back its own value right after the write
    Kn = rng.standard_normal((1, T, 1, d)); Kn /= np.linalg.norm(Kn, axis=-1, keepdims=True)
    O, _ = oracle.gdn_recurrence(Kn, Kn, V, ones, zeros, C=4)
    assert np.abs(O - V).max() < 1e-12


def test_recurrence_without_writes_only_decays_the_carried_state():
    x = wl.make("s", 1, 150, 2, 16, 16, 64, wl.F32, seed=41)
    Q = wl.queries(x, seed=42)
    S0 = wl.initial_state(x, seed=43)
    O, S = oracle.gdn_recurrence(Q, x.K, x.V, np.zeros_like(x.beta), x.g, 64, scale=2.0, S0=S0)
    g = x.g.astype(np.float64)[0]                                # [T,H]; total log-decay up to token t:
    tot = g.copy()
    tot[64:128] += g[63]
    tot[128:] += g[63] + g[127]
    for h in range(2):
        want = 2.0 * np.exp(tot[:, h])[:, None] * (Q[0, :, h].astype(np.float64) @ S0[0, h].astype(np.float64))
        assert np.abs(O[0, :, h] - want).max() < 1e-12
        assert np.abs(S[0, h] - np.exp(tot[-1, h]) * S0[0, h]).max() < 1e-12


def test_chunk_form_with_the_inverse_equals_the_recurrence():
    # the re-formulation the whole path rests on: U~ = U - W S with W = A diag(beta gamma) K, U = A diag(beta) V
    cu = np.array([0, 70, 71, 230], np.int32)
    for cu_seqlens, B, T in ((None, 2, 150), (cu, 1, 230)):
        x = wl.make("c", B, T, 2, 16, 24, 64, wl.F32, seed=44, cu_seqlens=cu_seqlens)
        Q = wl.queries(x, seed=45)
        S0 = wl.initial_state(x, seed=46)
        A = oracle.build_A(x.K, x.beta, x.g, 64, cu_seqlens=cu_seqlens)
        Kg = x.K.astype(np.float64) * np.exp(x.g.astype(np.float64))[..., None]
        W, _ = oracle.wy(A, Kg, None, x.beta, 64, cu_seqlens=cu_seqlens)
        _, U = oracle.wy(A, x.K, x.V, x.beta, 64, cu_seqlens=cu_seqlens)
        O1, S1 = oracle.chunk_scan(Q, x.K, W, U, x.g, 64, scale=0.25, S0=S0, cu_seqlens=cu_seqlens)
        O2, S2 = oracle.gdn_recurrence(Q, x.K, x.V, x.beta, x.g, 64, scale=0.25, S0=S0, cu_seqlens=cu_seqlens)
        assert np.abs(O1 - O2).max() < 1e-11 and np.abs(S1 - S2).max() < 1e-11
        # and the plain (not decay-weighted) W does NOT reproduce it: the decay factor belongs in W
        Wp, _ = oracle.wy(A, x.K, None, x.beta, 64, cu_seqlens=cu_seqlens)
        O3, _ = oracle.chunk_scan(Q, x.K, Wp, U, x.g, 64, scale=0.25, S0=S0, cu_seqlens=cu_seqlens)
        assert np.abs(O3 - O2).max() > 1e-3


# ---------------------------------------------------------------- the other decay forms of Table 1 (Comba, KDA rows)

def test_shifted_gate_hand_values_and_reductions():
    """Comba row, K K^T * A^{i-1/j}: N_ij = beta_i (k_i . k_j) exp(g_{i-1} - g_j).  Hand values on three tokens with
    integer keys; without decay it is the DeltaNet matrix; and it is NOT the GDN matrix when g decreases."""
    K = np.zeros((1, 3, 1, 2), np.float32)
    K[0, :, 0] = [[1, 0], [2, 1], [1, 3]]
    beta = np.array([0.5, 0.25, 2.0], np.float32).reshape(1, 3, 1)
    g = np.log(np.array([0.5, 0.25, 0.125])).astype(np.float32).reshape(1, 3, 1)
    A, N = oracle.build_A_shifted(K, beta, g, 4, return_N=True)
    n = N[0, :, 0, :3]
    # N_10 = 0.25 * 2 * exp(g0 - g0) = 0.5;  N_20 = 2 * 1 * exp(g1 - g0) = 2 * 0.5;  N_21 = 2 * 5 * exp(g1 - g1) = 10
    assert np.allclose(n, [[0, 0, 0], [0.5, 0, 0], [1.0, 10.0, 0]], atol=1e-7)
    a = A[0, :, 0, :3]
    assert np.allclose(a, [[1, 0, 0], [-0.5, 1, 0], [-1.0 + 10 * 0.5, -10.0, 1]], atol=1e-6)
    x = wl.make("s", 1, 128, 2, 16, 16, 64, wl.F32, seed=71)
    zero = np.zeros_like(x.g)
    assert np.array_equal(oracle.build_A_shifted(x.K, x.beta, zero, 64), oracle.build_A(x.K, x.beta, zero, 64))
    assert np.abs(oracle.build_A_shifted(x.K, x.beta, x.g, 64) - oracle.build_A(x.K, x.beta, x.g, 64)).max() > 1e-3
    # the shifted matrix is the plain one with row i rescaled by exp(g_{i-1} - g_i): N_shift = diag(exp(-a)) N
    _, Ns = oracle.build_A_shifted(x.K, x.beta, x.g, 64, return_N=True)
    _, Np = oracle.build_A(x.K, x.beta, x.g, 64, return_N=True)
    a_tok = x.g.astype(np.float64) - oracle.shifted_gate(x.g, 64)
    assert np.abs(Ns - Np * np.exp(-a_tok)[..., None]).max() < 1e-12


def test_comba_chunk_form_equals_its_recurrence():
    """S_t = (alpha_t I - beta_t k_t k_t^T) S_{t-1} + beta_t k_t v_t^T token by token against the chunk form built from the
    shifted-gate inverse: U~ = U - W S with W = A diag(beta exp(g_{i-1})) K, then the same output and state formulas
    as the GDN row.  A hand-worked scalar case separates it from the GDN recurrence."""
    # scalar state, one token: S0 = 1, alpha = 1/2, beta = 1/2, k = 1, v = 3:  S1 = (1/2 - 1/2) * 1 + 1/2 * 3 = 3/2
    one = np.ones((1, 1, 1, 1), np.float32)
    O, S = oracle.recurrence_ex(one, one, 3 * one, np.full((1, 1, 1), 0.5, np.float32), np.log(np.full((1, 1, 1), 0.5, np.float32)),
                                64, read_before_decay=True, S0=np.ones((1, 1, 1, 1)))
    assert abs(S[0, 0, 0, 0] - 1.5) < 1e-8 and abs(O[0, 0, 0, 0] - 1.5) < 1e-8     # g = ln(1/2) is carried in fp32
    # (the GDN form gives alpha S0 + beta (v - alpha S0) = 1/2 + 1/2 (3 - 1/2) = 7/4)
    _, Sg = oracle.gdn_recurrence(one, one, 3 * one, np.full((1, 1, 1), 0.5, np.float32), np.log(np.full((1, 1, 1), 0.5, np.float32)),
                                  64, S0=np.ones((1, 1, 1, 1)))
    assert abs(Sg[0, 0, 0, 0] - 1.75) < 1e-8
    cu = np.array([0, 70, 71, 230], np.int32)
    for cu_seqlens, B, T in ((None, 2, 150), (cu, 1, 230)):
        x = wl.make("c", B, T, 2, 16, 24, 64, wl.F32, seed=81, cu_seqlens=cu_seqlens)
        Q = wl.queries(x, seed=82)
        S0 = wl.initial_state(x, seed=83)
        A = oracle.build_A_shifted(x.K, x.beta, x.g, 64, cu_seqlens=cu_seqlens)
        gs = oracle.shifted_gate(x.g, 64, cu_seqlens=cu_seqlens)
        W, _ = oracle.wy(A, x.K.astype(np.float64) * np.exp(gs)[..., None], None, x.beta, 64, cu_seqlens=cu_seqlens)
        _, U = oracle.wy(A, x.K, x.V, x.beta, 64, cu_seqlens=cu_seqlens)
        O1, S1 = oracle.chunk_scan(Q, x.K, W, U, x.g, 64, scale=0.5, S0=S0, cu_seqlens=cu_seqlens)
        O2, S2 = oracle.recurrence_ex(Q, x.K, x.V, x.beta, x.g, 64, read_before_decay=True, scale=0.5, S0=S0, cu_seqlens=cu_seqlens)
        assert np.abs(O1 - O2).max() < 1e-11 and np.abs(S1 - S2).max() < 1e-11
        # the unshifted inverse does not reproduce it
        Ag = oracle.build_A(x.K, x.beta, x.g, 64, cu_seqlens=cu_seqlens)
        _, Ug = oracle.wy(Ag, x.K, x.V, x.beta, 64, cu_seqlens=cu_seqlens)
        O3, _ = oracle.chunk_scan(Q, x.K, W, Ug, x.g, 64, scale=0.5, S0=S0, cu_seqlens=cu_seqlens)
        assert np.abs(O3 - O2).max() > 1e-3


def test_per_channel_chunk_form_equals_its_recurrence():
    """KDA row: one decay per key feature.  The C oracle's N equals the numpy + LAPACK statement of the same formula; the
    chunk form built from it (W = A diag(beta) (K * Gamma), U = A diag(beta) V, then ``chunk_scan_kda``) equals the
    token-by-token recurrence; and with the same decay on every feature both reduce to the scalar-gate layer."""
    cu = np.array([0, 70, 71, 200], np.int32)
    for cu_seqlens, B, T in ((None, 2, 130), (cu, 1, 200)):
        x = wl.make("k", B, T, 2, 16, 24, 64, wl.F32, seed=91, cu_seqlens=cu_seqlens)
        G = wl.per_channel_gate(x, seed=92)
        Q = wl.queries(x, seed=93)
        S0 = wl.initial_state(x, seed=94)
        A, N = oracle.build_A_kda(x.K, G, x.beta, 64, cu_seqlens=cu_seqlens, return_N=True)
        A2, N2 = oracle.build_A_kda_numpy(x.K, G, x.beta, 64, cu_seqlens=cu_seqlens, return_N=True)
        assert np.abs(N - N2).max() < 1e-14 and np.abs(A - A2).max() < 1e-12
        Kg = x.K.astype(np.float64) * np.exp(G.astype(np.float64))
        W, _ = oracle.wy(A, Kg, None, x.beta, 64, cu_seqlens=cu_seqlens)
        _, U = oracle.wy(A, x.K, x.V, x.beta, 64, cu_seqlens=cu_seqlens)
        O1, S1 = oracle.chunk_scan_kda(Q, x.K, W, U, G, 64, scale=0.5, S0=S0, cu_seqlens=cu_seqlens)
        O2, S2 = oracle.recurrence_ex(Q, x.K, x.V, x.beta, None, 64, G=G, scale=0.5, S0=S0, cu_seqlens=cu_seqlens)
        assert np.abs(O1 - O2).max() < 1e-10 and np.abs(S1 - S2).max() < 1e-10
        # same decay on every feature: the scalar-gate layer
        Gs = np.repeat(x.g[..., None], x.d_k, axis=3)
        O3, S3 = oracle.recurrence_ex(Q, x.K, x.V, x.beta, None, 64, G=Gs, scale=0.5, S0=S0, cu_seqlens=cu_seqlens)
        O4, S4 = oracle.gdn_recurrence(Q, x.K, x.V, x.beta, x.g, 64, scale=0.5, S0=S0, cu_seqlens=cu_seqlens)
        assert np.abs(O3 - O4).max() < 1e-12 and np.abs(S3 - S4).max() < 1e-12


def test_per_channel_chunk_form_on_rescaled_operands():
    """The form the tensor-core scan runs for the KDA row: with G_ref the middle row of a chunk and G_last its last,
        [W exp(-G_ref) ; Q exp(G - G_ref)] . [diag(exp G_ref) S | (K exp(G_ref - G))^T]
    holds W S, (Q exp G) S and the decayed Q K^T, and the state increment is diag(exp(G_last - G_ref)) (K exp(G_ref - G))^T U~.
    Written out here in fp64 with three plain matrix products per chunk and compared with the oracle's chunk form (which takes
    the exponent of every difference) on ragged sequences: the two must agree to rounding."""
    rng = np.random.default_rng(91)
    C, H, d = 8, 2, 6
    cu = np.array([0, 5, 5, 21, 38], np.int32)
    T = int(cu[-1])
    Q, K, W, U = (rng.standard_normal((1, T, H, d)) for _ in range(4))
    G = np.zeros((1, T, H, d))
    for beg, end in zip(cu[:-1], cu[1:]):
        for t0 in range(beg, end, C):
            t1 = min(t0 + C, end)
            G[0, t0:t1] = -np.cumsum(rng.uniform(0.0, 0.6, size=(t1 - t0, H, d)), axis=0)   # cumulative log-decay inside the chunk
    S0 = rng.standard_normal((len(cu) - 1, H, d, d))
    O_ref, S_ref = oracle.chunk_scan_kda(Q, K, W, U, G, C, scale=0.7, S0=S0, cu_seqlens=cu)
    O = np.zeros_like(O_ref)
    S_out = np.zeros_like(S_ref)
    for s in range(len(cu) - 1):
        for h in range(H):
            S = S0[s, h].copy()
            for t0 in range(cu[s], cu[s + 1], C):
                t1 = min(t0 + C, cu[s + 1])
                r = t1 - t0
                g = G[0, t0:t1, h]
                g_ref, g_last = g[r // 2], g[r - 1]
                Wm = W[0, t0:t1, h] * np.exp(-g_ref)
                Qp = Q[0, t0:t1, h] * np.exp(g - g_ref)
                Km = K[0, t0:t1, h] * np.exp(g_ref - g)
                P1 = np.concatenate([Wm, Qp]) @ np.concatenate([np.exp(g_ref)[:, None] * S, Km.T], axis=1)   # one product
                Ut = U[0, t0:t1, h] - P1[:r, :d]
                P = np.tril(P1[r:, d:])
                O[0, t0:t1, h] = 0.7 * (P1[r:, :d] + P @ Ut)
                S = np.exp(g_last)[:, None] * S + np.exp(g_last - g_ref)[:, None] * (Km.T @ Ut)
            S_out[s, h] = S
    assert np.abs(O - O_ref).max() <= 1e-12 * max(1.0, np.abs(O_ref).max())
    assert np.abs(S_out - S_ref).max() <= 1e-12 * max(1.0, np.abs(S_ref).max())
