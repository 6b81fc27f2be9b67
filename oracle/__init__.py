"""fp64 CPU oracle (TEST INFRASTRUCTURE ONLY).

Slow, plain reference for the chunkwise delta-rule triangular inversion
``A = (I + N)^{-1}`` with ``N = tril(diag(beta) K K^T * exp(g_i - g_j), -1)``
(Eq. 3 with the GDN row of Table 1) and the WY factors
``W = A diag(beta) K``, ``U = A diag(beta) V``.

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s CPU-baseline
and ``--impl reference`` legs may import this package.  It shares no code with
the CUDA library and the CUDA library never calls it.

* ``build_A`` / ``wy``      -- the C implementation (``tri_inv_oracle.c``), plain
  triple loops in double, OpenMP over independent chunks.
* ``gdn_recurrence``        -- the layer as its token-by-token recurrence (C, double); ``chunk_scan`` -- the
  chunk form that consumes W and U (numpy).  Pins: a hand-worked scalar example, exact read-back of a write,
  orthonormal keys reducing to causal linear attention (Sec. 1), the no-write closed form, and the two
  agreeing with each other through ``build_A`` / ``wy``.
* ``build_A_kda``           -- per-channel decay (KDA row of Table 1), numpy + LAPACK.
* ``oracle.algorithms``     -- numpy fp64 restatements of the paper's inversion
  algorithms (Algs. 2, 4, 5 and the 2x2 block formula), step by step.

Parity pins (tests/test_oracle_pins.py): hand-worked 2x2/3x3/4x4 closed forms,
the first-difference matrix, the 2^{i-j-1} growth example and binomial powers
(Sec. 3.2), residuals to 1e-12, exact rational brute force, LAPACK, the
|A_ij| <= 1 invariant (Sec. 2.2), and the sequential delta-rule recurrence.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tri_inv_oracle.c")
_LIB = os.path.join(_HERE, "libtri_inv_oracle.so")

F32, BF16, F64 = 0, 1, 2
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i32 = ctypes.c_void_p, ctypes.c_int
        lib.tri_inv_oracle_build.restype = i32
        lib.tri_inv_oracle_build.argtypes = [vp, i32, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, i32, i32]
        lib.tri_inv_oracle_build_ex.restype = i32
        lib.tri_inv_oracle_build_ex.argtypes = [vp, i32, vp, vp, vp, i32, vp, vp, i32, i32, i32, i32, i32, vp, i32, i32]
        lib.tri_inv_oracle_recurrence_ex.restype = i32
        lib.tri_inv_oracle_recurrence_ex.argtypes = [vp, vp, vp, i32, vp, vp, vp, i32, vp, vp, vp, ctypes.c_double,
                                                     i32, i32, i32, i32, i32, i32, vp, i32, i32]
        lib.tri_inv_oracle_wy.restype = i32
        lib.tri_inv_oracle_wy.argtypes = [vp, vp, vp, i32, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, i32, i32]
        lib.tri_inv_oracle_gdn_recurrence.restype = i32
        lib.tri_inv_oracle_gdn_recurrence.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp, ctypes.c_double,
                                                      i32, i32, i32, i32, i32, i32, vp, i32, i32]
        lib.tri_inv_oracle_threads.restype = i32
        lib.tri_inv_oracle_threads.argtypes = [i32]
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _kv(a: np.ndarray):
    """Storage array -> (contiguous array, dtype code).  uint16 means bf16 bit patterns."""
    if a.dtype == np.float32:
        return np.ascontiguousarray(a), F32
    if a.dtype == np.uint16:
        return np.ascontiguousarray(a), BF16
    if a.dtype == np.float64:
        return np.ascontiguousarray(a), F64
    raise TypeError("K/V must be float32, float64 or uint16 (bf16 bits), got %s" % a.dtype)


def _widen(a: np.ndarray) -> np.ndarray:
    """Storage array -> float64, exactly."""
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return np.ascontiguousarray(a, dtype=np.float64)


def raw_front_end(K_raw, beta_logit, gate_logit, C, cu_seqlens=None):
    """The producers a Gated-DeltaNet layer runs before the inversion, in fp64 (the recipe the
    configurations state for their inputs): beta = sigmoid(beta_logit); per-token log-decay
    a = log sigmoid(gate_logit), g = its cumulative sum restarting at every chunk; keys divided by
    their L2 norm over the feature axis (a zero key stays zero).  Returns (K_hat f64, beta f64, g f64)."""
    Kd = _widen(np.asarray(K_raw))
    B, T, H, _ = Kd.shape
    nrm = np.sqrt((Kd * Kd).sum(axis=-1, keepdims=True))
    K_hat = np.divide(Kd, nrm, out=np.zeros_like(Kd), where=nrm > 0)
    x = np.asarray(beta_logit, dtype=np.float64)
    beta = 1.0 / (1.0 + np.exp(-x))
    z = np.asarray(gate_logit, dtype=np.float64)
    a = np.minimum(z, 0.0) - np.log1p(np.exp(-np.abs(z)))
    a = a.reshape(B * T, H)
    g = np.zeros_like(a)
    bounds = [(b * T, (b + 1) * T) for b in range(B)] if cu_seqlens is None else \
             [(int(cu_seqlens[i]), int(cu_seqlens[i + 1])) for i in range(len(cu_seqlens) - 1)]
    for beg, end in bounds:
        t = beg
        while t < end:
            e = min(t + C, end)
            run = np.zeros(H)
            for r in range(t, e):          # plain running sum, token by token
                run = run + a[r]
                g[r] = run
            t = e
    return K_hat, beta, g.reshape(B, T, H)


def build_A_kda_numpy(K, G, beta, C, cu_seqlens=None, return_N=False):
    """Per-channel decay (the KDA row of Table 1): phi = (K * Gamma)(K / Gamma)^T with Gamma = exp(G),
    G [B,T,H,d] the cumulative per-channel log-decay inside each chunk, and beta scaling rows:
        N_ij = beta_i * sum_c K_ic K_jc exp(G_ic - G_jc)   (i > j),      A = (I + N)^{-1}.
    The exponent is taken of the difference, so no factor can overflow when G decreases along a chunk.
    fp64 numpy; the inverse by LAPACK's triangular solve (forward substitution)."""
    from scipy.linalg import solve_triangular
    Kd, Gd = _widen(np.asarray(K)), np.asarray(G, dtype=np.float64)
    bd = np.asarray(beta, dtype=np.float64)
    B, T, H, d = Kd.shape
    Kf, Gf, bf = Kd.reshape(B * T, H, d), Gd.reshape(B * T, H, d), bd.reshape(B * T, H)
    A = np.zeros((B * T, H, C))
    N = np.zeros((B * T, H, C)) if return_N else None
    bounds = [(b * T, (b + 1) * T) for b in range(B)] if cu_seqlens is None else \
             [(int(cu_seqlens[i]), int(cu_seqlens[i + 1])) for i in range(len(cu_seqlens) - 1)]
    for beg, end in bounds:
        for t0 in range(beg, end, C):
            r = min(C, end - t0)
            for h in range(H):
                k, g, b = Kf[t0:t0 + r, h], Gf[t0:t0 + r, h], bf[t0:t0 + r, h]
                n = np.zeros((r, r))
                for i in range(r):
                    for j in range(i):
                        n[i, j] = b[i] * np.sum(k[i] * k[j] * np.exp(g[i] - g[j]))
                a = solve_triangular(np.eye(r) + n, np.eye(r), lower=True, unit_diagonal=True)
                A[t0:t0 + r, h, :r] = np.tril(a)
                if return_N:
                    N[t0:t0 + r, h, :r] = n
    A = A.reshape(B, T, H, C)
    return (A, N.reshape(B, T, H, C)) if return_N else A


def build_A_kda(K, G, beta, C, cu_seqlens=None, return_N=False, n_threads=0):
    """Per-channel decay (the KDA row of Table 1) by the C oracle: N_ij = beta_i sum_c K_ic K_jc exp(G_ic - G_jc) by
    plain loops, forward substitution for A.  ``build_A_kda_numpy`` is the same definition written with numpy and
    LAPACK's triangular solve; a pin holds the two against each other."""
    return _build_ex(K, beta, None, np.ascontiguousarray(G, dtype=np.float32), 0, C, cu_seqlens, n_threads, return_N)


def build_A_shifted(K, beta, g, C, cu_seqlens=None, return_N=False, n_threads=0):
    """The Comba row of Table 1, K K^T * A^{i-1/j}: N_ij = beta_i (k_i . k_j) exp(g_{i-1} - g_j) -- row i decays
    from token j up to the token BEFORE i.  A = (I + N)^{-1} by forward substitution (C oracle)."""
    return _build_ex(K, beta, np.ascontiguousarray(g, dtype=np.float32), None, 1, C, cu_seqlens, n_threads, return_N)


def _build_ex(K, beta, g, G, gate_shift, C, cu_seqlens, n_threads, return_N):
    K, dt = _kv(K)
    B, T, H, d_k = K.shape
    beta = np.ascontiguousarray(beta, dtype=np.float32)
    assert beta.shape == (B, T, H) and (g is None or g.shape == (B, T, H)) and (G is None or G.shape == (B, T, H, d_k))
    A = np.zeros((B, T, H, C), dtype=np.float64)
    N = np.zeros((B, T, H, C), dtype=np.float64) if return_N else None
    cu = None if cu_seqlens is None else np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    rc = _load().tri_inv_oracle_build_ex(_ptr(K), dt, _ptr(beta), _ptr(g), _ptr(G), int(gate_shift), _ptr(A), _ptr(N),
                                         B, T, H, d_k, C, _ptr(cu), 0 if cu is None else len(cu) - 1, int(n_threads))
    if rc != 0:
        raise ValueError("tri_inv_oracle_build_ex: invalid arguments")
    return (A, N) if return_N else A


def recurrence_ex(Q, K, V, beta, g, C, G=None, read_before_decay=False, scale=1.0, S0=None, cu_seqlens=None, n_threads=0):
    """Token-by-token recurrence for the other decay forms of Table 1 (C oracle, fp64): ``G`` [B,T,H,d_k] gives one
    decay per key feature (KDA row; ``g`` unused); ``read_before_decay`` makes the write's correction read the state
    before the token's decay (Comba row).  Returns (O, S_final) like ``gdn_recurrence``."""
    Q, dq = _kv(Q)
    K, dk = _kv(K)
    V, dv = _kv(V)
    if not (dq == dk == dv):
        Q, K, V, dk = _widen(Q), _widen(K), _widen(V), F64
    B, T, H, d_k = K.shape
    d_v = V.shape[3]
    beta = np.ascontiguousarray(beta, dtype=np.float32)
    g = None if g is None else np.ascontiguousarray(g, dtype=np.float32)
    G = None if G is None else np.ascontiguousarray(G, dtype=np.float32)
    cu = None if cu_seqlens is None else np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    n_seqs = B if cu is None else len(cu) - 1
    S0 = None if S0 is None else np.ascontiguousarray(S0, dtype=np.float64)
    O = np.zeros((B, T, H, d_v))
    S = np.zeros((n_seqs, H, d_k, d_v))
    rc = _load().tri_inv_oracle_recurrence_ex(_ptr(Q), _ptr(K), _ptr(V), dk, _ptr(beta), _ptr(g), _ptr(G),
                                              1 if read_before_decay else 0, _ptr(S0), _ptr(O), _ptr(S), float(scale),
                                              B, T, H, d_k, d_v, C, _ptr(cu), 0 if cu is None else n_seqs, int(n_threads))
    if rc != 0:
        raise ValueError("tri_inv_oracle_recurrence_ex: invalid arguments")
    return O, S


def gdn_recurrence(Q, K, V, beta, g, C, scale=1.0, S0=None, cu_seqlens=None, n_threads=0):
    """The gated delta-rule layer token by token (decay, delta-rule write, read) in fp64: the definition
    that the chunkwise path re-formulates.  Returns (O [B,T,H,d_v], S_final [n_sequences,H,d_k,d_v])."""
    Q, dq = _kv(Q)
    K, dk = _kv(K)
    V, dv = _kv(V)
    if not (dq == dk == dv):
        Q, K, V, dk = _widen(Q), _widen(K), _widen(V), F64
    B, T, H, d_k = K.shape
    d_v = V.shape[3]
    beta = np.ascontiguousarray(beta, dtype=np.float32)
    g = np.ascontiguousarray(g, dtype=np.float32)
    cu = None if cu_seqlens is None else np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    n_seqs = B if cu is None else len(cu) - 1
    S0 = None if S0 is None else np.ascontiguousarray(S0, dtype=np.float64)
    assert S0 is None or S0.shape == (n_seqs, H, d_k, d_v)
    O = np.zeros((B, T, H, d_v))
    S = np.zeros((n_seqs, H, d_k, d_v))
    rc = _load().tri_inv_oracle_gdn_recurrence(_ptr(Q), _ptr(K), _ptr(V), dk, _ptr(beta), _ptr(g), _ptr(S0),
                                               _ptr(O), _ptr(S), float(scale), B, T, H, d_k, d_v, C,
                                               _ptr(cu), 0 if cu is None else n_seqs, int(n_threads))
    if rc != 0:
        raise ValueError("tri_inv_oracle_gdn_recurrence: invalid arguments")
    return O, S


def chunk_scan(Q, K, W, U, g, C, scale=1.0, S0=None, cu_seqlens=None):
    """What the chunk-scan entry point computes from its inputs, in fp64, chunk by chunk in order.  With
    gamma_i = exp(g_i), D_ij = gamma_i / gamma_j (j <= i, else 0) and the state S entering the chunk:
        U~ = U - W S,   O = scale * (diag(gamma) Q S + ((Q K^T) * D) U~),
        S <- gamma_last S + (diag(gamma_last / gamma) K)^T U~.
    W is the decay-weighted factor A diag(beta * gamma) K, U = A diag(beta) V; with those two exact this is the
    token-by-token recurrence re-bracketed (the identity the pins check).  Returns (O, S_final)."""
    Qd, Kd, Wd, Ud = _widen(np.asarray(Q)), _widen(np.asarray(K)), _widen(np.asarray(W)), _widen(np.asarray(U))
    gd = np.asarray(g, dtype=np.float64)
    B, T, H, d_k = Kd.shape
    d_v = Ud.shape[3]
    bounds = [(b * T, (b + 1) * T) for b in range(B)] if cu_seqlens is None else \
             [(int(cu_seqlens[i]), int(cu_seqlens[i + 1])) for i in range(len(cu_seqlens) - 1)]
    Qf, Kf, Wf, Uf, gf = (x.reshape((B * T,) + x.shape[2:]) for x in (Qd, Kd, Wd, Ud, gd))
    O = np.zeros((B * T, H, d_v))
    S_all = np.zeros((len(bounds), H, d_k, d_v))
    for s, (beg, end) in enumerate(bounds):
        for h in range(H):
            S = np.zeros((d_k, d_v)) if S0 is None else np.array(S0[s, h], dtype=np.float64)
            for t0 in range(beg, end, C):
                t1 = min(t0 + C, end)
                q, k, w, u, gg = Qf[t0:t1, h], Kf[t0:t1, h], Wf[t0:t1, h], Uf[t0:t1, h], gf[t0:t1, h]
                D = np.tril(np.exp(gg[:, None] - gg[None, :]))
                ut = u - w @ S
                O[t0:t1, h] = scale * (np.exp(gg)[:, None] * (q @ S) + ((q @ k.T) * D) @ ut)
                S = np.exp(gg[-1]) * S + (np.exp(gg[-1] - gg)[:, None] * k).T @ ut
            S_all[s, h] = S
    return O.reshape(B, T, H, d_v), S_all


def chunk_scan_kda(Q, K, W, U, G, C, scale=1.0, S0=None, cu_seqlens=None):
    """The chunk scan with one decay per key feature (KDA row of Table 1), in fp64, chunk by chunk.  With
    Gamma_i = exp(G_i) (a vector over the key features) and the state S entering the chunk:
        U~ = U - W S,     P_ij = sum_c Q_ic K_jc exp(G_ic - G_jc)  (j <= i, else 0),
        O  = scale * ((Q * Gamma) S + P U~),     S <- diag(Gamma_last) S + (K * exp(G_last - G))^T U~.
    W is the decay-weighted factor A diag(beta) (K * Gamma), U = A diag(beta) V, A from ``build_A_kda``; with those
    exact this is ``recurrence_ex(G=...)`` re-bracketed (pinned).  Returns (O, S_final)."""
    Qd, Kd, Wd, Ud = _widen(np.asarray(Q)), _widen(np.asarray(K)), _widen(np.asarray(W)), _widen(np.asarray(U))
    Gd = np.asarray(G, dtype=np.float64)
    B, T, H, d_k = Kd.shape
    d_v = Ud.shape[3]
    bounds = [(b * T, (b + 1) * T) for b in range(B)] if cu_seqlens is None else \
             [(int(cu_seqlens[i]), int(cu_seqlens[i + 1])) for i in range(len(cu_seqlens) - 1)]
    Qf, Kf, Wf, Uf, Gf = (x.reshape((B * T,) + x.shape[2:]) for x in (Qd, Kd, Wd, Ud, Gd))
    O = np.zeros((B * T, H, d_v))
    S_all = np.zeros((len(bounds), H, d_k, d_v))
    for s, (beg, end) in enumerate(bounds):
        for h in range(H):
            S = np.zeros((d_k, d_v)) if S0 is None else np.array(S0[s, h], dtype=np.float64)
            for t0 in range(beg, end, C):
                t1 = min(t0 + C, end)
                q, k, w, u, gg = Qf[t0:t1, h], Kf[t0:t1, h], Wf[t0:t1, h], Uf[t0:t1, h], Gf[t0:t1, h]
                r = t1 - t0
                P = np.zeros((r, r))
                for i in range(r):
                    for j in range(i + 1):
                        P[i, j] = np.sum(q[i] * k[j] * np.exp(gg[i] - gg[j]))
                ut = u - w @ S
                O[t0:t1, h] = scale * ((q * np.exp(gg)) @ S + P @ ut)
                S = np.exp(gg[-1])[:, None] * S + (k * np.exp(gg[-1][None, :] - gg)).T @ ut
            S_all[s, h] = S
    return O.reshape(B, T, H, d_v), S_all


def shifted_gate(g, C, cu_seqlens=None):
    """g_{i-1} for every token (0 at the first token of each chunk): the row factor of the Comba row's decay matrix."""
    g = np.asarray(g, dtype=np.float64)
    B, T, H = g.shape
    gf = g.reshape(B * T, H)
    out = np.zeros_like(gf)
    bounds = [(b * T, (b + 1) * T) for b in range(B)] if cu_seqlens is None else \
             [(int(cu_seqlens[i]), int(cu_seqlens[i + 1])) for i in range(len(cu_seqlens) - 1)]
    for beg, end in bounds:
        for t in range(beg, end):
            if (t - beg) % C:
                out[t] = gf[t - 1]
    return out.reshape(B, T, H)


def threads(n_threads: int = 0) -> int:
    return int(_load().tri_inv_oracle_threads(int(n_threads)))


def build_A(K, beta, g, C, cu_seqlens=None, n_threads=0, return_N=False):
    """A = (I+N)^{-1} per chunk in fp64.

    K [B,T,H,d_k] float32 or uint16 (bf16 bits); beta, g [B,T,H] float32.
    Returns A [B,T,H,C] float64 (and N, same shape, when ``return_N``).
    """
    K, dt = _kv(K)
    B, T, H, d_k = K.shape
    beta = np.ascontiguousarray(beta, dtype=np.float32)
    g = np.ascontiguousarray(g, dtype=np.float32)   # the C ABI under test takes fp32 beta and g
    assert beta.shape == (B, T, H) and g.shape == (B, T, H)
    A = np.zeros((B, T, H, C), dtype=np.float64)
    N = np.zeros((B, T, H, C), dtype=np.float64) if return_N else None
    cu = None if cu_seqlens is None else np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    n_seqs = 0 if cu is None else len(cu) - 1
    rc = _load().tri_inv_oracle_build(_ptr(K), dt, _ptr(beta), _ptr(g), _ptr(A), _ptr(N),
                                      B, T, H, d_k, C, _ptr(cu), n_seqs, int(n_threads))
    if rc != 0:
        raise ValueError("tri_inv_oracle_build: invalid arguments")
    return (A, N) if return_N else A


def wy(A, K, V, beta, C, cu_seqlens=None, n_threads=0):
    """W = A diag(beta) K, U = A diag(beta) V in fp64 from a given A [B,T,H,C]."""
    K, dt = _kv(K)
    B, T, H, d_k = K.shape
    d_v = 0
    if V is not None:
        V, dtv = _kv(V)
        if dtv != dt:  # one storage type per call: widen both (exactly) to double
            K, V, dt = _widen(K), _widen(V), F64
        assert V.shape[:3] == (B, T, H)
        d_v = V.shape[3]
    A = np.ascontiguousarray(A, dtype=np.float64)
    assert A.shape == (B, T, H, C)
    beta = np.ascontiguousarray(beta, dtype=np.float32)
    W = np.zeros((B, T, H, d_k), dtype=np.float64)
    U = np.zeros((B, T, H, d_v), dtype=np.float64) if V is not None else None
    cu = None if cu_seqlens is None else np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    n_seqs = 0 if cu is None else len(cu) - 1
    rc = _load().tri_inv_oracle_wy(_ptr(A), _ptr(K), _ptr(V), dt, _ptr(beta), _ptr(W), _ptr(U),
                                   B, T, H, d_k, d_v, C, _ptr(cu), n_seqs, int(n_threads))
    if rc != 0:
        raise ValueError("tri_inv_oracle_wy: invalid arguments")
    return W, U
