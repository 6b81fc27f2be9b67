"""numpy fp64 restatements of the paper's inversion algorithms (TEST INFRASTRUCTURE ONLY).

Each function inverts ``I + L`` for one strictly lower triangular ``L`` (n a
power of two) by one of the schemes the paper analyses, written here from the
identity each scheme rests on.  They exist so the tests can check that the
schemes the CUDA library implements reach, in exact arithmetic, the same matrix
as forward substitution; they are never used by the product.

Sign convention: every routine here inverts ``I + L``; Eq. 3's ``I - phi .* L^-``
is the same thing with ``L := -phi .* L^-``.
"""
from __future__ import annotations

import numpy as np


def forward_substitution(L: np.ndarray) -> np.ndarray:
    """Column sweep in scalar form (Sec. 3.1): solve (I+L) X = I column by column."""
    n = L.shape[0]
    X = np.zeros((n, n))
    for j in range(n):
        X[j, j] = 1.0
        for i in range(j + 1, n):
            s = 0.0
            for k in range(j, i):
                s += L[i, k] * X[k, j]
            X[i, j] = -s
    return X


def neumann_series(L: np.ndarray) -> np.ndarray:
    """(I+L)^{-1} = I - L + L^2 - ... ; L^n = 0 so the sum is finite (Sec. 3.2)."""
    n = L.shape[0]
    X = np.eye(n)
    P = np.eye(n)
    for _ in range(1, n):
        P = -(P @ L)
        X = X + P
    return X


def mch(L: np.ndarray) -> np.ndarray:
    """Repeated squaring of the nilpotent series (Alg. 5 / Sec. 3.2).  With P_k = L^(2^k) the partial sum up to power
    2^(k+1) - 1 is S_k = (I - L)(I + P_1)(I + P_2) ... (I + P_k); each round squares P and multiplies the sum by the
    next factor, and log2(n) - 1 rounds reach power n - 1, beyond which every power vanishes."""
    n = L.shape[0]
    total = np.eye(n) - L
    power = L.copy()
    for _ in range(max(int(np.log2(n)) - 1, 0)):
        power = power @ power
        total = total @ (np.eye(n) + power)
    return total


def product_form(L: np.ndarray) -> np.ndarray:
    """prod_{k=0}^{log2(n)-1} (I + (-L)^{2^k}) -- the same series factorised."""
    n = L.shape[0]
    X = np.eye(n)
    P = -L
    for _ in range(max(int(np.log2(n)), 1)):
        X = X @ (np.eye(n) + P)
        P = P @ P
    return X


def mbh(L: np.ndarray, X0: np.ndarray | None = None, b0: int = 1) -> np.ndarray:
    """Bunch-Hopcroft recursion, bottom up (Alg. 4 / Sec. 3.3).  X0 holds the inverses of the b0 x b0 diagonal blocks
    of I + L (the identity for b0 = 1).  At block size b every adjacent pair (upper block r, lower block r + b) is
    joined by the 2x2 block identity for a lower triangular matrix: the pair's off-diagonal block becomes
    -X_low . L_low,up . X_up; doubling b until one block is left gives the inverse.  Only the blocks the next level
    reads are formed."""
    n = L.shape[0]
    X = np.eye(n) if X0 is None else np.array(X0, dtype=np.float64)
    b = b0
    while b < n:
        for r in range(0, n, 2 * b):
            up, low = slice(r, r + b), slice(r + b, r + 2 * b)
            X[low, up] = -(X[low, low] @ L[low, up] @ X[up, up])
        b *= 2
    return X


def mxr(L: np.ndarray, b0: int = 16) -> np.ndarray:
    """Alg. 2 with r = 0: Alg. 5 on the b0 x b0 diagonal blocks, then Alg. 4 from b0."""
    n = L.shape[0]
    b0 = min(b0, n)
    Y = np.zeros_like(L)
    for t in range(n // b0):
        s = slice(t * b0, (t + 1) * b0)
        Y[s, s] = mch(L[s, s])
    return mbh(L, Y, b0)


def newton_schulz(L: np.ndarray, m: int | None = None, x0_scale: float | None = None) -> np.ndarray:
    """Newton's iteration for the inverse of M = I + L (Alg. 3 / Sec. 3.5): X <- X (2I - M X), whose residual I - M X
    squares every round, from X_0 = I / n (the exponent-1 reading of Prop. 3.2's I / n^O(1)).  Default 2 log2(n) rounds."""
    n = L.shape[0]
    M = np.eye(n) + L
    X = np.eye(n) * (1.0 / n if x0_scale is None else x0_scale)
    for _ in range(2 * int(np.log2(n)) if m is None else m):
        X = X @ (2.0 * np.eye(n) - M @ X)
    return X


def iterative_refinement(X: np.ndarray, L: np.ndarray) -> np.ndarray:
    """One step of Sec. 3.6 for the matrix I + L: R <- I - X (I + L), X <- X + R X."""
    n = L.shape[0]
    R = np.eye(n) - X @ (np.eye(n) + L)
    return X + R @ X


def block_recursive(L: np.ndarray, leaf: int = 16) -> np.ndarray:
    """The 2x2 block identity of Sec. 3.3 written for a lower triangular matrix:
    inv([[M11, 0], [N21, M22]]) = [[X11, 0], [-X22 N21 X11, X22]], recursing down
    to ``leaf`` x ``leaf`` blocks that are inverted by forward substitution."""
    n = L.shape[0]
    if n <= leaf:
        return forward_substitution(L)
    h = n // 2
    X11 = block_recursive(L[:h, :h], leaf)
    X22 = block_recursive(L[h:, h:], leaf)
    X = np.zeros((n, n))
    X[:h, :h] = X11
    X[h:, h:] = X22
    X[h:, :h] = -(X22 @ L[h:, :h] @ X11)
    return X


def chunk_N(K: np.ndarray, beta: np.ndarray, g: np.ndarray) -> np.ndarray:
    """One chunk's N from its keys [C,d], betas [C] and cumulative log-decays [C]."""
    K = K.astype(np.float64)
    beta = beta.astype(np.float64)
    g = g.astype(np.float64)
    C = K.shape[0]
    N = np.zeros((C, C))
    for i in range(C):
        for j in range(i):
            N[i, j] = beta[i] * float(K[i] @ K[j]) * np.exp(g[i] - g[j])
    return N
