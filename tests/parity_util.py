"""Shared helpers of the GPU parity tests: error metrics against the fp64 oracle."""
import numpy as np


def local_index(inp):
    """Position of every flat token inside its chunk, and a mask of tokens that exist."""
    loc = np.zeros(inp.B * inp.T, dtype=np.int64)
    for t0, r in inp.chunk_list():
        loc[t0:t0 + r] = np.arange(r)
    return loc


def structure_errors(A_gpu_f32: np.ndarray, inp):
    """Bit-exact structure of A [B,T,H,C] fp32: upper triangle all-bits-zero, diagonal exactly 1.0f.
    Returns (#nonzero-bit upper entries, #diagonal entries != 1)."""
    B, T, H, C = A_gpu_f32.shape
    bits = np.ascontiguousarray(A_gpu_f32).view(np.uint32).reshape(B * T, H, C)
    loc = local_index(inp)
    cols = np.arange(C)[None, :]
    upper = cols > loc[:, None]                     # [tokens, C]
    bad_upper = int(np.count_nonzero(bits[np.broadcast_to(upper[:, None, :], bits.shape)]))
    diag = np.take_along_axis(A_gpu_f32.reshape(B * T, H, C), loc[:, None, None].repeat(H, 1), axis=2)
    bad_diag = int(np.count_nonzero(diag != np.float32(1.0)))
    return bad_upper, bad_diag


def max_ratio(x_gpu: np.ndarray, x_ref: np.ndarray) -> float:
    """max |x_gpu - x_ref| / max |x_ref| over the whole tensor (the forward error the tolerances are stated in)."""
    den = float(np.abs(x_ref).max())
    if den == 0.0:
        return float(np.abs(x_gpu).max())
    return float(np.abs(x_gpu.astype(np.float64) - x_ref).max() / den)


def max_residual(A_gpu: np.ndarray, N_ref: np.ndarray, inp, max_chunks=None) -> float:
    """max over chunks of ||(I + N) A_gpu - I||_max with the oracle's fp64 N."""
    B, T, H, C = A_gpu.shape
    a = A_gpu.reshape(B * T, H, C).astype(np.float64)
    n = N_ref.reshape(B * T, H, C)
    worst = 0.0
    chunks = inp.chunk_list()
    if max_chunks is not None and len(chunks) > max_chunks:
        step = len(chunks) // max_chunks
        chunks = chunks[::step]
    for t0, r in chunks:
        ac = a[t0:t0 + r, :, :r].transpose(1, 0, 2)     # [H, r, r]
        nc = n[t0:t0 + r, :, :r].transpose(1, 0, 2)
        I = np.eye(r)[None]
        res = np.abs((I + nc) @ ac - I).max()
        worst = max(worst, float(res))
    return worst


def paper_metrics(x_gpu: np.ndarray, x_ref: np.ndarray):
    """The three forward errors of Sec. 4.1: max abs, max rel (over |ref| > 1e-30), Frobenius relative."""
    d = np.abs(x_gpu.astype(np.float64) - x_ref)
    m = np.abs(x_ref) > 1e-30
    return {"max_abs": float(d.max()), "max_rel": float((d[m] / np.abs(x_ref[m])).max()) if m.any() else 0.0,
            "fro_rel": float(np.sqrt((d ** 2).sum()) / max(np.sqrt((x_ref ** 2).sum()), 1e-300))}
