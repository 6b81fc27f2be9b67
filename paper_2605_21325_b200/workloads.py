"""Seeded synthetic inputs for the chunkwise delta-rule triangular inversion.

This module only draws and lays out inputs (keys, values, betas, cumulative
log-decays, packed sequence offsets).  It holds none of the method's
arithmetic, so both the CPU oracle's tests and the CUDA path's tests and bench
may use it.  Everything is numpy on the host; bf16 tensors are carried as
uint16 bit patterns so that both sides see the same rounded values.

The five named configurations stand in for the GDN layers of Qwen-class models
and the Kimi-Linear long-context case (shapes, sizes and value distributions
only; no model weights or activations are involved):

  1  B=1  T=256    H=2   d=64   C=64   fp32          (8 chunk matrices)
  2  B=4  T=4096   H=16  d=128  C=64   bf16 K,V      (4096)
  3  B=1  T=32768  H=32  d=128  C=64   bf16          (16384)
  4  B=2  T=8192   H=16  d=128  C=128  bf16          (2048 of 128x128)
  5  64 packed sequences, lengths U{1..2048}, H=16, d=128, C=64, bf16,
     un-normalised keys N(0,1)/sqrt(d), beta ~ U(0.9,1), g = 0

Draw order per config is fixed: K, V, beta noise, g noise (lengths first for 5).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

F32, BF16 = 0, 1


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the 16-bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Inputs:
    """One workload: storage arrays plus its shape.  K/V are float32 or uint16 (bf16 bits)."""
    name: str
    B: int
    T: int
    H: int
    d_k: int
    d_v: int
    C: int
    kv_dtype: int
    K: np.ndarray
    V: np.ndarray
    beta: np.ndarray
    g: np.ndarray
    cu_seqlens: np.ndarray | None = None
    meta: dict = field(default_factory=dict)

    def seq_bounds(self):
        if self.cu_seqlens is None:
            return [(b * self.T, (b + 1) * self.T) for b in range(self.B)]
        cu = self.cu_seqlens
        return [(int(cu[i]), int(cu[i + 1])) for i in range(len(cu) - 1)]

    def chunk_list(self):
        """[(first flat token, real rows)] for every chunk, in flat token order."""
        out = []
        for beg, end in self.seq_bounds():
            t = beg
            while t < end:
                out.append((t, min(self.C, end - t)))
                t += self.C
        return out

    @property
    def n_matrices(self) -> int:
        return len(self.chunk_list()) * self.H

    def kv_as_f32(self, which="K") -> np.ndarray:
        a = getattr(self, which)
        return a if a.dtype == np.float32 else bf16_bits_to_f32(a)


def _store(x: np.ndarray, kv_dtype: int) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.float32) if kv_dtype == F32 else f32_to_bf16_bits(x)


def _chunk_cumsum(x: np.ndarray, bounds, C: int) -> np.ndarray:
    """Cumulative sum along flat tokens restarting at every chunk start.  x is [tokens, H]."""
    out = np.empty_like(x)
    for beg, end in bounds:
        t = beg
        while t < end:
            e = min(t + C, end)
            out[t:e] = np.cumsum(x[t:e], axis=0, dtype=np.float32)
            t = e
    return out


def make(name, B, T, H, d_k, d_v, C, kv_dtype, seed, kind="gdn", cu_seqlens=None, rng=None) -> Inputs:
    """Draw one workload.

    kind "gdn":    K,V ~ N(0,1), K rows L2-normalised in fp32 before storage rounding;
                   beta = sigmoid(N(0,1)); g = within-chunk cumsum of logsigmoid(N(2,1)).
    kind "stress": K ~ N(0,1)/sqrt(d) un-normalised, V ~ N(0,1); beta ~ U(0.9,1); g = 0.
    """
    rng = np.random.default_rng(seed) if rng is None else rng
    K = rng.standard_normal((B, T, H, d_k), dtype=np.float32)
    V = rng.standard_normal((B, T, H, d_v), dtype=np.float32)
    if kind == "gdn":
        K /= np.sqrt((K.astype(np.float32) ** 2).sum(axis=-1, keepdims=True, dtype=np.float32))
        zb = rng.standard_normal((B, T, H), dtype=np.float32)
        zg = rng.standard_normal((B, T, H), dtype=np.float32) + np.float32(2.0)
        beta = (1.0 / (1.0 + np.exp(-zb.astype(np.float64)))).astype(np.float32)
        logsig = (-np.log1p(np.exp(-zg.astype(np.float64)))).astype(np.float32)
        bounds = [(b * T, (b + 1) * T) for b in range(B)] if cu_seqlens is None else \
                 [(int(cu_seqlens[i]), int(cu_seqlens[i + 1])) for i in range(len(cu_seqlens) - 1)]
        g = _chunk_cumsum(logsig.reshape(B * T, H), bounds, C).reshape(B, T, H)
    elif kind == "stress":
        K *= np.float32(1.0 / np.sqrt(d_k))
        beta = rng.uniform(0.9, 1.0, size=(B, T, H)).astype(np.float32)
        g = np.zeros((B, T, H), dtype=np.float32)
    else:
        raise ValueError(kind)
    cu = None if cu_seqlens is None else np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    return Inputs(name, B, T, H, d_k, d_v, C, kv_dtype, _store(K, kv_dtype), _store(V, kv_dtype),
                  np.ascontiguousarray(beta), np.ascontiguousarray(g), cu, {"kind": kind, "seed": seed})


def make_raw(name, B, T, H, d, C, kv_dtype, seed, cu_seqlens=None):
    """Inputs of the fused front end: un-normalised keys K ~ N(0,1) (row norms around sqrt(d)), values
    V ~ N(0,1), beta logits ~ N(0,1) and gate logits ~ N(2,1) -- what the projections of a
    Gated-DeltaNet layer hand over before sigmoid, log-sigmoid + cumsum and key normalisation.
    Returned as an Inputs whose ``beta`` holds the beta logits and ``g`` the gate logits."""
    rng = np.random.default_rng(seed)
    K = rng.standard_normal((B, T, H, d), dtype=np.float32)
    V = rng.standard_normal((B, T, H, d), dtype=np.float32)
    zb = rng.standard_normal((B, T, H), dtype=np.float32)
    zg = rng.standard_normal((B, T, H), dtype=np.float32) + np.float32(2.0)
    cu = None if cu_seqlens is None else np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    return Inputs(name, B, T, H, d, d, C, kv_dtype, _store(K, kv_dtype), _store(V, kv_dtype), zb, zg, cu,
                  {"kind": "raw", "seed": seed})


def per_channel_gate(inp: Inputs, seed: int, mean: float = 2.0) -> np.ndarray:
    """Cumulative per-channel log-decay G [B,T,H,d_k] fp32 for the per-channel (KDA-type) variant:
    log sigmoid(N(mean,1)) per token and channel, summed along the tokens of each chunk.  mean = 2 is the configurations'
    gate (about -0.15 per token); a lower mean decays faster (mean = -0.5: about -1 per token)."""
    rng = np.random.default_rng(seed)
    z = rng.standard_normal((inp.B * inp.T, inp.H * inp.d_k), dtype=np.float32) + np.float32(mean)
    ls = (-np.log1p(np.exp(-z.astype(np.float64)))).astype(np.float32)
    G = _chunk_cumsum(ls, inp.seq_bounds(), inp.C)
    return np.ascontiguousarray(G.reshape(inp.B, inp.T, inp.H, inp.d_k))


def queries(inp: Inputs, seed: int):
    """Queries for the layer's read step: Q ~ N(0,1) rows L2-normalised (as the keys are), in the storage
    type of K.  [B,T,H,d_k]."""
    rng = np.random.default_rng(seed)
    Q = rng.standard_normal((inp.B, inp.T, inp.H, inp.d_k), dtype=np.float32)
    Q /= np.sqrt((Q ** 2).sum(axis=-1, keepdims=True, dtype=np.float32))
    return _store(Q, inp.kv_dtype)


def initial_state(inp: Inputs, seed: int) -> np.ndarray:
    """A carried-in recurrent state S0 [n_sequences,H,d_k,d_v] fp32 ~ N(0,1)/sqrt(d_k) (decode-after-prefill case)."""
    rng = np.random.default_rng(seed)
    n = inp.B if inp.cu_seqlens is None else len(inp.cu_seqlens) - 1
    return (rng.standard_normal((n, inp.H, inp.d_k, inp.d_v), dtype=np.float32) / np.float32(np.sqrt(inp.d_k)))


def ragged_lengths(n_seqs: int, max_len: int, rng) -> np.ndarray:
    lens = rng.integers(1, max_len + 1, size=n_seqs)
    return np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)


SEEDS = {1: 1001, 2: 1002, 3: 1003, 4: 1004, 5: 1005}


def config(cfg: int, shrink: int = 1) -> Inputs:
    """The named configurations.  ``shrink`` > 1 divides the token count (and, for 5,
    the number of sequences) to give a quick case with the same structure."""
    seed = SEEDS[cfg]
    if cfg == 1:
        return make("cfg1_fp32_small", 1, 256 // min(shrink, 4), 2, 64, 64, 64, F32, seed)
    if cfg == 2:
        return make("cfg2_qwen_gdn_prefill", 4, 4096 // shrink, 16, 128, 128, 64, BF16, seed)
    if cfg == 3:
        return make("cfg3_kimi_long_context", 1, 32768 // shrink, 32, 128, 128, 64, BF16, seed)
    if cfg == 4:
        return make("cfg4_chunk128", 2, 8192 // shrink, 16, 128, 128, 128, BF16, seed)
    if cfg == 5:
        rng = np.random.default_rng(seed)
        cu = ragged_lengths(max(64 // shrink, 2), 2048, rng)
        return make("cfg5_ragged_stress", 1, int(cu[-1]), 16, 128, 128, 64, BF16, seed,
                    kind="stress", cu_seqlens=cu, rng=rng)
    raise ValueError("unknown config %r" % cfg)


def paper_timing_case(T: int, C: int = 64) -> Inputs:
    """Shape of the paper's kernel timing experiment (Sec. 5.1): batch 32, 4 heads, sequence length T up to 16K.
    The head dimension is not stated there; 128 is assumed.  Same value distributions as the GDN configs."""
    return make("paper_timing_B32_H4_T%d_C%d" % (T, C), 32, T, 4, 128, 128, C, BF16, 1100 + T // 1024)


def first_difference_case(B, T, H, d, C, kv_dtype, cu_seqlens=None) -> Inputs:
    """Every key equals the same unit vector e_0, beta = 1, g = 0, so N is the all-ones
    strictly lower matrix (the example of Sec. 3.2) and every value involved is exactly
    representable in bf16 and fp32."""
    K = np.zeros((B, T, H, d), dtype=np.float32)
    K[..., 0] = 1.0
    V = np.ones((B, T, H, d), dtype=np.float32)
    beta = np.ones((B, T, H), dtype=np.float32)
    g = np.zeros((B, T, H), dtype=np.float32)
    cu = None if cu_seqlens is None else np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    return Inputs("first_difference", B, T, H, d, d, C, kv_dtype, _store(K, kv_dtype), _store(V, kv_dtype),
                  beta, g, cu, {"kind": "first_difference"})


def correlated_keys_case(B, T, H, d, C, kv_dtype, rho, seed, d_eff=None) -> Inputs:
    """Adversarial keys for the stability report: k_i ~ sqrt(rho) u + sqrt(1-rho) z_i
    (optionally confined to the first d_eff coordinates), normalised; beta = 1, g = 0.
    Large ||N||_2 is what makes the product series lose accuracy (Sec. 3.2)."""
    rng = np.random.default_rng(seed)
    de = d if d_eff is None else d_eff
    u = rng.standard_normal((B, 1, H, de), dtype=np.float32)
    z = rng.standard_normal((B, T, H, de), dtype=np.float32)
    Kd = np.sqrt(np.float32(rho)) * u + np.sqrt(np.float32(1.0 - rho)) * z
    Kd /= np.sqrt((Kd ** 2).sum(axis=-1, keepdims=True, dtype=np.float32))
    K = np.zeros((B, T, H, d), dtype=np.float32)
    K[..., :de] = Kd
    V = rng.standard_normal((B, T, H, d), dtype=np.float32)
    beta = np.ones((B, T, H), dtype=np.float32)
    g = np.zeros((B, T, H), dtype=np.float32)
    return Inputs("correlated_rho%.2f_deff%d" % (rho, de), B, T, H, d, d, C, kv_dtype,
                  _store(K, kv_dtype), _store(V, kv_dtype), beta, g, None,
                  {"kind": "correlated", "rho": rho, "d_eff": de, "seed": seed})
