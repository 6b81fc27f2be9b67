"""Thin ctypes binding over ``libtri_inv.so`` (the C ABI declared in ``include/tri_inv.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels.
torch is used for device memory and streams.  There is no CPU path: if the
library is missing or a call fails, these functions raise.

Tensors follow the header's layouts: K/V ``[B,T,H,d]`` (bf16 or fp32), beta/g
``[B,T,H]`` fp32, A ``[B,T,H,C]`` fp32, W/U like K/V.  All must be contiguous
CUDA tensors on the current device.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# TRI_INV_LIB selects another build of the same library (the bounds-checking debug build, a development build)
LIB_PATH = os.environ.get("TRI_INV_LIB") or os.path.join(_PKG, "libtri_inv.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_TOO_LARGE, ERR_DEBUG_CHECK = 0, 1, 2, 3, 4, 5, 6
STATIC_MAX_CHUNKS = 16384
F32, BF16 = 0, 1
BLOCK_RECURSIVE, PRODUCT_SERIES, NEWTON_SCHULZ = 0, 1, 2
LEAF_SERIES = 0x100
REFINE = 0x200
OPERANDS_F16 = 0x400
GATE_SHIFTED = 0x800


def ns_iters(m: int) -> int:
    """Method flag carrying a Newton-Schulz iteration count (1..15)."""
    return (int(m) & 0xF) << 12


FORCE_SIMT = 0x10000
W_DECAY = 0x20000

EXPORTS = ("tri_inv_build", "tri_inv_build_kda", "tri_inv_fused_kda", "tri_inv_chunk_scan_kda", "tri_inv_chunk_scan", "tri_inv_wy", "tri_inv_fused", "tri_inv_fused_raw", "tri_inv_fused_packed_static", "tri_inv_count_matrices",
           "tri_inv_fused_host", "tri_inv_fused_host_workspace", "tri_inv_selftest_wait_timeout", "tri_inv_selftest_scan_wait_timeout", "tri_inv_selftest_kda_wait_timeout", "tri_inv_selftest_bounds_check", "tri_inv_last_device_status", "tri_inv_launch_count", "tri_inv_status_string")


class Desc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32),
                ("d_k", ctypes.c_int32), ("d_v", ctypes.c_int32), ("C", ctypes.c_int32),
                ("kv_dtype", ctypes.c_int32), ("n_seqs", ctypes.c_int32),
                ("cu_seqlens", ctypes.c_void_p)]


class TriInvError(RuntimeError):
    def __init__(self, fn, status):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (fn, status_string(status), status))


_lib = None


def load():
    """Load the library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("%s not found: build it with `python -m paper_2605_21325_b200.build` "
                              "(there is no CPU fallback)" % LIB_PATH)
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, dp = ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(Desc)
        lib.tri_inv_build.argtypes = [vp, vp, vp, vp, dp, i32, vp]
        lib.tri_inv_wy.argtypes = [vp, vp, vp, vp, vp, vp, dp, vp]
        lib.tri_inv_fused.argtypes = [vp, vp, vp, vp, vp, vp, vp, dp, i32, vp]
        lib.tri_inv_build_kda.argtypes = [vp, vp, vp, vp, dp, i32, vp]
        lib.tri_inv_build_kda.restype = i32
        lib.tri_inv_chunk_scan.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, dp, vp]
        lib.tri_inv_chunk_scan.restype = i32
        if hasattr(lib, "tri_inv_fused_kda"):
            lib.tri_inv_chunk_scan_kda.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, dp, vp]
            lib.tri_inv_chunk_scan_kda.restype = i32
            lib.tri_inv_fused_kda.argtypes = [vp, vp, vp, vp, vp, vp, vp, dp, i32, vp]
            lib.tri_inv_fused_kda.restype = i32
        lib.tri_inv_fused_raw.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, dp, i32, vp]
        lib.tri_inv_fused_raw.restype = i32
        lib.tri_inv_fused_packed_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, dp, i32, vp]
        lib.tri_inv_fused_packed_static.restype = i32
        if hasattr(lib, "tri_inv_fused_host"):
            lib.tri_inv_fused_host_workspace.argtypes = [dp, ctypes.POINTER(ctypes.c_size_t)]
            lib.tri_inv_fused_host_workspace.restype = i32
            lib.tri_inv_fused_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, dp, i32, vp]
            lib.tri_inv_fused_host.restype = i32
        if hasattr(lib, "tri_inv_selftest_bounds_check"):
            lib.tri_inv_selftest_bounds_check.argtypes = [vp, vp, vp, vp, vp, vp, vp, dp, vp]
            lib.tri_inv_selftest_bounds_check.restype = i32
        if hasattr(lib, "tri_inv_selftest_scan_wait_timeout"):
            lib.tri_inv_selftest_scan_wait_timeout.argtypes = [vp, vp, vp, vp, vp, vp, dp, ctypes.c_uint64, vp]
            lib.tri_inv_selftest_scan_wait_timeout.restype = i32
        if hasattr(lib, "tri_inv_selftest_kda_wait_timeout"):
            lib.tri_inv_selftest_kda_wait_timeout.argtypes = [vp, vp, vp, vp, vp, vp, vp, dp, ctypes.c_uint64, vp]
            lib.tri_inv_selftest_kda_wait_timeout.restype = i32
        if hasattr(lib, "tri_inv_selftest_wait_timeout"):
            lib.tri_inv_selftest_wait_timeout.argtypes = [vp, vp, vp, vp, vp, vp, vp, dp, ctypes.c_uint64, ctypes.POINTER(ctypes.c_int), vp]
            lib.tri_inv_selftest_wait_timeout.restype = i32
        lib.tri_inv_count_matrices.argtypes = [dp, ctypes.POINTER(ctypes.c_int64)]
        lib.tri_inv_last_device_status.argtypes = [ctypes.POINTER(ctypes.c_int)]
        for f in ("tri_inv_build", "tri_inv_wy", "tri_inv_fused", "tri_inv_count_matrices", "tri_inv_last_device_status"):
            getattr(lib, f).restype = i32
        lib.tri_inv_launch_count.restype = ctypes.c_int64
        lib.tri_inv_launch_count.argtypes = []
        lib.tri_inv_status_string.restype = ctypes.c_char_p
        lib.tri_inv_status_string.argtypes = [i32]
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().tri_inv_status_string(int(status)).decode()


def launch_count() -> int:
    return int(load().tri_inv_launch_count())


def last_device_status() -> int:
    out = ctypes.c_int(0)
    rc = load().tri_inv_last_device_status(ctypes.byref(out))
    if rc != OK:
        raise TriInvError("tri_inv_last_device_status", rc)
    return out.value


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("K/V must be float32 or bfloat16, got %s" % t.dtype)


def make_desc(B, T, H, d_k, d_v, C, kv_dtype, cu_seqlens=None):
    """Returns (Desc, keepalive).  ``cu_seqlens`` is a host int array of n_seqs+1 offsets or None."""
    keep = None
    ptr, n_seqs = None, 0
    if cu_seqlens is not None:
        keep = np.ascontiguousarray(np.asarray(cu_seqlens), dtype=np.int32)
        ptr, n_seqs = keep.ctypes.data, len(keep) - 1
    return Desc(B, T, H, d_k, d_v, C, kv_dtype, n_seqs, ptr), keep


def count_matrices(desc: Desc) -> int:
    out = ctypes.c_int64(0)
    rc = load().tri_inv_count_matrices(ctypes.byref(desc), ctypes.byref(out))
    if rc != OK:
        raise TriInvError("tri_inv_count_matrices", rc)
    return out.value


def _p(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def build(K, beta, g, C, method=BLOCK_RECURSIVE, cu_seqlens=None, out=None, stream=None):
    """A = (I+N)^{-1} per chunk -> A [B,T,H,C] fp32 (rows of real tokens written)."""
    B, T, H, d_k = K.shape
    desc, keep = make_desc(B, T, H, d_k, d_k, C, _dtype_code(K), cu_seqlens)
    A = torch.zeros((B, T, H, C), dtype=torch.float32, device=K.device) if out is None else out
    rc = load().tri_inv_build(_p(K), _p(beta), _p(g), _p(A), ctypes.byref(desc), int(method), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_build", rc)
    return A


def build_kda(K, G, beta, C, method=BLOCK_RECURSIVE, cu_seqlens=None, out=None, stream=None):
    """Per-channel decay: A = (I+N)^{-1} with N_ij = beta_i sum_c K_ic K_jc exp(G_ic - G_jc); G [B,T,H,d] fp32."""
    B, T, H, d_k = K.shape
    desc, keep = make_desc(B, T, H, d_k, d_k, C, _dtype_code(K), cu_seqlens)
    A = torch.zeros((B, T, H, C), dtype=torch.float32, device=K.device) if out is None else out
    rc = load().tri_inv_build_kda(_p(K), _p(G), _p(beta), _p(A), ctypes.byref(desc), int(method), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_build_kda", rc)
    return A


def chunk_scan(Q, K, W, U, g, C, scale=1.0, S0=None, cu_seqlens=None, out=None, want_state=True, state_out=None, stream=None):
    """O, S_final of the chunk form of the layer's recurrence from the decay-weighted W and U (tri_inv_chunk_scan)."""
    B, T, H, d_k = K.shape
    d_v = U.shape[3]
    desc, keep = make_desc(B, T, H, d_k, d_v, C, _dtype_code(K), cu_seqlens)
    n_seqs = B if cu_seqlens is None else len(cu_seqlens) - 1
    O = torch.empty((B, T, H, d_v), dtype=U.dtype, device=K.device) if out is None else out
    S = state_out if state_out is not None else (
        torch.empty((n_seqs, H, d_k, d_v), dtype=torch.float32, device=K.device) if want_state else None)
    rc = load().tri_inv_chunk_scan(_p(Q), _p(K), _p(W), _p(U), _p(g), _p(S0), _p(O), _p(S), float(scale),
                                   ctypes.byref(desc), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_chunk_scan", rc)
    return O, S


def fused_kda(K, V, G, beta, C, method=BLOCK_RECURSIVE, cu_seqlens=None, out=None, stream=None):
    """Per-channel decay through the WY step -> (A, W, U) with W = A diag(beta) (K * exp G), U = A diag(beta) V."""
    B, T, H, d_k = K.shape
    d_v = V.shape[-1]
    desc, keep = make_desc(B, T, H, d_k, d_v, C, _dtype_code(K), cu_seqlens)
    if out is None:
        out = (torch.zeros((B, T, H, C), dtype=torch.float32, device=K.device), torch.zeros_like(K), torch.zeros_like(V))
    A, W, U = out
    rc = load().tri_inv_fused_kda(_p(K), _p(V), _p(G), _p(beta), _p(A), _p(W), _p(U), ctypes.byref(desc), int(method), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_fused_kda", rc)
    return A, W, U


def chunk_scan_kda(Q, K, W, U, G, C, scale=1.0, S0=None, cu_seqlens=None, out=None, want_state=True, stream=None):
    """tri_inv_chunk_scan_kda: the chunk scan with one decay per key feature -> (O, S_final or None)."""
    B, T, H, d_k = K.shape
    d_v = U.shape[3]
    desc, keep = make_desc(B, T, H, d_k, d_v, C, _dtype_code(K), cu_seqlens)
    n_seqs = B if cu_seqlens is None else len(cu_seqlens) - 1
    O = torch.empty((B, T, H, d_v), dtype=U.dtype, device=K.device) if out is None else out
    S = torch.empty((n_seqs, H, d_k, d_v), dtype=torch.float32, device=K.device) if want_state else None
    rc = load().tri_inv_chunk_scan_kda(_p(Q), _p(K), _p(W), _p(U), _p(G), _p(S0), _p(O), _p(S), float(scale),
                                       ctypes.byref(desc), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_chunk_scan_kda", rc)
    return O, S


def gdn_forward(Q, K, V, beta, g, C, scale=1.0, S0=None, method=BLOCK_RECURSIVE, cu_seqlens=None, stream=None):
    """The whole layer in two launches: fused build + inversion + WY with the decay-weighted W, then the chunk scan."""
    _, W, U = fused(K, V, beta, g, C, method=method | W_DECAY, cu_seqlens=cu_seqlens, want_A=False, stream=stream)
    return chunk_scan(Q, K, W, U, g, C, scale=scale, S0=S0, cu_seqlens=cu_seqlens, stream=stream)


def wy(A, K, V, beta, cu_seqlens=None, out=None, stream=None):
    """W = A diag(beta) K, U = A diag(beta) V from a stored A."""
    B, T, H, d_k = K.shape
    C = A.shape[-1]
    d_v = V.shape[-1] if V is not None else d_k
    desc, keep = make_desc(B, T, H, d_k, d_v, C, _dtype_code(K), cu_seqlens)
    if out is None:
        W = torch.zeros_like(K)
        U = torch.zeros_like(V) if V is not None else None
    else:
        W, U = out
    rc = load().tri_inv_wy(_p(A), _p(K), _p(V), _p(beta), _p(W), _p(U), ctypes.byref(desc), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_wy", rc)
    return W, U


def fused(K, V, beta, g, C, method=BLOCK_RECURSIVE, cu_seqlens=None, want_A=True, out=None, stream=None):
    """Fused build + invert + WY -> (A or None, W, U)."""
    B, T, H, d_k = K.shape
    d_v = V.shape[-1]
    desc, keep = make_desc(B, T, H, d_k, d_v, C, _dtype_code(K), cu_seqlens)
    if out is None:
        A = torch.zeros((B, T, H, C), dtype=torch.float32, device=K.device) if want_A else None
        W, U = torch.zeros_like(K), torch.zeros_like(V)
    else:
        A, W, U = out
    rc = load().tri_inv_fused(_p(K), _p(V), _p(beta), _p(g), _p(A), _p(W), _p(U), ctypes.byref(desc), int(method), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_fused", rc)
    return A, W, U


def fused_raw(K_raw, V, beta_logit, gate_logit, C, method=BLOCK_RECURSIVE, cu_seqlens=None, want_A=True,
              want_gates=False, out=None, stream=None):
    """Fused call that also runs the layer's front end (sigmoid, log-sigmoid + chunk cumsum, key
    normalisation) -> (A or None, W, U, beta or None, g or None)."""
    B, T, H, d_k = K_raw.shape
    d_v = V.shape[-1]
    desc, keep = make_desc(B, T, H, d_k, d_v, C, _dtype_code(K_raw), cu_seqlens)
    if out is None:
        A = torch.zeros((B, T, H, C), dtype=torch.float32, device=K_raw.device) if want_A else None
        W, U = torch.zeros_like(K_raw), torch.zeros_like(V)
        bo = torch.zeros((B, T, H), dtype=torch.float32, device=K_raw.device) if want_gates else None
        go = torch.zeros((B, T, H), dtype=torch.float32, device=K_raw.device) if want_gates else None
    else:
        A, W, U, bo, go = out
    rc = load().tri_inv_fused_raw(_p(K_raw), _p(V), _p(beta_logit), _p(gate_logit), _p(A), _p(W), _p(U), _p(bo), _p(go),
                                  ctypes.byref(desc), int(method), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_fused_raw", rc)
    return A, W, U, bo, go


def fused_packed_static(K, V, beta, g, C, cu_seqlens, method=BLOCK_RECURSIVE, out=None, stream=None):
    """Packed-sequence fused call through the entry point that makes no allocation of its own
    (the chunk table sits in a fixed array inside the library).  ``out`` = (A or None, W, U) must be
    given by callers that really cannot allocate; without it the outputs are allocated here with torch."""
    B, T, H, d_k = K.shape
    d_v = V.shape[-1]
    desc, keep = make_desc(B, T, H, d_k, d_v, C, _dtype_code(K), cu_seqlens)
    if out is None:
        out = (torch.zeros((B, T, H, C), dtype=torch.float32, device=K.device), torch.zeros_like(K), torch.zeros_like(V))
    A, W, U = out
    rc = load().tri_inv_fused_packed_static(_p(K), _p(V), _p(beta), _p(g), _p(A), _p(W), _p(U), ctypes.byref(desc),
                                            int(method), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_fused_packed_static", rc)
    return A, W, U


def selftest_wait_timeout(K, V, beta, g, C, wait_limit_ns, out, stream=None):
    """tri_inv_selftest_wait_timeout: the fused call with short wait limits and one product left out, so that
    one thread block's wait gives up.  ``out`` = (A, W, U).  Returns True when the work counters are back at zero."""
    B, T, H, d_k = K.shape
    desc, keep = make_desc(B, T, H, d_k, V.shape[-1], C, _dtype_code(K), None)
    A, W, U = out
    idle = ctypes.c_int(0)
    rc = load().tri_inv_selftest_wait_timeout(_p(K), _p(V), _p(beta), _p(g), _p(A), _p(W), _p(U), ctypes.byref(desc),
                                              ctypes.c_uint64(int(wait_limit_ns)), ctypes.byref(idle), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_selftest_wait_timeout", rc)
    return bool(idle.value)


def selftest_kda_wait_timeout(K, V, G, beta, C, wait_limit_ns, out, stream=None):
    """tri_inv_selftest_kda_wait_timeout: the per-channel fused call (``V`` None: the per-channel build) with short wait limits
    and one product of the first thread block left out.  ``out`` = (A, W, U) or (A, None, None)."""
    B, T, H, d_k = K.shape
    desc, keep = make_desc(B, T, H, d_k, d_k if V is None else V.shape[-1], C, _dtype_code(K), None)
    A, W, U = out
    none = ctypes.c_void_p(None)
    rc = load().tri_inv_selftest_kda_wait_timeout(_p(K), none if V is None else _p(V), _p(G), _p(beta), _p(A),
                                                  none if W is None else _p(W), none if U is None else _p(U), ctypes.byref(desc),
                                                  ctypes.c_uint64(int(wait_limit_ns)), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_selftest_kda_wait_timeout", rc)
    return out


def selftest_scan_wait_timeout(Q, K, W, U, g, C, wait_limit_ns, out, stream=None):
    """tri_inv_selftest_scan_wait_timeout: the chunk scan with short wait limits and one product of the first thread block
    left out, so that this block's waits give up.  ``out`` = O."""
    B, T, H, d_k = K.shape
    desc, keep = make_desc(B, T, H, d_k, U.shape[-1], C, _dtype_code(K), None)
    rc = load().tri_inv_selftest_scan_wait_timeout(_p(Q), _p(K), _p(W), _p(U), _p(g), _p(out), ctypes.byref(desc),
                                                   ctypes.c_uint64(int(wait_limit_ns)), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_selftest_scan_wait_timeout", rc)
    return out


def fused_host_workspace_bytes(B, T, H, d_k, d_v, C, kv_dtype, cu_seqlens=None) -> int:
    desc, keep = make_desc(B, T, H, d_k, d_v, C, kv_dtype, cu_seqlens)
    n = ctypes.c_size_t(0)
    rc = load().tri_inv_fused_host_workspace(ctypes.byref(desc), ctypes.byref(n))
    if rc != OK:
        raise TriInvError("tri_inv_fused_host_workspace", rc)
    return int(n.value)


def fused_host(hK, hV, hbeta, hg, C, hA, hW, hU, workspace, method=BLOCK_RECURSIVE, cu_seqlens=None, stream=None):
    """tri_inv_fused_host: every tensor argument is a HOST tensor (pinned for asynchronous copies), ``workspace`` a CUDA
    uint8 tensor of at least ``fused_host_workspace_bytes`` bytes.  hA may be None.  Enqueues and returns."""
    B, T, H, d_k = hK.shape
    desc, keep = make_desc(B, T, H, d_k, hV.shape[-1], C, _dtype_code(hK), cu_seqlens)
    hp = lambda t: None if t is None else ctypes.c_void_p(t.data_ptr())
    rc = load().tri_inv_fused_host(hp(hK), hp(hV), hp(hbeta), hp(hg), hp(hA), hp(hW), hp(hU), ctypes.c_void_p(workspace.data_ptr()),
                                   ctypes.c_size_t(workspace.numel() * workspace.element_size()), ctypes.byref(desc), int(method), _stream(stream))
    if rc != OK:
        raise TriInvError("tri_inv_fused_host", rc)


class HostPipeline:
    """tri_inv_fused for callers whose tensors live in pinned host memory.

    The batch is cut into slices (whole sequences when B >= n_slices, else runs of whole chunks of one sequence) and
    each slice goes host -> device, through the fused kernel, and device -> host on its own stream, so the
    upload of one slice overlaps the kernel of the previous one and the download of the one before.  Device
    buffers are allocated once here; ``run`` allocates nothing.  Dense mode only (packed batches: one slice)."""

    def __init__(self, B, T, H, d_k, d_v, C, dtype=torch.bfloat16, n_slices=8, n_streams=3, cu_seqlens=None, device="cuda"):
        self.shape = (B, T, H, d_k, d_v, C)
        self.cu_seqlens = cu_seqlens
        self.K = torch.empty((B, T, H, d_k), dtype=dtype, device=device)
        self.V = torch.empty((B, T, H, d_v), dtype=dtype, device=device)
        self.beta = torch.empty((B, T, H), dtype=torch.float32, device=device)
        self.g = torch.empty((B, T, H), dtype=torch.float32, device=device)
        self.A = torch.empty((B, T, H, C), dtype=torch.float32, device=device)
        self.W, self.U = torch.empty_like(self.K), torch.empty_like(self.V)
        # a slice is (sequence range, token range): whole sequences, or a run of whole chunks of one sequence --
        # either way a contiguous block of every tensor
        if cu_seqlens is not None or B * (T // C) < 2:
            self.slices = [(slice(None), slice(None))]
        elif B >= n_slices:
            step = -(-B // n_slices)
            self.slices = [(slice(b, min(b + step, B)), slice(None)) for b in range(0, B, step)]
        else:
            per_seq = max(1, min(n_slices // B, T // C))
            step = -(-(T // C) // per_seq) * C
            self.slices = [(slice(b, b + 1), slice(t, min(t + step, T))) for b in range(B) for t in range(0, T, step)]
        self.streams = [torch.cuda.Stream(device=device) for _ in range(min(n_streams, len(self.slices)))]

    @staticmethod
    def _cut(t, brng, trng):
        return t[brng, trng]

    def run(self, hK, hV, hbeta, hg, hA, hW, hU, method=BLOCK_RECURSIVE):
        """All arguments are pinned host tensors of the full batch; hA may be None.  Returns after enqueueing;
        the current stream is made to wait for every slice, so a synchronize (or event) on it covers the call."""
        C = self.shape[5]
        cur = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(cur)
        for n, (brng, trng) in enumerate(self.slices):
            st = self.streams[n % len(self.streams)]
            st.wait_event(start)
            with torch.cuda.stream(st):
                cut = lambda t: self._cut(t, brng, trng)
                for dst, src in ((self.K, hK), (self.V, hV), (self.beta, hbeta), (self.g, hg)):
                    cut(dst).copy_(cut(src), non_blocking=True)
                fused(cut(self.K), cut(self.V), cut(self.beta), cut(self.g), C, method=method, cu_seqlens=self.cu_seqlens,
                      out=(cut(self.A) if hA is not None else None, cut(self.W), cut(self.U)), stream=st)
                if hA is not None:
                    cut(hA).copy_(cut(self.A), non_blocking=True)
                cut(hW).copy_(cut(self.W), non_blocking=True)
                cut(hU).copy_(cut(self.U), non_blocking=True)
        for st in self.streams:
            cur.wait_stream(st)


# ---- moving workloads.Inputs (numpy, host) to the device and results back -------------------

def kv_to_torch(a: np.ndarray, device="cuda", pin=False) -> torch.Tensor:
    """float32 array or uint16 bf16 bit patterns -> torch tensor of the matching dtype."""
    t = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)
    if device == "cpu":
        return t.pin_memory() if pin else t
    return t.to(device)


def to_device(inp, device="cuda"):
    """workloads.Inputs -> dict of CUDA tensors."""
    return {"K": kv_to_torch(inp.K, device), "V": kv_to_torch(inp.V, device),
            "beta": torch.from_numpy(inp.beta).to(device), "g": torch.from_numpy(inp.g).to(device)}


def to_numpy_f64(t: torch.Tensor) -> np.ndarray:
    """Device result -> float64 numpy (bf16 widened exactly)."""
    return t.detach().to("cpu").to(torch.float64).numpy()
