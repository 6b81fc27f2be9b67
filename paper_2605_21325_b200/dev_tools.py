"""Read-outs of the development build (``python -m paper_2605_21325_b200.build --dev`` -> libtri_inv_dev.so, compiled with
-DTRI_INV_PHASE_CLOCKS; the default build has none of this).

    python -m paper_2605_21325_b200.dev_tools phases   [--config 2]     cycles between the kernel's phase marks, per warp of CTA 0
    python -m paper_2605_21325_b200.dev_tools timeline [--config 2]     when each CTA ran its first / last instruction, and on which SM
    python -m paper_2605_21325_b200.dev_tools scan_chunk [--config 2]   clock of every step of one chunk of the chunk scan, per warp of CTA 0

The first two run the fused call of one configuration a few times on cuda:0, the third the chunk scan.  The development build's TRI_INV_GRID_CAP=<n>
environment variable caps the grid (to vary the resident CTAs per SM).
"""
from __future__ import annotations

import argparse
import ctypes
import os
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
os.environ.setdefault("TRI_INV_LIB", os.path.join(PKG, "libtri_inv_dev.so"))
sys.path.insert(0, os.path.dirname(PKG))

PHASES = ["top", "gram wait", "gate", "leaf+sync", "merge16", "merge32(+64)", "read X / store A", "A'+sync", "W wait", "W store",
          "U wait", "U store+end"]


def main():
    import numpy as np
    import torch
    from paper_2605_21325_b200 import binding as b, workloads as wl
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["phases", "build_phases", "raw_phases", "timeline", "scan_chunk", "kda_phases"])
    ap.add_argument("--config", type=int, default=2)
    args = ap.parse_args()
    inp = wl.config(args.config)
    if args.what == "raw_phases":   # the same shape with the inputs the projections hand over (un-normalised keys, logits)
        inp = wl.make_raw(inp.name + "_raw", inp.B, inp.T, inp.H, inp.d_k, inp.C, inp.kv_dtype, 2000 + args.config, inp.cu_seqlens)
    d = b.to_device(inp)
    if args.what == "scan_chunk":
        return scan_chunk(b, wl, inp, d)
    if args.what == "kda_phases":
        return kda_phases(b, wl, inp, d)
    out = (torch.empty((inp.B, inp.T, inp.H, inp.C), dtype=torch.float32, device="cuda"), torch.empty_like(d["K"]), torch.empty_like(d["V"]))
    L = b.load()
    if not hasattr(L, "tri_inv_debug_counters"):
        raise SystemExit("%s is not a development build" % b.LIB_PATH)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    words = (ctypes.c_int * 128)()
    for _ in range(4):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        if args.what == "raw_phases":
            b.fused_raw(d["K"], d["V"], d["beta"], d["g"], inp.C, cu_seqlens=inp.cu_seqlens, out=(out[0], out[1], out[2], None, None))
        elif args.what == "build_phases":
            b.build(d["K"], d["beta"], d["g"], inp.C, cu_seqlens=inp.cu_seqlens, out=out[0])
        else:
            b.fused(d["K"], d["V"], d["beta"], d["g"], inp.C, cu_seqlens=inp.cu_seqlens, out=out)
        e1.record()
        torch.cuda.synchronize()
        L.tri_inv_debug_counters(words)          # read and clear: the last launch's counters stay in `words`
    resident = 148 * ((6 if args.what == "build_phases" else 4) if inp.C == 64 else 2)
    grid = min(int(os.environ.get("TRI_INV_GRID_CAP", resident)), resident, inp.n_matrices)
    if args.what in ("phases", "build_phases", "raw_phases"):
        items = -(-inp.n_matrices // grid)      # items of CTA 0, about
        for w in range(inp.C // 16):
            v = [words[8 + 12 * w + k] / items for k in range(12)]
            print("warp %d: " % w + ", ".join("%s %.0f" % (n, x) for n, x in zip(PHASES, v)) + "; total %.0f cycles per item" % sum(v))
        return
    buf = (ctypes.c_ulonglong * (grid * 4))()
    L.tri_inv_debug_cta_times(buf, grid * 4)
    t = np.array(buf[:], dtype=np.int64).reshape(grid, 4)
    t0 = t[:, 0].min()
    start, end, sm = (t[:, 0] - t0) / 1e3, (t[:, 2] - t0) / 1e3, t[:, 3]
    print("launch (CUDA events): %.1f us, grid %d" % (e0.elapsed_time(e1) * 1e3, grid))
    print("first instruction of a CTA, us after the first: min %.1f median %.1f max %.1f" % (start.min(), np.median(start), start.max()))
    print("last instruction of a CTA: min %.1f median %.1f max %.1f" % (end.min(), np.median(end), end.max()))
    print("SMs by number of CTAs they ran:", np.bincount(np.bincount(sm.astype(int))).tolist())


SCAN_COMPUTE = ["loop top", "last chunk's O written", "P1 seen", "chain: U tile seen | output: P loads done", "chain: W S loaded",
                "chain: U~' arrived | output: first 16 rows of P", "chain: U~ arrived | output: P arrived", "P3 seen", "state updated",
                "S^T stored", "S^T arrived"]
SCAN_CONTROL = ["state operand seen", "P1 issued", "copies issued", "U~' seen", "P3 issued", "U~ and P seen", "PU issued", "copies seen",
                "", "loop top"]


KDA_PHASES = ["K, G waited", "K+ K- pass", "Gram wait", "gate", "leaf", "merges", "A, A' pass", "W wait", "W loaded", "W stored",
              "U wait", "U stored, end"]


def kda_phases(b, wl, inp, d):
    """Cycles per item and warp between the PHASE marks of the one-kernel per-channel call (thread block 0)."""
    import torch
    G = torch.from_numpy(wl.per_channel_gate(inp, seed=1)).cuda()
    out = (torch.empty((inp.B, inp.T, inp.H, inp.C), dtype=torch.float32, device="cuda"), torch.empty_like(d["K"]), torch.empty_like(d["V"]))
    L = b.load()
    if not hasattr(L, "tri_inv_debug_counters"):
        raise SystemExit("%s is not a development build" % b.LIB_PATH)
    words = (ctypes.c_int * 128)()
    for _ in range(3):
        L.tri_inv_debug_counters(words)
        b.fused_kda(d["K"], d["V"], G, d["beta"], inp.C, cu_seqlens=inp.cu_seqlens, out=out)
        torch.cuda.synchronize()
    L.tri_inv_debug_counters(words)
    grid = min(148 * 3, inp.n_matrices)
    items = -(-inp.n_matrices // grid)
    for w in range(4):
        v = [words[8 + 12 * w + k] / items for k in range(12)]
        print("warp %d: " % w + ", ".join("%s %.0f" % (n, x) for n, x in zip(KDA_PHASES, v)) + "; total %.0f cycles per item" % sum(v))


def scan_chunk(b, wl, inp, d):
    """The development build stamps clock64 at every step of the 21st chunk of CTA 0 (macro TL in scan_kernel.cu);
    printed here in cycles from the moment the control thread sees that chunk's state operand."""
    import numpy as np
    import torch
    Q = b.kv_to_torch(wl.queries(inp, seed=1))
    W = torch.randn_like(d["K"].float()).mul_(0.1).to(torch.bfloat16)
    U = d["V"].clone()
    O = torch.empty_like(d["V"])
    L = b.load()
    if not hasattr(L, "tri_inv_debug_counters"):
        raise SystemExit("%s is not a development build" % b.LIB_PATH)
    words = (ctypes.c_int * 128)()
    for _ in range(3):
        L.tri_inv_debug_counters(words)
        b.chunk_scan(Q, d["K"], W, U, d["g"], inp.C, scale=0.1, cu_seqlens=inp.cu_seqlens, out=O, want_state=False)
        torch.cuda.synchronize()
    L.tri_inv_debug_counters(words)
    w = np.array(words[:], dtype=np.int64)[8:].reshape(10, 12)
    base = w[8, 0]
    for i in range(8):
        role = "chain " if (i & 3) < 2 else "output"
        print("warp %d (%s): " % (i, role) + ", ".join("%s %d" % (n, w[i, k] - base) for k, n in enumerate(SCAN_COMPUTE) if w[i, k]))
    print("control thread: " + ", ".join("%s %d" % (n, w[8, k] - base) for k, n in enumerate(SCAN_CONTROL) if w[8, k]))


if __name__ == "__main__":
    main()
