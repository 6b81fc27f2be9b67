"""Read-outs of the development build (``python -m paper_2605_21325_b200.build --dev`` -> libtri_inv_dev.so, compiled with
-DTRI_INV_PHASE_CLOCKS; the default build has none of this).

    python -m paper_2605_21325_b200.dev_tools phases   [--config 2]     cycles between the kernel's phase marks, per warp of CTA 0
    python -m paper_2605_21325_b200.dev_tools timeline [--config 2]     when each CTA ran its first / last instruction, and on which SM

Both run the fused call of one configuration a few times on cuda:0.  The development build's TRI_INV_GRID_CAP=<n>
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
    ap.add_argument("what", choices=["phases", "timeline"])
    ap.add_argument("--config", type=int, default=2)
    args = ap.parse_args()
    inp = wl.config(args.config)
    d = b.to_device(inp)
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
        b.fused(d["K"], d["V"], d["beta"], d["g"], inp.C, cu_seqlens=inp.cu_seqlens, out=out)
        e1.record()
        torch.cuda.synchronize()
        L.tri_inv_debug_counters(words)          # read and clear: the last launch's counters stay in `words`
    resident = 148 * (4 if inp.C == 64 else 2)
    grid = min(int(os.environ.get("TRI_INV_GRID_CAP", resident)), resident, inp.n_matrices)
    if args.what == "phases":
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


if __name__ == "__main__":
    main()
