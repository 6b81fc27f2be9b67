#!/usr/bin/env python
"""Throughput of the fused build + invert + WY path on synthetic GDN-shaped data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--method block_recursive]
    python bench.py --impl reference ...        # the fp64 CPU oracle, timed on the host cores

A step is one pass of the whole hot path (stage K/V, Gram, gate, inversion, store A, WY,
store W/U: one fused kernel launch) over one batch of the chosen configuration; the default is
configuration 2 (B=4, T=4096, H=16, d=128, C=64, bf16: 4096 chunk matrices), the one the metric
is quoted on.  Inputs are seeded synthetic tensors resident in HBM before the timed region; L2 is
flushed (a 256 MiB write followed by a 256 MiB read) before every timed step; each step is timed with CUDA events on the
launching stream.  With N > 1 (torchrun, one rank per GPU) every rank runs its own copy of the
batch -- chunks are independent, so there is no collective on the data path -- and the value is
the total over ranks divided by the slowest rank's time (weak scaling).

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "chunk matrices inverted/sec (C=64, d=128, bf16) + % of roofline; max err vs fp64 oracle"
UNIT = "chunk-matrices/s"
FALLBACK_HBM_GBS = 6650.0
OUTPUTS = {"fused": "A fp32 + W,U", "raw": "A fp32 + W,U", "build": "A fp32", "kda": "A fp32", "kda_fused": "A fp32 + W,U", "wy": "W,U", "scan": "O", "layer": "O", "kda_scan": "O", "kda_layer": "O"}

def ncu_traffic_bytes_per_matrix(call, config, method):
    """DRAM bytes per chunk matrix (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture divided by the matrices
    of that launch) from profiles/ncu_traffic.json, which is rewritten whenever the kernel is captured again; None when
    that call / configuration / method has no capture."""
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_traffic.json")) as f:
            return json.load(f)["%s:cfg%d:%s" % (call, config, method)]["dram_bytes_per_matrix"]
    except Exception:
        return None


def algorithmic_bytes_per_matrix(C, d_k, d_v, elt, want_A=True, call="fused"):
    """Compulsory traffic per chunk matrix.  fused: K, V, beta, g read once; A, W, U written once.
    build: K, beta, g read; A written.  wy: the strict lower triangle of A, K, V, beta read; W, U written."""
    if call == "build":
        return C * d_k * elt + 2 * C * 4 + C * C * 4
    if call == "scan":  # Q, K, W, U, g read; O written
        return 3 * C * d_k * elt + C * d_v * elt + C * 4 + C * d_v * elt
    if call == "kda_scan":  # what ONE kernel would move: Q, K, W, U and G (fp32 per channel) read; O written (the call is two launches)
        return 3 * C * d_k * elt + C * d_v * elt + C * d_k * 4 + C * d_v * elt
    if call == "kda_layer":  # kda_fused without A, plus kda_scan
        return (C * d_k * elt + C * d_k * 4 + C * d_v * elt + C * 4 + C * d_k * elt + C * d_v * elt) + \
               (3 * C * d_k * elt + C * d_v * elt + C * d_k * 4 + C * d_v * elt)
    if call == "layer":  # fused kernel (K, V, beta, g in; W, U out, A not stored) + scan
        return (C * d_k * elt + C * d_v * elt + 2 * C * 4 + C * d_k * elt + C * d_v * elt) + \
               (3 * C * d_k * elt + C * d_v * elt + C * 4 + C * d_v * elt)
    if call == "kda":  # K, G (fp32 per channel) and beta read; A written
        return C * d_k * elt + C * d_k * 4 + C * 4 + C * C * 4
    if call == "kda_fused":  # what ONE kernel would move: K, G, V, beta read once; A, W, U written once (one kernel at C = 64, two launches at C = 128)
        return C * d_k * elt + C * d_k * 4 + C * d_v * elt + C * 4 + C * C * 4 + C * d_k * elt + C * d_v * elt
    if call == "wy":
        return C * (C - 1) // 2 * 4 + C * d_k * elt + C * d_v * elt + C * 4 + C * d_k * elt + C * d_v * elt
    b = C * d_k * elt + C * d_v * elt + 2 * C * 4 + C * d_k * elt + C * d_v * elt
    if want_A:
        b += C * C * 4
    return b


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def time_oracle(inp, target_seconds=15.0, n_threads=0):
    """The fp64 oracle, as it stands, on a bounded sample of the workload: leading tokens of each sequence."""
    import numpy as np
    import oracle
    from paper_2605_21325_b200 import workloads as wl
    cores = oracle.threads(n_threads)
    # calibrate on a small slice, then size the sample for ~target_seconds
    def run(T):
        sub = wl.Inputs(inp.name, inp.B, T, inp.H, inp.d_k, inp.d_v, inp.C, inp.kv_dtype,
                        np.ascontiguousarray(inp.K[:, :T]), np.ascontiguousarray(inp.V[:, :T]),
                        np.ascontiguousarray(inp.beta[:, :T]), np.ascontiguousarray(inp.g[:, :T]))
        t0 = time.perf_counter()
        A = oracle.build_A(sub.K, sub.beta, sub.g, sub.C, n_threads=n_threads)
        oracle.wy(A, sub.K, sub.V, sub.beta, sub.C, n_threads=n_threads)
        return sub.n_matrices, time.perf_counter() - t0
    n0, t0 = run(min(inp.T, 2 * inp.C))
    per = t0 / max(n0, 1)
    chunks = int(max(1, min(inp.T // inp.C, target_seconds / max(per * inp.B * inp.H, 1e-9))))
    # repeat the sample until about target_seconds of CPU work has been done
    n, t, passes = 0, 0.0, 0
    while t < target_seconds and passes < 1000:
        dn, dt = run(chunks * inp.C)
        n, t, passes = n + dn, t + dt, passes + 1
    return {"value": n / t, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "first %d tokens of each of the %d sequences of %s, %d passes (%d chunk matrices, %.1f s; build + WY in fp64)"
                      % (chunks * inp.C, inp.B, inp.name, passes, n, t)}, n, t


def reduce_max(value: float, device="cpu") -> float:
    """Max over ranks of a host scalar (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(local_ms_per_step: float, matrices_per_rank: int, world: int, device="cpu"):
    """Whole-job value under weak scaling: every rank processed `matrices_per_rank` per step and the job
    runs at the pace of its slowest rank."""
    ms = reduce_max(local_ms_per_step, device)
    return world * matrices_per_rank / (ms * 1e-3), ms


def run_reference(args):
    """--impl reference: the oracle is the reference arm (there is no reference implementation to install)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2605_21325_b200 import workloads as wl
    inp = wl.paper_timing_case(args.paper_T) if args.paper_T else wl.config(args.config)
    per_step_target = max(2.0, min(15.0, 120.0 / max(args.steps + args.warmup, 1)))
    vals = []
    base = None
    for s in range(args.warmup + args.steps):
        base, n, t = time_oracle(inp, target_seconds=per_step_target)
        if s >= args.warmup:
            vals.append((n, t))
    n_tot = sum(n for n, _ in vals)
    t_tot = sum(t for _, t in vals)
    value = n_tot / t_tot
    base["value"] = value
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": 1e3 * t_tot / max(len(vals), 1), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": inp.name, "B": inp.B, "T": inp.T, "H": inp.H, "d_k": inp.d_k, "d_v": inp.d_v, "C": inp.C,
                      "chunk_matrices_per_gpu": inp.n_matrices, "method": args.method, "call": args.call,
                      "outputs": OUTPUTS[args.call], "l2": "n/a (host)", "parallelism": "host cores, rank 0 only",
                      "note": "each step is a bounded sample of the workload; the oracle is forward substitution whatever `method` says"},
           "cpu_baseline": base,
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--method", default="block_recursive", choices=["block_recursive", "mixed_recursion", "product_series", "block_recursive_refined", "product_series_f16"])
    ap.add_argument("--paper-T", type=int, default=0,
                    help="instead of --config: the paper's timing shape B=32, H=4, d=128 at this sequence length (1024..16384)")
    ap.add_argument("--call", default="fused", choices=["fused", "build", "wy", "raw", "kda", "kda_fused", "scan", "layer", "kda_scan", "kda_layer"],
                    help="entry point timed: the fused path (default, the metric), tri_inv_build alone, tri_inv_wy alone, "
                         "tri_inv_fused_raw (front end folded in; same shapes, un-normalised keys and logits as inputs), "
                         "tri_inv_build_kda (per-channel decay), tri_inv_chunk_scan alone (W and U produced outside the timed "
                         "region), or the layer forward (fused call with decay-weighted W, then the scan)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-flush", action="store_true", help="skip the L2 flush between steps (profiling runs)")
    ap.add_argument("--simt", action="store_true", help="force the CUDA-core kernel")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    if args.impl == "reference":
        run_reference(args)
        return

    import numpy as np
    import torch
    import torch.distributed as dist

    import __graft_entry__ as entry
    from paper_2605_21325_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        entry.build()
    if world > 1:
        dist.barrier()
    from paper_2605_21325_b200 import binding

    method = {"block_recursive": binding.BLOCK_RECURSIVE, "mixed_recursion": binding.BLOCK_RECURSIVE | binding.LEAF_SERIES,
              "product_series": binding.PRODUCT_SERIES, "block_recursive_refined": binding.BLOCK_RECURSIVE | binding.REFINE,
              "product_series_f16": binding.PRODUCT_SERIES | binding.OPERANDS_F16}[args.method]
    if args.simt:
        method |= binding.FORCE_SIMT

    # same seeded batch on every rank (weak scaling)
    inp = wl.paper_timing_case(args.paper_T) if args.paper_T else wl.config(args.config)
    if args.call == "raw":  # same shape, inputs as the projections hand them over
        inp = wl.make_raw(inp.name + "_raw", inp.B, inp.T, inp.H, inp.d_k, inp.C, inp.kv_dtype, 2000 + args.config, inp.cu_seqlens)
    n_mat = inp.n_matrices
    dev = binding.to_device(inp)
    K, V, beta, g = dev["K"], dev["V"], dev["beta"], dev["g"]
    A = torch.empty((inp.B, inp.T, inp.H, inp.C), dtype=torch.float32, device="cuda")
    W, U = torch.empty_like(K), torch.empty_like(V)
    KDA_CALLS = ("kda", "kda_fused", "kda_scan", "kda_layer")
    G = torch.from_numpy(wl.per_channel_gate(inp, seed=3000 + args.config)).cuda() if args.call in KDA_CALLS else None
    Q = O = None
    SCAN_CALLS = ("scan", "layer", "kda_scan", "kda_layer")
    if args.call in SCAN_CALLS:  # the consumer of W and U: queries, outputs, zero initial state
        Q_host = wl.queries(inp, seed=4000 + args.config)
        Q = binding.kv_to_torch(Q_host)
        O = torch.empty_like(V)
        q_scale = float(inp.d_k) ** -0.5
    flush = None if args.no_flush else torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    flush_rd = None if args.no_flush else torch.zeros(64 * 1024 * 1024, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()

    def flush_l2():
        """Write 256 MiB (evicts everything), then read another 256 MiB so that the lines left in L2 are
        clean: the timed kernel starts with a cold L2 and does not pay for writing back the flush's data."""
        if flush is not None:
            flush.fill_(1)
            flush_rd.sum()

    def step():
        if args.call == "fused":
            binding.fused(K, V, beta, g, inp.C, method=method, cu_seqlens=inp.cu_seqlens, out=(A, W, U), stream=stream)
        elif args.call == "raw":
            binding.fused_raw(K, V, beta, g, inp.C, method=method, cu_seqlens=inp.cu_seqlens, out=(A, W, U, None, None), stream=stream)
        elif args.call == "build":
            binding.build(K, beta, g, inp.C, method=method, cu_seqlens=inp.cu_seqlens, out=A, stream=stream)
        elif args.call == "scan":
            binding.chunk_scan(Q, K, W, U, g, inp.C, scale=q_scale, cu_seqlens=inp.cu_seqlens, out=O, want_state=False, stream=stream)
        elif args.call == "layer":
            binding.fused(K, V, beta, g, inp.C, method=method | binding.W_DECAY, cu_seqlens=inp.cu_seqlens, out=(None, W, U), stream=stream)
            binding.chunk_scan(Q, K, W, U, g, inp.C, scale=q_scale, cu_seqlens=inp.cu_seqlens, out=O, want_state=False, stream=stream)
        elif args.call == "kda_fused":
            binding.fused_kda(K, V, G, beta, inp.C, method=method, cu_seqlens=inp.cu_seqlens, out=(A, W, U), stream=stream)
        elif args.call == "kda_scan":
            binding.chunk_scan_kda(Q, K, W, U, G, inp.C, scale=q_scale, cu_seqlens=inp.cu_seqlens, out=O, want_state=False, stream=stream)
        elif args.call == "kda_layer":
            binding.fused_kda(K, V, G, beta, inp.C, method=method, cu_seqlens=inp.cu_seqlens, out=(A, W, U), stream=stream)
            binding.chunk_scan_kda(Q, K, W, U, G, inp.C, scale=q_scale, cu_seqlens=inp.cu_seqlens, out=O, want_state=False, stream=stream)
        elif args.call == "kda":
            binding.build_kda(K, G, beta, inp.C, method=method, cu_seqlens=inp.cu_seqlens, out=A, stream=stream)
        else:
            binding.wy(A, K, V, beta, cu_seqlens=inp.cu_seqlens, out=(W, U), stream=stream)

    if args.call == "scan":  # the scan reads stored W (decay-weighted) and U: produce them once, outside the timed region
        binding.fused(K, V, beta, g, inp.C, method=method | binding.W_DECAY, cu_seqlens=inp.cu_seqlens, out=(None, W, U), stream=stream)
    if args.call == "kda_scan":
        binding.fused_kda(K, V, G, beta, inp.C, method=method, cu_seqlens=inp.cu_seqlens, out=(A, W, U), stream=stream)
    if args.call == "wy":  # tri_inv_wy reads a stored A: produce it once, outside the timed region
        binding.build(K, beta, g, inp.C, method=method, cu_seqlens=inp.cu_seqlens, out=A, stream=stream)

    for _ in range(max(args.warmup, 3)):
        flush_l2()
        step()
    torch.cuda.synchronize()
    if binding.last_device_status() != 0:
        raise SystemExit("device status word raised during warm-up")

    sampler = ClockSampler(local_rank)
    if rank == 0:
        # the timed region lasts milliseconds: keep the GPU busy with the same flush + step pattern until the
        # sampler has produced readings under load, then go straight into the timed steps
        sampler.start()
        t_end = time.time() + 5.0
        while sampler.proc and len(sampler.lines) < 4 and time.time() < t_end:
            for _ in range(20):
                flush_l2()
                step()
            torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = binding.launch_count()
    evs = []
    for _ in range(args.steps):
        flush_l2()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        step()
        e1.record(stream)
        evs.append((e0, e1))
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    launches = binding.launch_count() - launches0
    times_ms = [a.elapsed_time(b) for a, b in evs]
    total_ms = sum(times_ms)
    clocks = sampler.stop() if rank == 0 else None
    value, ms_per_step = aggregate_throughput(total_ms / args.steps, n_mat, world, "cuda")

    # ---- end to end through the public API with host buffers: H2D of the inputs, kernel, D2H of A, W, U
    hK, hV = binding.kv_to_torch(inp.K, "cpu", pin=True), binding.kv_to_torch(inp.V, "cpu", pin=True)
    hb, hg = torch.from_numpy(inp.beta).pin_memory(), torch.from_numpy(inp.g).pin_memory()
    hA = torch.empty(A.shape, dtype=A.dtype).pin_memory()
    hW, hU = torch.empty(W.shape, dtype=W.dtype).pin_memory(), torch.empty(U.shape, dtype=U.dtype).pin_memory()
    h2d = sum(x.numel() * x.element_size() for x in (hK, hV, hb, hg))
    d2h = sum(x.numel() * x.element_size() for x in (hA, hW, hU))

    pipe = None
    if args.call == "fused":   # the C-ABI call that takes host buffers: tri_inv_fused_host with a device workspace of the caller's
        pipe = torch.empty(binding.fused_host_workspace_bytes(inp.B, inp.T, inp.H, inp.d_k, inp.d_v, inp.C, binding._dtype_code(K),
                                                              inp.cu_seqlens), dtype=torch.uint8, device="cuda")

    def e2e_step():
        if pipe is not None:  # slices of the batch overlap upload, kernel and download inside the call
            binding.fused_host(hK, hV, hb, hg, inp.C, hA, hW, hU, pipe, method=method, cu_seqlens=inp.cu_seqlens, stream=stream)
            return
        K.copy_(hK, non_blocking=True); V.copy_(hV, non_blocking=True)
        beta.copy_(hb, non_blocking=True); g.copy_(hg, non_blocking=True)
        step()
        hA.copy_(A, non_blocking=True); hW.copy_(W, non_blocking=True); hU.copy_(U, non_blocking=True)

    e2e_steps = max(3, min(args.steps, 10))
    e2e_step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_value, _ = aggregate_throughput(e0.elapsed_time(e1) / e2e_steps, n_mat, world, "cuda")

    # ---- accuracy of what was just timed: the WHOLE batch against the fp64 oracle (slab by slab along the tokens of a
    # dense batch, to bound the host copies; a packed batch in one piece)
    err = None
    if rank == 0:
        import oracle
        slab = 4096
        pieces = [slice(None)] if inp.cu_seqlens is not None else [slice(t, min(t + slab, inp.T)) for t in range(0, inp.T, slab)]
        cu = inp.cu_seqlens
        num, den = {}, {}

        def acc(key, x, ref):
            num[key] = max(num.get(key, 0.0), float(np.abs(x - ref).max()))
            den[key] = max(den.get(key, 0.0), float(np.abs(ref).max()))

        Gs = G.cpu().numpy() if args.call in KDA_CALLS else None
        if args.call in ("kda_scan", "kda_layer"):
            O_ref, _ = oracle.recurrence_ex(Q_host, inp.K, inp.V, inp.beta, None, inp.C, G=Gs, scale=q_scale, cu_seqlens=cu)
            acc("O", binding.to_numpy_f64(O), O_ref)
        elif args.call in ("scan", "layer"):
            O_ref, _ = oracle.gdn_recurrence(Q_host, inp.K, inp.V, inp.beta, inp.g, inp.C, scale=q_scale, cu_seqlens=cu)
            acc("O", binding.to_numpy_f64(O), O_ref)
        else:
            for sl in pieces:
                Ko, bo, go = inp.K[:, sl], inp.beta[:, sl], inp.g[:, sl]
                if args.call == "raw":
                    Ko, bo, go = oracle.raw_front_end(Ko, bo, go, inp.C, cu_seqlens=cu)
                if args.call in ("kda", "kda_fused"):
                    A_ref = oracle.build_A_kda(inp.K[:, sl], Gs[:, sl], inp.beta[:, sl], inp.C, cu_seqlens=cu)
                    Ko = wl.bf16_bits_to_f32(Ko).astype(np.float64) * np.exp(Gs[:, sl].astype(np.float64)) if Ko.dtype == np.uint16 \
                        else Ko.astype(np.float64) * np.exp(Gs[:, sl].astype(np.float64))   # W = A diag(beta) (K * Gamma)
                else:
                    A_ref = oracle.build_A(Ko, bo, go, inp.C, cu_seqlens=cu)
                if args.call != "wy":
                    acc("A", binding.to_numpy_f64(A[:, sl]), A_ref)
                if args.call not in ("build", "kda"):
                    W_ref, _ = oracle.wy(A_ref, Ko, None, bo, inp.C, cu_seqlens=cu)
                    _, U_ref = oracle.wy(A_ref, inp.K[:, sl], inp.V[:, sl], bo, inp.C, cu_seqlens=cu)
                    acc("W", binding.to_numpy_f64(W[:, sl]), W_ref)
                    acc("U", binding.to_numpy_f64(U[:, sl]), U_ref)
        err = {"sample": "all tokens"}
        if args.call in SCAN_CALLS:
            err["reference"] = "token-by-token recurrence"
        for key in num:
            err[key + "_max_ratio"] = num[key] / den[key] if den[key] > 0 else num[key]

    if rank == 0:
        elt = 2 if inp.kv_dtype == wl.BF16 else 4
        alg_bytes = algorithmic_bytes_per_matrix(inp.C, inp.d_k, inp.d_v, elt, call=args.call)
        kernel_ms = statistics.mean(times_ms)               # one launch per step, timed alone by its event pair
        achieved = alg_bytes * n_mat / (kernel_ms * 1e-3) / 1e9
        peak, peak_kind = measured_peak_gbs()
        traffic = None if args.paper_T else ncu_traffic_bytes_per_matrix(args.call, args.config, args.method)
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": None if traffic is None else traffic * n_mat, "peak_source": "of " + peak_kind,
                    "kernel": {"fused": "fused build+invert+WY", "raw": "front end + build+invert+WY", "build": "build+invert", "kda": "per-channel-decay build+invert", "kda_fused": "per-channel-decay build+invert+WY (one kernel)" if inp.C == 64 else "per-channel-decay build+invert (+ scaled keys), then WY (2 launches)", "wy": "WY apply", "scan": "chunk scan (state recurrence + output)", "layer": "fused build+invert+WY, then chunk scan (2 launches)", "kda_scan": "per-channel-decay chunk scan: operand preparation, then the scan (2 launches)", "kda_layer": "per-channel-decay build+invert+WY, operand preparation, chunk scan (3 launches)"}[args.call], "kernel_ms": kernel_ms, "kernel_ms_min": min(times_ms),
                    "algorithmic_bytes_per_launch": alg_bytes * n_mat}
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu, _, _ = time_oracle(inp, target_seconds=15.0)
            one, _, _ = time_oracle(inp, target_seconds=5.0, n_threads=1)
            cpu["one_thread"] = {"value": one["value"], "cores": one["cores"], "sample": one["sample"]}
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
               "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
               "dtype": "bf16" if inp.kv_dtype == wl.BF16 else "f32", "data": "synthetic",
               "config": {"workload": inp.name, "B": inp.B, "T": inp.T, "H": inp.H, "d_k": inp.d_k, "d_v": inp.d_v, "C": inp.C,
                          "chunk_matrices_per_gpu": n_mat, "method": args.method, "call": args.call,
                          "outputs": OUTPUTS[args.call],
                          "l2": "flushed before every timed step (256 MiB write, then a 256 MiB read so no dirty lines remain)" if flush is not None else "not flushed",
                          "parallelism": "independent replicas, no collective" if world > 1 else "single GPU"},
               "gb_per_s": achieved, "roofline": roofline, "cpu_baseline": cpu,
               "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                       "api": "tri_inv_fused_host (C ABI: pinned host buffers in and out, device workspace of the caller's)" if pipe is not None else "copies + " + args.call},
               "gpu_launches": launches, "clocks": clocks, "error_vs_oracle": err}
        print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
