"""Host side of the multi-GPU bench path, exercised with two gloo ranks on CPU: the weak-scaling
aggregation (sum of per-rank work over the slowest rank's time) and the reference arm's rule that
only rank 0 works and prints."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_ranks(script, world=2, port=29611):
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), PYTHONPATH=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", script], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True, cwd=ROOT))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
    return [o for o, _ in outs]


def test_weak_scaling_aggregation_over_gloo():
    script = textwrap.dedent("""
        import os, json
        import torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        local_ms = 2.0 if rank == 0 else 5.0          # rank 1 is the slow one
        value, ms = bench.aggregate_throughput(local_ms, 4096, world)
        print(json.dumps({"rank": rank, "value": value, "ms": ms, "mx": bench.reduce_max(float(rank))}))
        dist.barrier(); dist.destroy_process_group()
    """)
    outs = [json.loads(o.strip().splitlines()[-1]) for o in run_ranks(script)]
    for o in outs:
        assert o["ms"] == 5.0 and o["mx"] == 1.0
        assert abs(o["value"] - 2 * 4096 / 5e-3) < 1e-6


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    value, ms = bench.aggregate_throughput(0.5, 100, 1)
    assert ms == 0.5 and value == 100 / 0.5e-3


def test_reference_arm_runs_on_rank0_only():
    outs = []
    for rank in (0, 1):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), PYTHONPATH=ROOT)
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                            "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                           timeout=300, cwd=ROOT)
        assert r.returncode == 0, r.stderr
        outs.append(r.stdout.strip())
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["unit"] == "chunk-matrices/s"
    assert outs[1] == ""
