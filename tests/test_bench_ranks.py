"""The N > 1 logic of bench.py on CPU: two gloo ranks.  The path does not shard (replicas only), so
what there is to check is the aggregation -- the slowest rank's time, units added over ranks -- and
that under a multi-rank launch only rank 0 of the reference arm works and prints."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["VS_ROOT"])
import torch, torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
t = torch.tensor([10.0 + rank, 5.0 - rank, 7.0], dtype=torch.float64)     # ms per phase, rank-dependent
bench.max_over_ranks(t, world)
fps = bench.replica_throughput(world, 64, t[0].item())
print(json.dumps({"rank": rank, "times": t.tolist(), "fps": fps}))
dist.barrier()
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(cmd, world, extra_env=None):
    port = _free_port()
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), VS_ROOT=ROOT, OMP_NUM_THREADS="2")
        env.update(extra_env or {})
        procs.append(subprocess.Popen(cmd, env=env, cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    return [(p.returncode, o, e) for p, (o, e) in zip(procs, outs)]


def test_max_over_ranks_and_replica_throughput_two_gloo_ranks():
    res = _launch([sys.executable, "-c", WORKER], 2)
    for rc, out, err in res:
        assert rc == 0, err[-2000:]
    rows = [json.loads(out.strip().splitlines()[-1]) for _, out, _ in res]
    for row in rows:
        assert row["times"] == [11.0, 5.0, 7.0]                  # element-wise maximum over the ranks
        assert abs(row["fps"] - 2 * 64 / 11.0e-3) < 1e-6         # both replicas' frames over the slower one's time


def test_reference_arm_prints_on_rank_zero_only():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--workload", "tiny"]
    res = _launch(cmd, 2)
    for rc, out, err in res:
        assert rc == 0, err[-2000:]
    lines0 = [l for l in res[0][1].splitlines() if l.strip()]
    assert len(lines0) == 1 and res[1][1].strip() == ""
    rec = json.loads(lines0[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"].startswith("oracle") and rec["e2e"]["h2d_bytes_per_step"] == 0
