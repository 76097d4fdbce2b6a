"""The multi-GPU path of this build is "replicas only": every rank runs the same workload on its own
rows, and the one collective is the max-over-ranks of the step time behind the whole-job rate.  These
tests run that aggregation with world_size 2 on CPU (gloo), and check that the reference arm prints on
rank 0 only."""
import json
import os
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
ms_local = 0.2 if rank == 0 else 0.5          # the slower rank sets the job's step time
ms_max, tflops = bench.aggregate_replicas(ms_local, 10**12, world, device="cpu")
with open(os.path.join(%r, "rank%%d.json" %% rank), "w") as f:     # one file per rank: stdout of ranks can interleave
    json.dump({"rank": rank, "ms_max": ms_max, "tflops": tflops}, f)
dist.destroy_process_group()
"""


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(args, env_extra=None):
    env = dict(os.environ, **(env_extra or {}))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + args
    return subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=str(ROOT))


def test_replica_aggregation_takes_the_max_over_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % (str(ROOT), str(tmp_path)))
    out = _torchrun([str(script)])
    assert out.returncode == 0, out.stderr[-2000:]
    recs = [json.loads((tmp_path / f"rank{r}.json").read_text()) for r in (0, 1)]
    assert sorted(r["rank"] for r in recs) == [0, 1]
    for r in recs:
        assert r["ms_max"] == 0.5
        assert abs(r["tflops"] - 2 * 1e12 / 0.5e-3 / 1e12) < 1e-9      # two replicas, slower rank's time


def test_reference_arm_prints_once_under_torchrun():
    out = _torchrun([str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"])
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert lines[0]["impl"] == "reference" and lines[0]["cpu_baseline"]["kind"] == "oracle"
    assert lines[0]["e2e"]["h2d_bytes_per_step"] == 0 and lines[0]["value"] > 0
