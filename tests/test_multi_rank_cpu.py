"""The N > 1 path of the benchmark on CPU: two gloo ranks.

The decode path has no exchange step ("replicas only"): every rank runs an independent copy of the
workload, timings are reduced with MAX over ranks and the whole-job value is N x per-rank bytes /
slowest time.  The reference arm under a multi-rank launch prints on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["REPO_ROOT"])
import torch.distributed as dist
import bench
rank, local, world = bench.dist_env()
dist.init_process_group("gloo", rank=rank, world_size=world)
mine = [10.0 + rank, 5.0 - rank, 7.0]                 # rank 0: [10, 5, 7]; rank 1: [11, 4, 7]
red = bench.max_over_ranks(mine, world)
val = bench.aggregate_throughput(2_000_000_000, red[0], world)
dist.barrier()
print(json.dumps({"rank": rank, "world": world, "reduced": red, "value": val}))
dist.destroy_process_group()
"""


def _launch(argv, extra_env=None, world=2):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), REPO_ROOT=ROOT)
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable] + argv, cwd=ROOT, env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=600)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_max_over_ranks_and_whole_job_value_with_two_gloo_ranks():
    outs = _launch(["-c", WORKER])
    res = [json.loads(o.strip().splitlines()[-1]) for o in outs]
    for r in res:
        assert r["world"] == 2
        assert r["reduced"] == [11.0, 5.0, 7.0]                      # slowest rank decides
        assert abs(r["value"] - 2 * 2.0 / 11.0e-3) < 1e-6            # 2 ranks x 2 GB per 11 ms, in GB/s
    assert sorted(r["rank"] for r in res) == [0, 1]


def test_reference_arm_prints_on_rank_zero_only():
    outs = _launch(["bench.py", "--impl", "reference", "--workload", "tiny", "--gpus", "2", "--steps", "1",
                    "--warmup", "0"])
    lines0 = [l for l in outs[0].splitlines() if l.strip()]
    lines1 = [l for l in outs[1].splitlines() if l.strip()]
    assert len(lines0) == 1 and lines1 == []
    rec = json.loads(lines0[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["config"]["workload"] == "tiny"
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["value"] > 0
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["e2e"]["d2h_bytes_per_step"] == 0
