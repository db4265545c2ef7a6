"""Host logic of the multi-GPU bench path on CPU: two gloo ranks.  The module
shards over independent images (replicas, no data-path collective), so what
needs checking is the bookkeeping: distinct per-rank inputs, max-over-ranks
timing, whole-job throughput, and that only rank 0 of the reference arm works."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, os.environ["MSLA_ROOT"])
import numpy as np
import torch.distributed as dist
import bench
from paper_2205_14756_b200 import inputs
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
base = inputs.ModuleShape("t", "bf16", 1, 16, 4, 4, 1, 16, seed=7)
s = bench.rank_shape(base, rank)
x = inputs.module_inputs(s)["x"]
ms = bench.max_over_ranks([10.0 + 5.0 * rank, 3.0 - rank])
val = bench.whole_job_value(s.B * s.N, world, ms[0], steps=4)
with open(os.path.join(os.environ["MSLA_OUT"], f"rank{rank}.json"), "w") as f:
    json.dump({"rank": rank, "seed": s.seed, "x0": float(x.ravel()[0]), "ms": ms, "value": val}, f)
dist.barrier()
dist.destroy_process_group()
"""


def _torchrun(args, env_extra=None, nproc=2):
    env = dict(os.environ, MSLA_ROOT=ROOT, MSLA_SKIP_AUTOBUILD="1", OMP_NUM_THREADS="1")
    env.update(env_extra or {})
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", "29731"] + args
    return subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300, cwd=ROOT)


def test_two_ranks_take_the_max_and_sum_the_tokens(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    r = _torchrun([str(script)], {"MSLA_OUT": str(tmp_path)})
    assert r.returncode == 0, r.stderr[-2000:]
    recs = [json.load(open(tmp_path / f"rank{i}.json")) for i in range(2)]
    assert sorted(x["rank"] for x in recs) == [0, 1]
    by = {x["rank"]: x for x in recs}
    assert by[0]["seed"] != by[1]["seed"] and by[0]["x0"] != by[1]["x0"]      # each rank has its own image
    for x in recs:
        assert x["ms"] == [15.0, 3.0]                                          # slowest rank per entry
        assert abs(x["value"] - 16 * 2 / (15.0e-3 / 4)) < 1e-6                 # all ranks' tokens / slowest time


def test_reference_arm_runs_on_rank0_only():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                   "--workload", "cfg1_module_f32_16x16"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["e2e"]["h2d_bytes_per_step"] == 0
