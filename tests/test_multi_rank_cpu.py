"""The N > 1 plumbing of the benchmark on CPU (gloo, two ranks): ranks are independent replicas, so
what there is to check is that every rank draws its own inputs, that the reported time is the
slowest rank's and the value the whole job's, and that the reference arm prints one line from rank 0."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
from paper_2602_02199_b200 import synth
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
layers = bench.rank_layers(rank, 2)
w = synth.workload("tiny")
digest = [int(synth.q_window(w, l, 0).astype("int64").sum()) for l in layers]
ms = [10.0 + 5.0 * rank, 3.0 - rank]            # rank 1 is slower on the first, rank 0 on the second
got = bench.max_over_ranks(ms, world, torch.device("cpu"))
gathered = [None] * world
dist.all_gather_object(gathered, (layers, digest))
if rank == 0:
    print(json.dumps({{"max": got, "ranks": gathered, "value": bench.whole_job_value(100.0, 4, world, got[0])}}))
dist.destroy_process_group()
"""


def _torchrun(args, timeout=600):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(29500 + os.getpid() % 2000)] + args
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_gloo_ranks_draw_disjoint_layers_and_report_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT))
    r = _torchrun([str(script)])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["max"] == [15.0, 3.0]
    (l0, d0), (l1, d1) = out["ranks"]
    assert l0 == [0, 1] and l1 == [2, 3]                    # disjoint seeds
    assert len({*d0, *d1}) == 4                            # and the inputs they produce differ
    assert np.isclose(out["value"], 2 * 100.0 * 4 / 15e-3)  # whole job, slowest rank's clock


def test_reference_arm_under_torchrun_prints_one_line_from_rank_zero():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "tiny"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
