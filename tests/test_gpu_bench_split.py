"""bench.py with the heads split over two ranks, run as two processes that share the one GPU of the test box
(control plane over gloo; the ranks' kernels never wait on one another, each rank just plans and attends its own
slice of the heads).  Checks the line rank 0 prints: strong scaling, all heads' work counted once."""
import json
import os
import socket
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _bench(nproc, extra):
    env = dict(os.environ, WAVEAL_DIST_BACKEND="gloo", WAVEAL_BENCH_ONE_DEVICE="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"),
           "--gpus", str(nproc), "--steps", "2", "--warmup", "3", "--no-e2e", "--no-cpu", "--ab-pairs", "2"] + extra
    out = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


def test_heads_split_over_two_ranks_counts_every_head_once():
    single = _bench(1, ["--config", "wan480p", "--heads", "6"])
    split = _bench(2, ["--config", "wan480p", "--heads", "6"])
    assert single["n_gpus"] == 1 and single["scaling"] == "weak" and single["config"]["heads_per_rank"] == 6
    assert split["n_gpus"] == 2 and split["scaling"] == "strong"
    assert split["config"]["heads"] == 6 and split["config"]["heads_per_rank"] == 3
    assert split["config"]["sharding"].startswith("heads split")
    # value = all heads' FLOPs / max-over-ranks time: the FLOPs behind it are those of the single run
    flops_single = single["value"] * single["ms_per_step"]
    flops_split = split["value"] * split["ms_per_step"]
    assert abs(flops_split / flops_single - 1) < 1e-6
    assert split["gpu_launches"] > 0 and split["cpu_baseline"] is None
    # replicas keep one full batch element per rank
    rep = _bench(2, ["--config", "wan480p", "--heads", "6", "--replicas"])
    assert rep["scaling"] == "weak" and rep["config"]["heads_per_rank"] == 6
    assert abs(rep["value"] * rep["ms_per_step"] / flops_single - 2) < 1e-6
