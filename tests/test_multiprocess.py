"""The multi-GPU arm of the benchmark is N independent replicas (the path has no exchange step): what the ranks share
is the timing protocol.  Two CPU processes over gloo check it: the reported time is the maximum over the ranks, and
the reference arm prints one line from rank 0 while the other ranks leave without work."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
vals = bench.max_over_ranks([1.0 + rank, 5.0 - rank], "cpu")
dist.barrier()
open(os.path.join(%r, "rank%%d.json" %% rank), "w").write(json.dumps(dict(rank=rank, vals=vals)))
dist.destroy_process_group()
"""


def _torchrun(args, script_args, timeout=600):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port())] + args + script_args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_time_is_the_maximum_over_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % (ROOT, str(tmp_path)))
    r = _torchrun([str(script)], [])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads((tmp_path / ("rank%d.json" % k)).read_text()) for k in range(2)]
    assert sorted(l["rank"] for l in lines) == [0, 1]
    for l in lines:
        assert l["vals"] == [2.0, 5.0]


def test_reference_arm_prints_one_line_from_rank_zero():
    r = _torchrun([os.path.join(ROOT, "bench.py")], ["--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--config", "1"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
