"""The N > 1 path of the benchmark on CPU: two gloo ranks, barrier, max-over-ranks timing,
whole-job aggregation; and the reference arm's rule that only rank 0 works and prints."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
from paper_1804_01526_b200 import replicas
rep = replicas.init(backend="gloo")
replicas.barrier(rep)
mine = 1.0 + rep.rank            # rank 1 is slower
worst = replicas.max_over_ranks(rep, mine)
agg = replicas.aggregate_throughput(rep, 100.0, worst)
replicas.barrier(rep)
with open(os.path.join({out!r}, "rank%d.json" % rep.rank), "w") as f:   # one file per rank: stdout lines of two ranks can interleave
    json.dump(dict(rank=rep.rank, world=rep.world, worst=worst, agg=agg, root=rep.is_root), f)
replicas.shutdown(rep)
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _torchrun(args, nproc=2, timeout=180):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, out=str(tmp_path)))
    r = _torchrun([str(script)])
    assert r.returncode == 0, r.stderr[-2000:]
    rows = [json.loads((tmp_path / f"rank{i}.json").read_text()) for i in range(2)]
    assert sorted(x["rank"] for x in rows) == [0, 1]
    for x in rows:
        assert x["world"] == 2 and x["worst"] == 2.0 and x["agg"] == 2 * 100.0 / 2.0
    assert [x["root"] for x in sorted(rows, key=lambda x: x["rank"])] == [True, False]


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_1804_01526_b200 import replicas
    env = {k: os.environ.pop(k) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK") if k in os.environ}
    try:
        rep = replicas.init()
        assert rep.world == 1 and rep.is_root and replicas.max_over_ranks(rep, 3.5) == 3.5
        replicas.barrier(rep)
        replicas.shutdown(rep)
    finally:
        os.environ.update(env)


def test_reference_arm_under_torchrun_only_rank0_prints():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--size", "256"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["n_gpus"] == 2
