"""N > 1 runs are independent replicas; their bookkeeping (per-rank seeds, barrier, max of the
times, sum of the tokens, one printing rank) is exercised here with two gloo ranks on the CPU."""
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


def _torchrun(args, timeout=240):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port())] + args
    env = dict(os.environ, OMP_NUM_THREADS="1")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_gloo_ranks_aggregate_as_replicas(tmp_path):
    p = _torchrun([os.path.join(ROOT, "tests", "replica_worker.py"), str(tmp_path)])
    assert p.returncode == 0, p.stderr[-2000:]
    r = [json.load(open(tmp_path / f"rank{k}.json")) for k in range(2)]
    assert [x["rank"] for x in r] == [0, 1] and all(x["world"] == 2 for x in r)
    assert r[0]["is_root"] and not r[1]["is_root"]
    assert r[0]["seed"] != r[1]["seed"]  # each replica has its own batch
    for x in r:  # every rank sees the job totals: 16 + 17 tokens, the slower rank's 2 ms
        assert x["tokens"] == 33 and x["ms"] == 2.0


def test_reference_arm_prints_one_line_from_rank_zero():
    p = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup",
                   "0", "--workload", "c1_tiny"])
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
