"""Two gloo ranks on the CPU: the multi-rank bookkeeping of bench.py (replicas, no data-path collective):
max-over-ranks step time, whole-job throughput = N x per-rank pixels / slowest time, distinct per-rank batches."""
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


def test_two_ranks_gloo(tmp_path):
    env = dict(os.environ, ESC_TEST_OUT=str(tmp_path), OMP_NUM_THREADS="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.join(ROOT, "tests", "_dist_worker.py")]
    r = subprocess.run(cmd, env=env, cwd=ROOT, capture_output=True, text=True, timeout=240)
    assert r.returncode == 0, r.stderr[-2000:]
    res = [json.load(open(tmp_path / f"rank{k}.json")) for k in range(2)]
    assert [x["world"] for x in res] == [2, 2]
    assert res[0]["worst_ms"] == res[1]["worst_ms"] == 3.0          # the slowest rank sets the step time
    expect = 2 * 4096 / 3.0e-3 / 1e6
    assert abs(res[0]["value"] - expect) < 1e-9 and res[0]["value"] == res[1]["value"]
    assert res[0]["x0"] != res[1]["x0"]                              # every rank draws its own batch


def test_reference_arm_other_ranks_exit_quietly():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, cwd=ROOT, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
