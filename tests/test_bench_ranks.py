"""The bench's multi-rank path on CPU: two gloo ranks, max-over-ranks timing, whole-job value."""
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


def test_two_ranks_take_the_slowest_rank_and_sum_the_replicas(tmp_path):
    out = tmp_path / "rank0.json"
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.join(ROOT, "tests", "dist_worker.py"), str(out)]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    got = json.loads(out.read_text())
    assert got["world"] == 2
    assert got["worst"] == [12.5, 30.0]                     # element-wise maximum over the ranks
    assert abs(got["value"] - 2 * 61 / 12.5e-3) < 1e-6      # two replicas, time of the slower one
    assert got["seeds"][0] != got["seeds"][1]               # replicas decode different requests


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.slowest_rank([3.0, 4.0], 1, "cpu") == [3.0, 4.0]
    assert bench.job_value(1, 4, 61, 10.0) == 4 * 61 / 10e-3
