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


def test_gpus_flag_without_a_launcher_starts_that_many_ranks(monkeypatch):
    """`python bench.py --gpus 4` with no WORLD_SIZE in the environment re-launches itself under
    torch.distributed.run with four ranks on 127.0.0.1 and its own arguments."""
    sys.path.insert(0, ROOT)
    import bench
    seen = {}
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: seen.setdefault("cmd", cmd) and 0)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "7"])
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    bench.main()
    cmd = seen["cmd"]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "7"] and cmd[-5].endswith("bench.py")
    assert abs(bench.setup_flops(dict(d_model=4, n_heads=1, n_kv_heads=1, head_dim=4, d_ff=8, vocab=10, n_layers=1,
                                      n_visual=1, n_prompt=1)) - (2 * (48 + 16 + 96) * 2 + 2 * 2 * 4 * 3 + 2 * 40)) < 1e-9
