"""`python bench.py --gpus N` must start N ranks by itself (CPU only: the ranks use the gloo backend and a stub
step; what is under test is the launch, the barrier and the max / sum over ranks that the real bench uses)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run(args, env=None):
    e = dict(os.environ)
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        e.pop(k, None)
    e.update(env or {})
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, capture_output=True, text=True,
                         timeout=300, env=e, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout               # rank 0 alone prints
    return json.loads(lines[0])


def test_gpus_2_starts_two_ranks_and_reduces_over_them():
    import bench
    d = run(["--gpus", "2", "--dist-selftest"])
    assert d["n_gpus"] == 2 and d["scaling"] == "weak"
    assert abs(d["ms_per_step"] - 2.0) < 1e-9         # the slower rank (2 ms) sets the step time
    assert abs(d["value"] - 2 * bench.step_bytes() / 2e-3 / 1e9) < 1e-6 * d["value"]


def test_gpus_1_runs_in_process():
    d = run(["--gpus", "1", "--dist-selftest"])
    assert d["n_gpus"] == 1 and abs(d["ms_per_step"] - 1.0) < 1e-9


def test_under_an_external_launcher_no_second_launch():
    # the driver's own launch line: ranks already exist, bench.py must not start more
    import bench
    port = bench.free_port()
    e = dict(os.environ)
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK"):
        e.pop(k, None)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"),
                          "--gpus", "2", "--dist-selftest"], capture_output=True, text=True, timeout=300, env=e, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1 and json.loads(lines[0])["n_gpus"] == 2
