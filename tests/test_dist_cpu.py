"""The multi-process path of the benchmark (replicas only: barrier, maximum over ranks of the device time, whole-job
value, one line from rank 0), run as two gloo ranks on the CPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_two_ranks_take_the_slowest_time_and_rank0_prints_one_line():
    port = 29500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.join(ROOT, "tests", "dist_worker.py")]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout
    out = json.loads(lines[0])
    assert out["rank"] == 0 and out["world"] == 2
    assert out["ms_max"] == 20.0                                   # the slower rank
    assert abs(out["value"] - 2 * 1000 * 4 / 20e-3) < 1e-6           # both ranks' tokens over the slowest time


def test_single_process_needs_no_process_group():
    from paper_2511_15927_b200 import dist_util as D
    env = {k: os.environ.pop(k, None) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    try:
        D.init("gloo")
        assert D.max_over_ranks(3.5) == 3.5
        assert D.whole_job_value(100, 2, 10.0) == 100 * 2 / 10e-3
        D.barrier()
    finally:
        for k, v in env.items():
            if v is not None:
                os.environ[k] = v
