"""The N > 1 path of bench.py on CPU: two gloo ranks (the path has no data-path collective;
each rank evaluates its own replica, the job's time is the max over ranks)."""
import json
import socket
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(script_args, timeout=300):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), *script_args]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=timeout, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    return [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]


def test_max_over_ranks_and_whole_job_value_world2():
    lines = _torchrun([str(ROOT / "tests" / "_multi_rank_worker.py")])
    assert len(lines) == 1
    out = lines[0]
    assert out["world"] == 2
    assert out["slowest"] == 15.0                       # rank 1 is the slower one
    assert abs(out["value"] - 2 * 24 * 7 / 15e-3) < 1e-6


def test_reference_arm_under_torchrun_prints_one_line_from_rank0():
    lines = _torchrun([str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                       "--warmup", "0", "--workload", "tiny"])
    assert len(lines) == 1
    ref = lines[0]
    assert ref["impl"] == "reference" and ref["n_gpus"] == 2
    assert ref["cpu_baseline"]["kind"] == "oracle" and ref["cpu_baseline"]["value"] == ref["value"]
    assert ref["e2e"] == {"value": ref["value"], "unit": ref["unit"], "h2d_bytes_per_step": 0,
                          "d2h_bytes_per_step": 0}


def test_single_rank_helpers():
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.whole_job_value(1, 24, 10, 0.5) == 480.0
