"""The N > 1 path of bench.py on CPU: two gloo ranks launched the way the driver launches the GPU job."""
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


def _torchrun(script_args, timeout=600):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port())] + script_args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    out = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)
    assert out.returncode == 0, out.stderr[-2000:]
    return [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]


def test_whole_job_time_is_the_slowest_ranks_and_throughput_counts_every_rank():
    lines = _torchrun([os.path.join(ROOT, "tests", "multirank_worker.py")])
    assert len(lines) == 1                               # rank 0 alone prints
    assert lines[0]["world"] == 2
    assert lines[0]["ms_total"] == 20.0                  # MAX over the ranks' 10 ms and 20 ms
    assert abs(lines[0]["value"] - 1000 * 2 * 4 / 20e-3) < 1e-6


def test_reference_arm_under_two_ranks_prints_one_line_from_rank_zero():
    lines = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                       "--workload", "llama60m_mlp"])
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
