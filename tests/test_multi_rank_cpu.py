"""The N > 1 path of bench.py on CPU: world size 2 over gloo (replicas, max-over-ranks timing)."""
import json
import os
import signal
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(script_args, nproc=2, timeout=180):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + script_args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    # own session, so that a hung run can be ended as a whole (launcher and workers) by its process group id
    proc = subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, cwd=ROOT, env=env,
                            start_new_session=True)
    try:
        out, err = proc.communicate(timeout=timeout)
    except subprocess.TimeoutExpired:
        os.killpg(proc.pid, signal.SIGKILL)
        out, err = proc.communicate()
        return subprocess.CompletedProcess(cmd, -9, out, "timed out after %d s\n" % timeout + err)
    return subprocess.CompletedProcess(cmd, proc.returncode, out, err)


def test_max_over_ranks_and_whole_job_value(tmp_path):
    res = _torchrun([os.path.join(ROOT, "tests", "gloo_worker.py"), str(tmp_path)])
    assert res.returncode == 0, res.stderr[-2000:]
    outs = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(2)]
    for o in outs:
        assert o["world"] == 2
        assert o["slowest_ms"] == 15.0                      # max over ranks, not the mean, not rank 0's
        assert abs(o["value"] - 2 * 3.0e12 / 15e-3 / 1e12) < 1e-9  # both replicas' work in the slowest time


def test_reference_arm_under_torchrun_prints_one_line_from_rank_0():
    res = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                     "--warmup", "0", "--workload", "tiny"])
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["unit"] == "TFLOP/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
