"""N > 1 path of the benchmark on CPU: two gloo ranks on 127.0.0.1.

The step itself has no exchange between GPUs (N GPUs run N independent optimizer
replicas), so what N > 1 adds is the process-group set-up, the barrier, the
max-over-ranks timing and the rule that only rank 0 prints."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def torchrun(script_args, nproc=2, timeout=240):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
           f"--nproc-per-node={nproc}", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port())] + script_args
    env = dict(os.environ, OMP_NUM_THREADS="2", CUDA_VISIBLE_DEVICES="")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def json_lines(text):
    """Every JSON object in the output (two ranks may print on one line)."""
    out, dec, i = [], json.JSONDecoder(), 0
    while True:
        i = text.find("{", i)
        if i < 0:
            return out
        try:
            obj, end = dec.raw_decode(text, i)
            out.append(obj)
            i = end
        except json.JSONDecodeError:
            i += 1


def test_two_gloo_ranks_barrier_and_max_over_ranks():
    r = torchrun([os.path.join("tests", "dist_worker.py")])
    assert r.returncode == 0, r.stderr[-2000:]
    rows = sorted(json_lines(r.stdout), key=lambda x: x["rank"])
    assert [x["rank"] for x in rows] == [0, 1]
    assert all(x["world"] == 2 for x in rows)
    assert all(x["slowest"] == 20.0 for x in rows)  # the slower rank's time, on both
    assert rows[0]["g0"] != rows[1]["g0"]           # replicas draw different streams


def test_sharded_step_orchestration_over_two_gloo_ranks():
    """The coordinate-sharded step's host logic (phase order, which buffers are summed, who
    gets the gradient and the update) with all-reduces over gloo: two ranks, each holding a
    numpy stand-in of one shard that follows the library's phase protocol, must together
    reproduce the unsharded oracle - state bit for bit, ties at the threshold split across
    the boundary included."""
    r = torchrun([os.path.join("tests", "shard_worker.py")])
    assert r.returncode == 0, r.stderr[-2000:]
    rows = sorted(json_lines(r.stdout), key=lambda x: x["rank"])
    assert [x["rank"] for x in rows] == [0, 1]
    assert all(x["order_ok"] for x in rows)
    assert rows[0]["state_ok"]
    assert rows[0]["worst_u"] <= 1e-6


def test_reference_arm_prints_once_under_two_ranks():
    r = torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "2",
                  "--warmup", "1", "--workload", "c1_d65536_m32"])
    assert r.returncode == 0, r.stderr[-2000:]
    rows = json_lines(r.stdout)
    assert len(rows) == 1
    line = rows[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["metric"] == "efcp_steps_per_sec" and line["unit"] == "steps/s"
    assert line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
