"""The N > 1 path of bench.py without GPUs: ranks are independent replicas, so what there is
to check is the plumbing - rendezvous, barrier, max-over-ranks timing, the whole-job value -
and that the reference arm prints one line from rank 0 only.  gloo backend, world size 2."""

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


def _torchrun(script_and_args, timeout):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + script_and_args
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="4")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def _json_lines(text):
    """Every JSON object in the output (two ranks may write to the same line)."""
    dec, out, i = json.JSONDecoder(), [], 0
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


def test_rank_plumbing_world_size_2():
    res = _torchrun([os.path.join("tests", "_dist_worker.py")], timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = sorted(_json_lines(res.stdout), key=lambda d: d["rank"])
    assert [d["rank"] for d in lines] == [0, 1] and all(d["world"] == 2 for d in lines)
    # both ranks agree on the slowest rank's time, and the value is the whole job's
    assert all(d["ms"] == 12.5 for d in lines)
    assert all(abs(d["tokens_per_s"] - 2 * 8192 / 12.5e-3) < 1e-6 for d in lines)


def test_reference_arm_prints_once_from_rank_0():
    res = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                    timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = _json_lines(res.stdout)
    assert len(lines) == 1
    d = lines[0]
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
