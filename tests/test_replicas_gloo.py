"""The N > 1 path on CPU: two gloo ranks run independent replicas; only the barrier and the
max-over-ranks of the time cross ranks. Also the reference arm under a two-rank launch:
rank 0 alone works and prints, the other rank exits 0."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torchrun(script_args, port):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + script_args
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="1")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)


def _json_lines(text):
    """Every JSON object in the text (two ranks may write to the same line)."""
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


def test_two_gloo_ranks_run_independent_replicas():
    res = _torchrun([os.path.join("tests", "_replica_worker.py")], 29533)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = sorted(_json_lines(res.stdout), key=lambda d: d["rank"])
    assert [d["rank"] for d in lines] == [0, 1] and all(d["world"] == 2 for d in lines)
    assert all(d["slow"] == 2.0 for d in lines)                       # max over ranks of (1, 2)
    assert all(abs(d["rate"] - 2 * 64 / 2.0) < 1e-9 for d in lines)   # all ranks' units / slowest time
    assert lines[0]["idx_head"] != lines[1]["idx_head"]               # each replica draws its own routing


def test_reference_arm_under_two_ranks_prints_once():
    res = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "1",
                     "--workload", "C1"], 29534)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = _json_lines(res.stdout)
    assert len(lines) == 1
    d = lines[0]
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
