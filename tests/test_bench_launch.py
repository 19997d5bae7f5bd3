"""bench.py starts its own ranks when it is given --gpus N outside a torchrun environment (CPU, gloo)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _clean_env():
    env = dict(os.environ)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    return env


def test_plain_python_launch_starts_n_ranks():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rank-check"],
                       capture_output=True, text=True, timeout=300, env=_clean_env(), cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout                      # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2
    assert lines[0]["slowest_ms"] == 2.0                  # the max over ranks of rank + 1
    assert lines[0]["value"] == 2 * 1000.0 / 2.0e-3       # whole-job rate: both ranks' units over the slowest time


def test_single_rank_needs_no_launcher():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "1", "--rank-check"],
                       capture_output=True, text=True, timeout=300, env=_clean_env(), cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][0])
    assert line["n_gpus"] == 1 and line["slowest_ms"] == 1.0


def test_both_arms_name_the_workload_with_the_same_keys():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2209_10778_b200 import workloads as W
    w = W.WORKLOADS["gelu_ffn_100m"]
    c = bench._config(w, w.numel(0))
    assert c["workload"] == "gelu_ffn_100m" and c["elements"] == 64 * 512 * 3072 >= 64 * 2**20
    assert c["shape"] == [64, 512, 3072] and c["kinds"] == ["gelu_erf", "gelu_tanh"]
