"""The multi-rank plumbing of the benchmark, run as two gloo ranks on CPU: barrier,
max-over-ranks of the time, whole-job rate, and 'only rank 0 reports'."""
import json
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys, time
    sys.path.insert(0, {root!r})
    from paper_2209_10778_b200 import ranks
    w = ranks.world_from_env()
    ranks.init(w, "gloo")
    ranks.barrier(w, cuda=False)
    my_ms = 10.0 + 5.0 * w.rank                      # rank 1 is the slow one
    slowest = ranks.max_over_ranks(w, my_ms)
    rate = ranks.whole_job_rate(w, units_per_rank_per_step=1000.0, steps=4, ms_slowest=slowest)
    ranks.barrier(w, cuda=False)
    if w.is_main:
        print(json.dumps({{"slowest": slowest, "rate": rate, "size": w.size}}))
    ranks.finish(w)
""")


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert outs[1][0].strip() == ""                  # rank 1 prints nothing
    line = json.loads(outs[0][0].strip())
    assert line["size"] == 2
    assert line["slowest"] == 15.0                   # the maximum over ranks, seen by rank 0
    assert line["rate"] == 2 * 1000.0 * 4 / 0.015    # both ranks' units in the slowest rank's time


def test_single_rank_is_a_no_op():
    from paper_2209_10778_b200 import ranks
    w = ranks.World(0, 0, 1)
    ranks.init(w, "gloo")
    ranks.barrier(w, cuda=False)
    assert ranks.max_over_ranks(w, 3.5) == 3.5
    assert ranks.whole_job_rate(w, 10.0, 2, 1.0) == 20000.0
    ranks.finish(w)


def test_reference_arm_runs_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
