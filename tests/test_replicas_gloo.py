"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks, no GPU.

The scoring path shards into independent replicas, so the only multi-rank logic is: every rank
joins the group, a barrier brackets the timed region, the reported time is the MAX over ranks, the
whole-job rate counts every rank's units, and only rank 0 prints.
"""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_SCRIPT = r"""
import json, sys, time
sys.path.insert(0, {root!r})
from paper_2506_15733_b200.replicas import Replicas
r = Replicas.from_env()
r.init("gloo")
r.barrier()
elapsed = 0.25 if r.rank == 0 else 0.75          # rank 1 is the slow one
slowest = r.max_over_ranks(elapsed)
rate = r.whole_job_rate(1000.0, elapsed)
r.barrier()
if r.rank == 0:
    print(json.dumps({{"world": r.world, "slowest": slowest, "rate": rate}}))
r.shutdown()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _env(rank, world, port):
    env = dict(os.environ)
    env.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(port))
    return env


def test_two_gloo_ranks_report_the_slowest_time_once():
    port = _free_port()
    script = RANK_SCRIPT.format(root=ROOT)
    procs = [subprocess.Popen([sys.executable, "-c", script], env=_env(rank, 2, port), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for rank in range(2)]
    outs = [p.communicate(timeout=120) for p in procs]
    assert [p.returncode for p in procs] == [0, 0], outs
    assert outs[1][0].strip() == "", "only rank 0 prints"
    line = json.loads(outs[0][0].strip())
    assert line["world"] == 2
    assert line["slowest"] == 0.75                            # MAX over ranks, seen by rank 0
    assert abs(line["rate"] - 2 * 1000.0 / 0.75) < 1e-9      # both ranks' units over the slowest rank's time


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_2506_15733_b200.replicas import Replicas
    r = Replicas(0, 0, 1)
    r.init("gloo")
    r.barrier()
    assert r.backend is None and r.max_over_ranks(1.5) == 1.5 and r.whole_job_rate(10.0, 2.0) == 5.0
    r.shutdown()


def test_reference_arm_runs_on_rank_zero_only():
    # under a multi-rank launch the other ranks leave at once, without joining any group or printing
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         env=_env(1, 2, _free_port()), capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
