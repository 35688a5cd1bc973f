"""The replica plumbing under world_size 2 on CPU (gloo): barrier, slowest-rank time, summed units."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    from paper_2402_13720_b200 import dist_util
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    g = dist_util.init(world, rank, "gloo")
    dist_util.barrier(g)
    ms = 10.0 * (rank + 1)                       # rank 1 is the slow one
    assert dist_util.max_over_ranks(ms, g) == 20.0
    assert dist_util.sum_over_ranks(3.0, g) == 6.0
    rate = dist_util.aggregate_throughput(100.0, ms, g)
    assert abs(rate - 200.0 / 0.020) < 1e-6, rate
    dist_util.finish(g)
    print("ok", rank)
""") % ROOT


def test_two_replicas_gloo(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29641")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert "ok 0" in outs[0] and "ok 1" in outs[1]


def test_single_process_is_a_no_op():
    from paper_2402_13720_b200 import dist_util
    assert dist_util.init(1, 0, "gloo") is None
    dist_util.barrier(None)
    assert dist_util.max_over_ranks(5.0, None) == 5.0 and dist_util.aggregate_throughput(10.0, 1000.0, None) == 10.0
