"""The N > 1 path is N independent replicas; its only communication is the
benchmark's bookkeeping.  Two gloo ranks on CPU check that bookkeeping."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    from paper_2604_13349_b200 import dist
    dist.init("gloo")
    r = int(os.environ["RANK"])
    assert dist.world_size() == 2
    dist.barrier()
    ms = dist.max_over_ranks(10.0 if r == 0 else 25.0)
    tot = dist.sum_over_ranks(100.0 + r)
    thr = dist.aggregate_throughput(1000.0 * (r + 1), 10.0 if r == 0 else 20.0)
    assert ms == 25.0 and tot == 201.0, (ms, tot)
    assert abs(thr - 3000.0 / 0.020) < 1e-6, thr
    dist.finish()
    print("rank", r, "ok")
""") % ROOT


def test_two_gloo_ranks_aggregate_like_the_benchmark():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", LOCAL_RANK=str(r),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for p in procs:
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert "ok" in out


def test_single_process_needs_no_process_group():
    from paper_2604_13349_b200 import dist
    assert dist.world_size() == 1
    dist.barrier()
    assert dist.max_over_ranks(3.5) == 3.5 and dist.sum_over_ranks(2.0) == 2.0
    assert dist.aggregate_throughput(10.0, 500.0) == 20.0
