"""The N > 1 plumbing (barrier, max over ranks, whole-job throughput) on two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    from paper_2510_08522_b200 import dist_util as DU
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    DU.init(world, "gloo")
    DU.barrier()
    local_ms = 10.0 * (rank + 1)                     # rank 1 is the slow one
    assert DU.max_over_ranks(local_ms) == 20.0
    assert abs(DU.job_throughput(5.0, local_ms) - 2 * 5.0 / 0.020) < 1e-9
    DU.finish()
    print("rank", rank, "ok")
""" % ROOT)


def test_two_gloo_ranks():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", LOCAL_RANK=str(r), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT))
    for r, p in enumerate(procs):
        out, _ = p.communicate(timeout=240)
        assert p.returncode == 0, out.decode()
        assert ("rank %d ok" % r) in out.decode()


def test_single_rank_is_a_no_op():
    from paper_2510_08522_b200 import dist_util as DU
    DU.init(1)
    DU.barrier()
    assert DU.max_over_ranks(3.5) == 3.5 and DU.job_throughput(7.0, 1000.0) == 7.0
    DU.finish()
