"""The benchmark's multi-process plumbing on CPU (gloo, two ranks): barrier, max over ranks, request rotation."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    from paper_2601_04426_b200 import dist_util, inputs
    assert dist_util.init_from_env("gloo")
    rank = int(os.environ["RANK"])
    dist_util.barrier()
    got = dist_util.max_over_ranks(10.0 + rank)
    assert got == 11.0, got
    w = inputs.make_workload("C3", batch=8, steps=4, vocab_size=1024)
    r = dist_util.rotate_requests(w, rank)
    assert sorted(r.request_grammar) == sorted(w.request_grammar)
    assert (r.request_grammar == w.request_grammar) == (rank == 0)
    assert all(r.trajectories[i] == w.trajectories[(i + rank * 7) %% 8] for i in range(8))
    dist_util.finish()
    print("rank", rank, "ok")
""") % ROOT


def test_two_ranks_gloo():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD], env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    for p in procs:
        out, _ = p.communicate(timeout=240)
        assert p.returncode == 0, out
        assert "ok" in out


def test_single_process_is_a_no_op():
    from paper_2601_04426_b200 import dist_util
    assert dist_util.max_over_ranks(3.5) == 3.5
    dist_util.barrier()
