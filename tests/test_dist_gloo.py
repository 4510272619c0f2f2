"""World-size-2 gloo run on CPU of the multi-process plumbing the benchmark uses
at N > 1: the problem split is a partition, and the reported time is the max."""
import os
import socket
import subprocess
import sys
import textwrap
from pathlib import Path

from paper_2604_21335_b200 import dist as D

ROOT = Path(__file__).resolve().parent.parent


def test_shard_range_is_a_balanced_partition():
    for n in (0, 1, 7, 32, 1024):
        for world in (1, 2, 3, 8):
            parts = [D.shard_range(n, r, world) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == n
            assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in parts]
            assert max(sizes) - min(sizes) <= 1
    got = sum((D.shard_problems(3, 4, r, 2) for r in range(2)), [])
    assert got == [(b, h) for b in range(3) for h in range(4)]


WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    from paper_2604_21335_b200 import dist as D
    r = D.init_from_env("gloo")
    assert r.world == 2
    D.barrier(r)
    t = D.max_over_ranks(r, 1.5 if r.rank == 0 else 4.25)
    s = D.sum_over_ranks(r, float(len(D.shard_problems(5, 3, r.rank, r.world))))
    D.barrier(r)
    if r.is_main:
        print("RESULT", t, s)
    D.shutdown(r)
""")


def test_two_rank_gloo_max_and_sum():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER % str(ROOT)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=240)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert "RESULT 4.25 15.0" in outs[0]
