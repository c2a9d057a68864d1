"""The N > 1 plumbing on CPU: two gloo ranks shard requests, meet at the barrier and agree on the
max-over-ranks time and the whole-job throughput."""
import os
import socket
import subprocess
import sys
import textwrap

from paper_2609_03494_b200 import shard

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_request_sharding_is_a_partition():
    for n, world in ((64, 2), (7, 3), (5, 8), (256, 8)):
        parts = [shard.shard_requests(n, r, world) for r in range(world)]
        assert sorted(sum(parts, [])) == list(range(n))
        assert max(map(len, parts)) - min(map(len, parts)) <= 1
    assert shard.shard_seed(1, 0) == 1 and len({shard.shard_seed(1, r) for r in range(8)}) == 8


def test_two_gloo_ranks_agree_on_job_throughput():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    code = textwrap.dedent("""
        import sys
        sys.path.insert(0, %r)
        from paper_2609_03494_b200 import shard
        rank, local, world = shard.init("gloo")
        assert world == 2
        mine = shard.shard_requests(7, rank, world)
        shard.barrier()
        value, ms = shard.job_throughput(len(mine) * 10, 100.0 + 50.0 * rank)
        assert ms == 150.0 and abs(value - 70 / 0.150) < 1e-9, (value, ms)
        assert shard.max_over_ranks(rank) == 1.0 and shard.sum_over_ranks(1.0) == 2.0
        shard.barrier()
        shard.finish()
        shard.finish()                     # idempotent
        print("rank", rank, "ok")
    """ % ROOT)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for p in procs:
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert "ok" in out
