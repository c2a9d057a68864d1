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


def test_kv_head_slices_are_whole_groups_and_a_partition():
    for hq, hkv, world in ((32, 8, 8), (32, 8, 2), (64, 8, 4), (8, 2, 2), (4, 4, 1)):
        g = hq // hkv
        qs = [shard.kv_head_slice(hq, hkv, r, world) for r in range(world)]
        assert sorted(sum((list(range(q.start, q.stop)) for q, _ in qs), [])) == list(range(hq))
        assert sorted(sum((list(range(k.start, k.stop)) for _, k in qs), [])) == list(range(hkv))
        for q, k in qs:
            assert q.start == k.start * g and q.stop == k.stop * g          # a KV head travels with its query heads
    import pytest
    with pytest.raises(ValueError):
        shard.kv_head_slice(32, 8, 0, 3)


def test_two_gloo_ranks_complete_the_mean_of_eq8_from_their_heads():
    # Every rank scores its own KV heads (the oracle's per-unit working sets, on seeded synthetic summaries and
    # keys), adds its K^S and K^L up, the ranks all-reduce the two integers per request, and Delta from the completed
    # sums equals the oracle's mean over ALL (layer, head) units, on both ranks.
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    code = textwrap.dedent("""
        import sys
        sys.path.insert(0, %r)
        import numpy as np, torch
        from oracle import growpage_oracle as O
        from paper_2609_03494_b200 import shard
        rank, local, world = shard.init("gloo")
        L, HQ, HKV, D, N, R = 3, 8, 4, 16, 48, 5
        G = HQ // HKV
        rng = np.random.default_rng(17)                    # the same numbers on both ranks
        keys = rng.standard_normal((R, L, HKV, N, D))
        qs_short = rng.standard_normal((R, L, HQ, D))
        qs_long = rng.standard_normal((R, L, HQ, D))
        qs_short[0::2] *= 3.0                              # sharper short view: concentrating, Delta < 0
        qs_long[1::2] *= 3.0                               # sharper long view: widening, Delta > 0
        def unit(r, l, h):
            ks = [O.p_coverage_demand(O.summary_attention(q[r, l, h * G:(h + 1) * G], keys[r, l, h]), 0.9)
                  for q in (qs_short, qs_long)]
            return ks
        full = np.array([[[unit(r, l, h) for h in range(HKV)] for l in range(L)] for r in range(R)])     # [R][L][H][2]
        want = (full[..., 0].sum(axis=(1, 2)) - full[..., 1].sum(axis=(1, 2))) / (L * HKV * N)
        _, kv = shard.kv_head_slice(HQ, HKV, rank, world)
        mine = full[:, :, kv]
        sums = torch.zeros((8, 2), dtype=torch.int32)      # the array has max_requests rows; rows past the step's stay zero
        sums[:R, 0] = torch.from_numpy(mine[..., 0].sum(axis=(1, 2)).astype(np.int32))
        sums[:R, 1] = torch.from_numpy(mine[..., 1].sum(axis=(1, 2)).astype(np.int32))
        shard.complete_boundary_sums(sums)
        got = (sums[:R, 0].numpy().astype(np.int64) - sums[:R, 1].numpy()) / (L * HKV * N)
        assert np.array_equal(got, want), (got, want)
        assert int(sums[R:].abs().sum()) == 0
        assert len(set(np.sign(want))) > 1                 # both signs occur: grow and compress decisions
        shard.finish()
        print("rank", rank, "ok")
    """ % ROOT)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for p in procs:
        out, _ = p.communicate(timeout=180)
        assert p.returncode == 0, out
        assert "ok" in out
