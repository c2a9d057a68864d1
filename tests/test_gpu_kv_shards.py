"""The decode step with the model's KV heads spread over several pools (gp_decode_step_local / gp_decode_step_finish).

Two pools on one GPU stand for the two ranks of a tensor-parallel group: each holds one of the two KV heads (and its
four query heads) of every request, runs the local half of the step on its heads, the test adds the two arrays of
sums up (what the all-reduce does between ranks; the pools' kernels never wait for one another), and each pool
finishes the step.  The oracle holds all heads in one pool.  Compared every step: both pools take the oracle's
action, each pool's attention output equals the oracle's for its heads; at every boundary: K^S and K^L of each
pool's units equal the oracle's for those heads, Delta equals the oracle's (a mean over ALL units), the retained
token sets are the oracle's; at the end: pages, slots, position, page tables and free list of both pools equal the
oracle's."""
import numpy as np
import pytest

from oracle import growpage_oracle as O
from paper_2609_03494_b200 import binding as B
from paper_2609_03494_b200 import harness as H
from paper_2609_03494_b200 import shard
from paper_2609_03494_b200 import workload as W

from tests.lockstep import ATTN_MAX_ABS

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("tau,n_pages", [(-0.05, 40), (-1.0, 17)])
def test_two_head_shards_decide_as_one_pool(tau, n_pages):
    import torch
    L, HQ, HKV, D, b, cap, T = 2, 8, 2, 64, 16, 6, 150
    shape = W.Shape(L, HQ, HKV, D)
    prompts = (40, 21, 75)
    reqs = [W.RequestSpec(i, p, T, 0.05) for i, p in enumerate(prompts)]
    wl = W.Workload("shards", 5, shape, reqs, n_resident=3, initial_pages=0, max_pages_per_req=cap, n_pages=n_pages, k_loc=4)
    world = 2
    ocfg = O.OracleConfig(L, HQ, HKV, D, n_pages=n_pages, max_pages_per_req=cap, max_requests=4, k_loc=4, tau=tau)
    ora = O.OraclePool(ocfg)
    pools, slices = [], []
    try:
        for r in range(world):
            qs, ks = shard.kv_head_slice(HQ, HKV, r, world)
            slices.append((qs, ks))
            cfg = B.make_config(L, HQ // world, HKV // world, D, n_pages=n_pages, max_pages_per_req=cap, max_requests=4, k_loc=4,
                                tau=tau, kv_shard_count=world)
            pools.append(B.Pool(cfg, 0))
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to("cuda:0")
        streams = [wl.stream(s) for s in reqs]
        q_all = np.empty((T, L, 3, HQ, D), dtype=np.uint16)
        k_all = np.empty((T, L, 3, HKV, D), dtype=np.uint16)
        v_all = np.empty_like(k_all)
        for i, st in enumerate(streams):
            kp, vp = st.prompt_kv()
            assert ora.request_add(-1, 0, H.decode_bits(kp), H.decode_bits(vp), prompts[i], 0) == (O.OK, i)
            for (qs, ks), pool in zip(slices, pools):
                assert pool.request_add(-1, 0, dev(kp[:, :, ks]), dev(vp[:, :, ks]), prompts[i], 0) == (B.GP_OK, i)
            q_all[:, :, i], k_all[:, :, i], v_all[:, :, i] = st.steps(0, T)
        ids = torch.arange(3, dtype=torch.int32, device="cuda:0")
        q_dev = [dev(q_all[:, :, :, qs]) for qs, _ in slices]          # every pool's slice of every step's inputs
        k_dev = [dev(k_all[:, :, :, ks]) for _, ks in slices]
        v_dev = [dev(v_all[:, :, :, ks]) for _, ks in slices]
        outs = [torch.zeros((L, 3, HQ // world, D), dtype=torch.float32, device="cuda:0") for _ in range(world)]
        acts = [torch.zeros(3, dtype=torch.int32, device="cuda:0") for _ in range(world)]
        sums = [shard.shard_sums_tensor(p) for p in pools]
        seen = set()
        n_boundaries = 0
        for t in range(T):
            # the local halves, the sum over the "ranks", the second halves
            for r, pool in enumerate(pools):
                B.gp_decode_step_local(pool.handle, ids.data_ptr(), 3, q_dev[r][t].data_ptr(), k_dev[r][t].data_ptr(),
                                       v_dev[r][t].data_ptr(), outs[r].data_ptr(), acts[r].data_ptr(), pool.stream())
            with pytest.raises(B.GpError):           # between the halves the pool takes nothing else
                pools[0].release(0)
            total = sums[0] + sums[1]
            for s_ in sums:
                s_.copy_(total)
            for pool, act in zip(pools, acts):
                B.gp_decode_step_finish(pool.handle, ids.data_ptr(), 3, act.data_ptr(), pool.stream())
            torch.cuda.synchronize()
            rec = ora.step_compute([0, 1, 2], H.decode_bits(q_all[t]), H.decode_bits(k_all[t]), H.decode_bits(v_all[t]))
            for orid, info in rec.boundary.items():
                n_boundaries += 1
                for r, ((qs, ks), pool) in enumerate(zip(slices, pools)):
                    g_ks, g_kl, g_delta = B.gp_debug_boundary(pool.handle, orid, L, HKV // world)
                    assert np.array_equal(g_ks, info.K_s[:, ks]) and np.array_equal(g_kl, info.K_l[:, ks]), (t, orid, r)
                    assert g_delta == info.delta, (t, orid, r, g_delta, info.delta)
            ora.step_apply(rec, {})
            for r, ((qs, ks), pool) in enumerate(zip(slices, pools)):
                a = acts[r].cpu().numpy()
                assert np.array_equal(a, np.asarray(rec.actions)), (t, r, a, rec.actions)
                seen |= set(int(x) for x in a)
                stepped = a >= 0
                err = np.abs(outs[r].cpu().numpy().astype(np.float64) - rec.out[:, :, qs])[:, stepped]
                assert err.size == 0 or err.max() <= ATTN_MAX_ABS, (t, r, float(err.max()))
                if rec.boundary:
                    for orid in rec.boundary:
                        P, n, pos, _ = B.gp_debug_request(pool.handle, orid, cap)
                        oP, on, opos, _ = ora.request_state(orid)
                        assert (P, n, pos) == (oP, on, opos), (t, r, orid)
                        for l in range(L):
                            for hl, h in enumerate(range(ks.start, ks.stop)):
                                got = B.gp_debug_retained(pool.handle, orid, l, hl, n)
                                assert np.array_equal(got, ora.requests[orid].tok[l, h, :n]), (t, r, orid, l, h)
        assert n_boundaries > 10 and B.GP_ACT_GROW in seen
        assert (B.GP_ACT_COMPRESS in seen) or (B.GP_ACT_COMPRESS_FALLBACK in seen)      # compactions on both pools
        o_free = ora.n_free() if hasattr(ora, "n_free") else None
        for pool in pools:
            n_free, ref, counters = B.gp_debug_pool(pool.handle, n_pages)
            assert counters[7] == 0
            if o_free is not None:
                assert n_free == o_free
            for i in range(3):
                P, n, pos, table = B.gp_debug_request(pool.handle, i, cap)
                oP, on, opos, otable = ora.request_state(i)
                assert (P, n, pos) == (oP, on, opos) and list(table[:P]) == list(otable[:oP])
    finally:
        for p in pools:
            p.close()
