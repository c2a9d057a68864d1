"""Asynchronous boundary work (App. "Asynchronous Decoding and Compression"): the boundary chain of a step runs
on the pool's own stream beside the next step, and the requests it concerns sit that step out.  The CUDA path is
compared with the oracle's reading of the same mode: step by step with every decision, working set and retained
set (the comparer's getters wait for the chain), and free-running, with nothing between the steps that waits
for the pool's stream, so that the overlap itself is what is tested."""
import numpy as np
import pytest

from oracle import growpage_oracle as O
from paper_2609_03494_b200 import binding as B
from paper_2609_03494_b200 import harness as H
from paper_2609_03494_b200 import workload as W
from tests import lockstep as LS

pytestmark = pytest.mark.gpu
NO_NEAR_TIES = {"ws": 0, "sel": 0, "act": 0}


def _report(name, st):
    print(f"\n[async {name}] steps {st.steps} tokens {st.tokens} attn max {st.attn_max_abs:.2e} decisions {st.decisions} "
          f"near-ties {st.near_ties} actions {st.actions}")


def test_tiny_every_step_with_held_requests():
    st = LS.run_lockstep(W.parity_instance(1), summary_every=1, check_pool_every=1, async_boundary=True)
    _report("tiny", st)
    assert st.tokens == 1024 and st.steps > 256                 # the same tokens in more steps: boundaries cost a step
    # every boundary but a request's last one (its final token) is followed by a step out
    assert st.actions.get(B.GP_ACT_PENDING, 0) == 64 and st.actions.get(B.GP_ACT_HELD, 0) == 60
    assert st.actions.get(B.GP_ACT_COMPRESS, 0) > 0 and st.near_ties == NO_NEAR_TIES


@pytest.mark.parametrize("config,over", [(1, dict(tau=-0.07)), (1, dict(tau=-1.0, n_pages=4 * 5 + 3)), (2, {}), (3, {}),
                                         (5, {}), (5, dict(policy=B.GP_POLICY_SHRINK, shrink_below=0.0, min_capacity=48))])
def test_configurations_with_grants_fallbacks_stalls_sharing_and_shrinks(config, over):
    st = LS.run_lockstep(W.parity_instance(config), async_boundary=True, **over)
    _report(f"config{config} {over}", st)
    assert st.decisions["act"] > 0
    if config == 5:
        assert st.counters[4] > 0                                # copy-on-write happened beside a running step


@pytest.mark.parametrize("slots", [8, 48, 148])
def test_free_running_steps_match_the_oracle(slots):
    """No getter and no device-wide wait between the steps: the chain of step t really runs beside step t + 1.
    Outputs and actions are compared every step (reading them waits for the caller's stream only), everything
    else at the end."""
    import torch
    wl = W.layer8b(n_requests=12, n_steps=150, prompt_range=(100, 400))
    s = wl.shape
    gpu, ora = LS.make_pools(wl, 0, async_boundary=True, async_slots=slots, tau=-0.002)
    sch = H.Scheduler(wl)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()
    try:
        while True:
            op = sch.next_admission()
            if op is None:
                break
            g = gpu.request_add(-1, 0, op.k_tail, op.v_tail, op.n_tail, op.initial_pages)
            o = ora.request_add(-1, 0, H.decode_bits(op.k_tail), H.decode_bits(op.v_tail), op.n_tail, op.initial_pages)
            assert g == (B.GP_OK, o[1])
            sch.admitted(op, g[1])
        seen = {}
        steps = 0
        while sch.resident and steps < 120:
            specs, rids, q, k, v = sch.batch()
            ids = torch.tensor(rids, dtype=torch.int32, device="cuda")
            out = torch.zeros((s.n_layers, len(rids), s.n_q_heads, s.head_dim), dtype=torch.float32, device="cuda")
            act = torch.zeros(len(rids), dtype=torch.int32, device="cuda")
            gpu.decode_step(ids, dev(q), dev(k), dev(v), out, act)
            rec = ora.decode_step(rids, H.decode_bits(q), H.decode_bits(k), H.decode_bits(v))
            g_act = act.cpu().numpy()                            # waits for the caller's stream, not for the pool's
            assert g_act.tolist() == rec.actions.tolist(), steps
            stepped = [i for i in range(len(rids)) if g_act[i] in (B.GP_ACT_NONE, B.GP_ACT_PENDING)]
            err = np.abs(out.cpu().numpy()[:, stepped] - rec.out[:, stepped])
            assert err.max() <= LS.ATTN_MAX_ABS
            for a in g_act.tolist():
                seen[a] = seen.get(a, 0) + 1
            sch.after_step(specs, g_act)
            steps += 1
        assert seen.get(B.GP_ACT_PENDING, 0) > 10 and seen.get(B.GP_ACT_HELD, 0) > 10
        # the end state: pages, counters, decisions, retained tokens and summaries of every request
        n_free, ref, counters = B.gp_debug_pool(gpu.handle, gpu.cfg.n_pages)
        assert counters[7] == 0 and n_free == ora.n_free()
        assert sorted(ref[ref > 0].tolist()) == sorted(ora.refcount[ora.refcount > 0].tolist())
        for name, gi in (("grow", 0), ("compress", 1), ("fallback", 2), ("stalled", 3), ("moved_rows", 8), ("scored_tokens", 9)):
            assert int(counters[gi]) == ora.counters[name], name
        assert counters[0] > 0 and counters[1] > 0               # both kinds of decision happened
        for res in sch.resident.values():
            rid = res.rid
            P, n, pos, _ = B.gp_debug_request(gpu.handle, rid, gpu.cfg.max_pages_per_req)
            assert (P, n, pos) == ora.request_state(rid)[:3]
            assert B.gp_boundary_outcome(gpu.handle, rid) == ora.boundary_outcome(rid)
            for h in range(s.n_kv_heads):
                assert np.array_equal(B.gp_debug_retained(gpu.handle, rid, 0, h, n), ora.retained(rid, 0, h)), (rid, h)
            gs = B.gp_debug_summaries(gpu.handle, rid, s.n_layers, s.n_q_heads, s.head_dim)
            os_ = ora.summaries(rid)
            rel = np.linalg.norm(gs - os_, axis=-1) / np.linalg.norm(os_, axis=-1)
            assert rel.max() <= LS.SUMMARY_REL
    finally:
        gpu.close()


def test_layer_entry_points_are_refused_and_admissions_wait_for_the_chain():
    import torch
    cfg = B.make_config(1, 8, 2, 64, n_pages=16, max_pages_per_req=4, max_requests=4, async_boundary=True)
    pool = B.Pool(cfg)
    try:
        rng = np.random.default_rng(1)
        bits = lambda *sh: W.f32_to_bf16_bits(rng.standard_normal(sh).astype(np.float32))
        assert pool.request_add(-1, 0, bits(1, 31, 2, 64), bits(1, 31, 2, 64), 31, 0) == (B.GP_OK, 0)
        ids = torch.zeros(1, dtype=torch.int32, device="cuda")
        act = torch.zeros(1, dtype=torch.int32, device="cuda")
        with pytest.raises(B.GpError) as e:
            B.gp_step_begin(pool.handle, ids.data_ptr(), 1, act.data_ptr(), pool.stream())
        assert e.value.status == B.GP_ERR_STATE
        out = torch.zeros((1, 1, 8, 64), dtype=torch.float32, device="cuda")
        dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda()
        pool.decode_step(ids, dev(bits(1, 1, 8, 64)), dev(bits(1, 1, 2, 64)), dev(bits(1, 1, 2, 64)), out, act)
        assert act.cpu().tolist() == [B.GP_ACT_PENDING]           # 32 tokens fill both pages
        # the release comes right behind the step: it must wait for the chain, which is compressing the request
        pool.release(0)
        B.gp_async_join(pool.handle, pool.stream())
        n_free, ref, counters = B.gp_debug_pool(pool.handle, 16)
        assert n_free == 16 and counters[7] == 0 and int(ref.sum()) == 0 and counters[1] == 1
    finally:
        pool.close()
