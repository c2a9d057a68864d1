"""GPU parity: the CUDA path against the float64 oracle on the same seeded inputs, through the C ABI."""
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
    print(f"\n[{name}] steps {st.steps} tokens {st.tokens} attn max {st.attn_max_abs:.2e} mean {st.attn_mean_abs:.2e} "
          f"summary rel {st.summary_max_rel:.1e} decisions {st.decisions} near-ties {st.near_ties} actions {st.actions}")


def test_config1_tiny_every_step():
    st = LS.run_lockstep(W.parity_instance(1), summary_every=1, check_pool_every=1)
    _report("tiny", st)
    assert st.steps == 256 and st.tokens == 1024
    assert st.actions.get(B.GP_ACT_COMPRESS, 0) > 0
    assert st.near_ties == NO_NEAR_TIES


@pytest.mark.parametrize("config", [2, 3, 4, 5])
def test_configs_2_to_5_reduced(config):
    st = LS.run_lockstep(W.parity_instance(config))
    _report(f"config{config}", st)
    assert st.decisions["sel"] > 0
    assert st.near_ties == NO_NEAR_TIES       # the standard configurations need no excuse: every decision is the oracle's
    if config == 5:
        assert st.counters[4] > 0            # copy-on-write happened


def test_tiny_with_negative_threshold_mixes_grow_fallback_and_compress():
    st = LS.run_lockstep(W.parity_instance(1), tau=-0.07)
    _report("tiny tau=-0.07", st)
    assert st.actions.get(B.GP_ACT_GROW, 0) > 0 and st.actions.get(B.GP_ACT_COMPRESS, 0) > 0
    st = LS.run_lockstep(W.parity_instance(1), tau=-1.0)            # always wants to grow: cap 16 forces fallback
    _report("tiny tau=-1", st)
    assert st.actions.get(B.GP_ACT_COMPRESS_FALLBACK, 0) > 0 and st.actions.get(B.GP_ACT_COMPRESS, 0) == 0


def test_tiny_with_rope():
    st = LS.run_lockstep(W.parity_instance(1), rope_theta=1e6, tau=-0.05)
    _report("tiny rope", st)


def test_tiny_under_pool_pressure_falls_back_and_stalls():
    wl = W.parity_instance(1)
    st = LS.run_lockstep(wl, tau=-1.0, n_pages=4 * 5 + 3)           # three spare pages for four growers
    _report("tiny small pool", st)
    assert st.actions.get(B.GP_ACT_GROW, 0) == 3 and st.actions.get(B.GP_ACT_COMPRESS_FALLBACK, 0) > 0


def test_other_quota_and_coverage_settings():
    st = LS.run_lockstep(W.parity_instance(1), k_loc=0, top_p=0.9, beta_s=0.5, beta_l=0.95, max_steps=120)
    _report("tiny k_loc=0", st)
    st = LS.run_lockstep(W.parity_instance(1), k_loc=16, tau=-0.02, max_steps=120)
    _report("tiny k_loc=16", st)


def _single_request_case(shape, n_prompt, n_steps, seed=11, **over):
    wl = W.Workload("adhoc", seed, shape, [W.RequestSpec(0, n_prompt, n_steps, 0.05)], n_resident=1, initial_pages=0,
                    max_pages_per_req=n_prompt // 16 + 4, n_pages=n_prompt // 16 + 8)
    return LS.run_lockstep(wl, **(over or dict(tau=-1.0)))


@pytest.mark.parametrize("hq,hkv,d,n_prompt", [(32, 8, 128, 1530), (64, 8, 128, 777), (4, 4, 64, 1100),
                                               (2, 1, 64, 15), (8, 8, 128, 1), (16, 2, 128, 260)])
def test_long_sequences_span_chunks_and_ragged_tails(hq, hkv, d, n_prompt):
    st = _single_request_case(W.Shape(2, hq, hkv, d), n_prompt, 40)
    _report(f"long {hq}/{hkv}/{d} n={n_prompt}", st)


def test_batch_edge_cases_and_host_entry_point():
    import torch
    shape = W.Shape(1, 8, 2, 64)
    cfg = B.make_config(1, 8, 2, 64, n_pages=32, max_pages_per_req=4, max_requests=8, host_staging=True)
    pool = B.Pool(cfg)
    try:
        rng = np.random.default_rng(0)
        kt = W.f32_to_bf16_bits(rng.standard_normal((1, 20, 2, 64)).astype(np.float32))
        vt = W.f32_to_bf16_bits(rng.standard_normal((1, 20, 2, 64)).astype(np.float32))
        st, a = pool.request_add(-1, 0, kt, vt, 20, 0)
        assert (st, a) == (B.GP_OK, 0)
        st, b_ = pool.request_add(-1, 0, kt, vt, 20, 0)
        assert (st, b_) == (B.GP_OK, 1)
        assert pool.request_add(5, 1, None, None, 0, 0)[0] == B.GP_ERR_INVALID      # donor not live
        assert pool.request_add(a, 2, None, None, 0, 0)[0] == B.GP_ERR_INVALID      # only one full prompt page
        assert pool.request_add(-1, 0, kt, vt, 20, 9)[0] == B.GP_ERR_NO_PAGES       # above the per-request cap
        # empty batch is a no-op
        B.gp_decode_step(pool.handle, 0, 0, 0, 0, 0, 0, 0, pool.stream())
        # invalid, duplicate and dead ids are flagged per request; the valid ones still run
        ids = torch.tensor([a, 7, a, b_, -1], dtype=torch.int32)
        q = W.f32_to_bf16_bits(rng.standard_normal((1, 5, 8, 64)).astype(np.float32))
        k = W.f32_to_bf16_bits(rng.standard_normal((1, 5, 2, 64)).astype(np.float32))
        v = W.f32_to_bf16_bits(rng.standard_normal((1, 5, 2, 64)).astype(np.float32))
        out = torch.zeros((1, 5, 8, 64), dtype=torch.float32).pin_memory()
        act = torch.zeros(5, dtype=torch.int32).pin_memory()
        tq, tk, tv = (torch.from_numpy(x.view(np.int16)).pin_memory() for x in (q, k, v))
        pool.decode_step_host(ids.pin_memory(), tq, tk, tv, out, act)
        assert act.tolist() == [B.GP_ACT_NONE, B.GP_ACT_INVALID, B.GP_ACT_INVALID, B.GP_ACT_NONE, B.GP_ACT_INVALID]
        # the host entry point gives what the oracle gives
        f = W.bf16_bits_to_f64
        for col, rid in ((0, a), (3, b_)):
            K = np.concatenate([f(kt)[0].transpose(1, 0, 2), f(k)[0, col][:, None, :]], axis=1)
            V = np.concatenate([f(vt)[0].transpose(1, 0, 2), f(v)[0, col][:, None, :]], axis=1)
            want = O.attention_decode(f(q)[0, col], K, V)
            assert np.abs(out[0, col].numpy() - want).max() <= 1e-2
            P, n, pos, _ = B.gp_debug_request(pool.handle, rid, 4)
            assert (P, n, pos) == (2, 21, 21)
        pool.release(a)
        with pytest.raises(B.GpError):
            pool.release(a)
        n_free, ref, counters = B.gp_debug_pool(pool.handle, 32)
        assert n_free == 30 and counters[7] == 0
        assert B.gp_launch_count(pool.handle) > 0
    finally:
        pool.close()


def test_batch_larger_than_the_scratch_bound_is_reported_per_request():
    """Twelve requests reach their capacity boundary in the same step, with max_batch_tokens far below their
    summed lengths: the scoring scratch takes the candidates of two of them per step.  Each step two requests
    take their boundary; the others report GP_ACT_SCRATCH with their state unchanged and are stepped again in
    the next batch, until all are through.  Every stepped request's output is its softmax-weighted mean of
    values, and no error bit is raised."""
    import torch
    L, Hq, Hkv, d, b = 1, 8, 2, 64, 16
    n_req, P0 = 12, 24
    n0 = P0 * b - 1
    cfg = B.make_config(L, Hq, Hkv, d, n_pages=n_req * (P0 + 2), max_pages_per_req=P0 + 2, max_requests=n_req,
                        max_batch_tokens=1024)
    pool = B.Pool(cfg)
    try:
        rng = np.random.default_rng(3)
        bits = lambda *shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
        kp, vp = bits(n_req, L, n0, Hkv, d), bits(n_req, L, n0, Hkv, d)
        for i in range(n_req):
            assert pool.request_add(-1, 0, kp[i], vp[i], n0, P0) == (B.GP_OK, i)
        q, k, v = bits(L, n_req, Hq, d), bits(L, n_req, Hkv, d), bits(L, n_req, Hkv, d)
        dev = lambda x: torch.from_numpy(x.view(np.int16)).to("cuda:0")
        ids = torch.arange(n_req, dtype=torch.int32, device="cuda:0")
        out = torch.zeros((L, n_req, Hq, d), dtype=torch.float32, device="cuda:0")
        act = torch.zeros(n_req, dtype=torch.int32, device="cuda:0")
        f = W.bf16_bits_to_f64
        steps_done = np.zeros(n_req, dtype=np.int64)
        for step in range(6):
            before = [B.gp_debug_request(pool.handle, i, cfg.max_pages_per_req)[:3] for i in range(n_req)]
            pool.decode_step(ids, dev(q), dev(k), dev(v), out, act)
            a = act.cpu().numpy()
            o = out.cpu().numpy().astype(np.float64)
            waiting = [i for i in range(n_req) if steps_done[i] == 0]
            for i in range(n_req):
                after = B.gp_debug_request(pool.handle, i, cfg.max_pages_per_req)[:3]
                if steps_done[i] == 0 and i in waiting[:2]:           # the first two still at their boundary fit
                    assert a[i] in (B.GP_ACT_GROW, B.GP_ACT_COMPRESS), (step, i, a[i])
                    assert after[2] == n0 + 1 and after[:2] in ((P0 + 1, n0 + 1), (P0, (P0 - 1) * b))
                    K = np.concatenate([f(kp[i])[0].transpose(1, 0, 2), f(k)[0, i][:, None, :]], axis=1)   # [Hkv][n][d]
                    V = np.concatenate([f(vp[i])[0].transpose(1, 0, 2), f(v)[0, i][:, None, :]], axis=1)
                    assert np.abs(o[0, i] - O.attention_decode(f(q)[0, i], K, V)).max() <= 1e-2, f"request {i}"
                    steps_done[i] = 1
                elif steps_done[i] == 0:
                    assert a[i] == B.GP_ACT_SCRATCH and after == before[i], (step, i, a[i])
                else:
                    assert a[i] == B.GP_ACT_NONE and after[2] == before[i][2] + 1
        assert steps_done.all()
        assert B.gp_debug_pool(pool.handle, 0)[2][7] == 0
    finally:
        pool.close()


def test_synchronised_boundaries_put_several_boundary_items_on_every_cta():
    # equal prompt lengths: every request reaches its capacity boundary in the same step, so the attention
    # kernel's CTAs each get several boundary work items in a row (their calibrated summaries share one buffer
    # per CTA) and the selection kernel has more jobs than CTAs
    shape = W.Shape(2, 16, 8, 64)
    reqs = [W.RequestSpec(i, 180, 40, 0.02 + 0.004 * i) for i in range(40)]
    wl = W.Workload("sync-boundaries", 21, shape, reqs, n_resident=40, initial_pages=0, max_pages_per_req=16,
                    n_pages=40 * 16)
    st = LS.run_lockstep(wl, tau=-0.07)
    _report("synchronised boundaries", st)
    assert st.actions.get(B.GP_ACT_COMPRESS, 0) + st.actions.get(B.GP_ACT_COMPRESS_FALLBACK, 0) > 0


@pytest.mark.parametrize("shrink", [False, True])
def test_equal_scores_take_the_general_selection_paths(shrink):
    # zero queries: summaries and calibrated summaries are zero, every candidate gets the same probability, so
    # the single-histogram fast paths find one crowded bin and hand over to the general radix descent; ties are
    # broken by slot order on both sides (Eq. 7 by count, Eq. 10 keeps the older slots).  Once with Compress &
    # Hold, once with the Shrink policy set so that Delta_t = 0 shrinks (two pages worth go).
    import torch
    L, Hq, Hkv, d, n_prompt, steps = 1, 4, 2, 64, 100, 70
    kw = dict(n_pages=16, max_pages_per_req=9, max_requests=4, k_loc=2)
    pol = dict(policy=B.GP_POLICY_SHRINK, shrink_below=0.5, min_capacity=48) if shrink else {}
    n_ev = 32 if shrink else 16
    gpu = B.Pool(B.make_config(L, Hq, Hkv, d, tau=1.0, **kw, **pol))
    ora = O.OraclePool(O.OracleConfig(L, Hq, Hkv, d, tau=1.0, **kw, **pol))
    try:
        rng = np.random.default_rng(5)
        bits = lambda *shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
        kp, vp = bits(L, n_prompt, Hkv, d), bits(L, n_prompt, Hkv, d)
        assert gpu.request_add(-1, 0, kp, vp, n_prompt, 0) == (B.GP_OK, 0)
        assert ora.request_add(-1, 0, H.decode_bits(kp), H.decode_bits(vp), n_prompt, 0) == (O.OK, 0)
        ids = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        out = torch.zeros((L, 1, Hq, d), dtype=torch.float32, device="cuda:0")
        act = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        n_compress = 0
        for t in range(steps):
            q = np.zeros((L, 1, Hq, d), dtype=np.uint16)
            k, v = bits(L, 1, Hkv, d), bits(L, 1, Hkv, d)
            dev = lambda a: torch.from_numpy(a.view(np.int16)).to("cuda:0")
            gpu.decode_step(ids, dev(q), dev(k), dev(v), out, act)
            rec = ora.step_compute([0], H.decode_bits(q), H.decode_bits(k), H.decode_bits(v))
            assert np.abs(out.cpu().numpy() - rec.out).max() <= LS.ATTN_MAX_ABS
            for rid, info in rec.boundary.items():
                ks, kl, delta = B.gp_debug_boundary(gpu.handle, 0, L, Hkv)
                assert np.array_equal(ks, info.K_s) and np.array_equal(kl, info.K_l) and delta == info.delta
                if int(act.cpu()[0]) in (B.GP_ACT_COMPRESS, B.GP_ACT_COMPRESS_FALLBACK, B.GP_ACT_SHRINK):
                    assert (int(act.cpu()[0]) == B.GP_ACT_SHRINK) == (shrink and info.n_c >= 48)
                    n_compress += 1
                    r = ora.requests[0]
                    K_t = info.n_c - (n_ev if int(act.cpu()[0]) == B.GP_ACT_SHRINK else 16)
                    for l in range(L):
                        for h in range(Hkv):
                            keep, _ = O.select_retained(O.token_scores(info.a_s[l, h], info.a_l[l, h]), r.P - 1, 16, K_t, 2)
                            got = B.gp_debug_retained(gpu.handle, 0, l, h, K_t + 16)
                            assert np.array_equal(got[:K_t], r.tok[l, h, keep]), f"step {t} ({l},{h}): retained set differs"
            ora.step_apply(rec, {})
            assert int(act.cpu()[0]) == int(rec.actions[0]), f"step {t}"
        assert n_compress >= 3
        assert B.gp_debug_pool(gpu.handle)[2][7] == 0
    finally:
        gpu.close()


def test_candidate_set_larger_than_the_staging_buffers():
    # more than 6144 candidate tokens: the scores of a unit no longer fit the selection kernel's shared memory
    # and go through global scratch
    st = _single_request_case(W.Shape(1, 4, 2, 64), 6300, 80)
    _report("6300-token prompt", st)
    assert st.actions.get(B.GP_ACT_COMPRESS_FALLBACK, 0) >= 1
    # more (page, column) pairs than the table of softmax factors holds (6528): with 8 heads per group, 13200
    # tokens are 825 candidate pages x 8 columns for a working-set job and x 16 for an eviction job, and the
    # factors are recomputed per token
    st = _single_request_case(W.Shape(1, 16, 2, 64), 13200, 80)
    _report("13200-token prompt, G = 8", st)
    assert st.actions.get(B.GP_ACT_COMPRESS_FALLBACK, 0) >= 1
    st = _single_request_case(W.Shape(1, 16, 2, 64), 13200, 40, policy=B.GP_POLICY_SHRINK, shrink_below=0.5, tau=1.0)
    _report("13200-token prompt, G = 8, shrink", st)
    assert st.actions.get(B.GP_ACT_SHRINK, 0) >= 1


def test_shrink_at_the_default_floor_and_beyond_the_staging_buffers():
    # every admissible boundary shrinks (shrink_below above any Delta_t).  With the default minimum capacity of
    # 1024 tokens a 1530-token request shrinks; a 6300-token one takes the Shrink's eviction list through the
    # global score scratch
    always = dict(policy=B.GP_POLICY_SHRINK, shrink_below=0.5, tau=1.0)
    st = _single_request_case(W.Shape(2, 32, 8, 128), 1530, 40, **always)
    _report("1530-token prompt, shrink", st)
    assert st.actions.get(B.GP_ACT_SHRINK, 0) >= 2 and st.actions.get(B.GP_ACT_COMPRESS, 0) == 0
    st = _single_request_case(W.Shape(1, 4, 2, 64), 1030, 40, **always)       # 65 pages: one Shrink, then the floor
    _report("1030-token prompt, shrink", st)
    assert st.actions.get(B.GP_ACT_SHRINK, 0) == 1 and st.actions.get(B.GP_ACT_COMPRESS, 0) >= 1
    st = _single_request_case(W.Shape(1, 4, 2, 64), 6300, 50, **always)
    _report("6300-token prompt, shrink", st)
    assert st.actions.get(B.GP_ACT_SHRINK, 0) >= 2


def test_decode_steps_replayed_from_a_cuda_graph_match_direct_launches():
    # gp_decode_step only enqueues kernels (chained with programmatic dependent launch) and keeps the step's number
    # on the device: a sequence of steps, or one step over fixed buffers replayed once per token as a serving loop
    # does, can come from a CUDA graph; either must leave exactly the state and outputs of direct launches
    import torch
    wl = W.parity_instance(2)
    s = wl.shape
    n, T = 6, 24
    cfg = dict(n_pages=wl.n_pages, max_pages_per_req=wl.max_pages_per_req, max_requests=8, k_loc=wl.k_loc)
    q = np.empty((T, s.n_layers, n, s.n_q_heads, s.head_dim), dtype=np.uint16)
    k = np.empty((T, s.n_layers, n, s.n_kv_heads, s.head_dim), dtype=np.uint16)
    v = np.empty_like(k)
    prompts = []
    for i in range(n):
        st = wl.stream(wl.requests[i])
        prompts.append(st.prompt_kv())
        q[:, :, i], k[:, :, i], v[:, :, i] = st.steps(0, T)
    dev = lambda a: torch.from_numpy(a.view(np.int16)).to("cuda:0")
    qd, kd, vd = dev(q), dev(k), dev(v)
    ids = torch.arange(n, dtype=torch.int32, device="cuda:0")
    results = []
    for mode in ("direct", "sequence", "one_step"):
        pool = B.Pool(B.make_config(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, tau=-0.05, **cfg))
        try:
            for i in range(n):
                assert pool.request_add(-1, 0, prompts[i][0], prompts[i][1], wl.requests[i].prompt_len, 0)[0] == B.GP_OK
            outs = torch.zeros((T, s.n_layers, n, s.n_q_heads, s.head_dim), dtype=torch.float32, device="cuda:0")
            acts = torch.zeros((T, n), dtype=torch.int32, device="cuda:0")
            torch.cuda.synchronize()
            if mode == "sequence":             # all T steps in one graph, replayed once
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    for t in range(T):
                        pool.decode_step(ids, qd[t], kd[t], vd[t], outs[t], acts[t])
                g.replay()
            elif mode == "one_step":           # a serving loop: ONE captured step over fixed buffers, replayed per token
                qs, ks, vs = torch.empty_like(qd[0]), torch.empty_like(kd[0]), torch.empty_like(vd[0])
                o1, a1 = torch.zeros_like(outs[0]), torch.zeros_like(acts[0])
                g = torch.cuda.CUDAGraph()
                st = torch.cuda.Stream()
                with torch.cuda.stream(st):
                    for t in range(T):
                        qs.copy_(qd[t]); ks.copy_(kd[t]); vs.copy_(vd[t])
                        if t == 0:
                            with torch.cuda.graph(g, stream=st):
                                pool.decode_step(ids, qs, ks, vs, o1, a1)
                        g.replay()
                        outs[t].copy_(o1); acts[t].copy_(a1)
                st.synchronize()
            else:
                for t in range(T):
                    pool.decode_step(ids, qd[t], kd[t], vd[t], outs[t], acts[t])
            torch.cuda.synchronize()
            state = [B.gp_debug_request(pool.handle, i, cfg["max_pages_per_req"])[:3] for i in range(n)]
            kept = [B.gp_debug_retained(pool.handle, i, 0, 0, state[i][1]) for i in range(n)]
            assert B.gp_debug_pool(pool.handle)[2][7] == 0
            results.append((outs.cpu().numpy(), acts.cpu().numpy(), state, kept))
        finally:
            pool.close()
    for replay in results[1:]:
        direct = results[0]
        assert np.array_equal(direct[1], replay[1]) and direct[2] == replay[2]
        assert all(np.array_equal(a, b_) for a, b_ in zip(direct[3], replay[3]))
        assert np.array_equal(direct[0], replay[0])
    assert (results[0][1] != B.GP_ACT_NONE).any()


@pytest.mark.parametrize("over", [dict(policy=B.GP_POLICY_INVERSE), dict(policy=B.GP_POLICY_INVERSE, tau=-0.05),
                                  dict(policy=B.GP_POLICY_RANDOM, policy_seed=7),
                                  dict(policy=B.GP_POLICY_RANDOM, policy_seed=11, p_compress=0.3)])
def test_inverse_and_random_capacity_control_policies(over):
    # the controls of the paper's policy ablation: the reversed reading of Delta and a coin with P(compress) = p
    st = LS.run_lockstep(W.parity_instance(1), **over)
    _report(f"tiny {over}", st)
    grows = st.actions.get(B.GP_ACT_GROW, 0) + st.actions.get(B.GP_ACT_COMPRESS_FALLBACK, 0)
    comps = st.actions.get(B.GP_ACT_COMPRESS, 0)
    assert grows > 0 and comps + st.actions.get(B.GP_ACT_COMPRESS_FALLBACK, 0) > 0
    if over["policy"] == B.GP_POLICY_RANDOM:
        frac = comps / max(grows + comps, 1)
        assert abs(frac - over.get("p_compress", 0.7)) < 0.25


@pytest.mark.parametrize("config,over,mixed", [
    (1, dict(min_capacity=64), False),                 # the paper's thresholds: the floor stops most Shrinks
    (1, dict(min_capacity=48, tau=-0.06, shrink_below=-0.085), True),
    (5, dict(min_capacity=64), False),                 # shared prompt pages: copy-on-write before a Shrink writes
    (5, dict(min_capacity=64, tau=-0.03, shrink_below=-0.036), True)])
def test_shrink_policy_of_eq13(config, over, mixed):
    """Three-way capacity control: grants, Compress & Hold, and Shrinks that evict two pages worth per (layer,
    head) and hand a page back, against the oracle step by step (actions, retained sets, page tables, free list,
    reference counts).  The thresholds of the mixed cases sit inside the range Delta_t takes on these inputs, so
    that all three actions occur."""
    st = LS.run_lockstep(W.parity_instance(config), policy=B.GP_POLICY_SHRINK, **over)
    _report(f"config {config} shrink {over}", st)
    assert st.actions.get(B.GP_ACT_SHRINK, 0) > 0 and st.counters[10] == st.actions[B.GP_ACT_SHRINK]
    if mixed:
        assert st.actions.get(B.GP_ACT_GROW, 0) > 0 and st.actions.get(B.GP_ACT_COMPRESS, 0) > 0
    if config == 5:
        assert st.counters[4] > 0


def test_layer_by_layer_entry_points_equal_the_whole_step():
    # gp_step_begin / gp_attn_layer (layers in a shuffled order) / gp_step_end against gp_decode_step on the same
    # inputs: actions, page state, retained sets and summaries bit for bit, outputs to fp32 rounding; and the
    # state checks
    import torch
    shape = W.Shape(5, 8, 2, 64)
    reqs = [W.RequestSpec(i, 150 + 37 * i, 60, 0.05) for i in range(6)]
    wl = W.Workload("layers", 31, shape, reqs, n_resident=6, initial_pages=0, max_pages_per_req=48, n_pages=6 * 48)
    s, n, T = shape, 6, 60
    q = np.empty((T, s.n_layers, n, s.n_q_heads, s.head_dim), dtype=np.uint16)
    k = np.empty((T, s.n_layers, n, s.n_kv_heads, s.head_dim), dtype=np.uint16)
    v = np.empty_like(k)
    prompts = []
    for i in range(n):
        st = wl.stream(reqs[i])
        prompts.append(st.prompt_kv())
        q[:, :, i], k[:, :, i], v[:, :, i] = st.steps(0, T)
    dev = lambda a: torch.from_numpy(a.view(np.int16)).to("cuda:0")
    qd, kd, vd = dev(q), dev(k), dev(v)
    ids = torch.arange(n, dtype=torch.int32, device="cuda:0")
    rng = np.random.default_rng(0)
    results = []
    for by_layer in (False, True):
        pool = B.Pool(B.make_config(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, n_pages=wl.n_pages,
                                    max_pages_per_req=48, max_requests=8, tau=-0.05))
        try:
            for i in range(n):
                assert pool.request_add(-1, 0, prompts[i][0], prompts[i][1], reqs[i].prompt_len, 0)[0] == B.GP_OK
            outs = torch.zeros((T, s.n_layers, n, s.n_q_heads, s.head_dim), dtype=torch.float32, device="cuda:0")
            acts = torch.zeros((T, n), dtype=torch.int32, device="cuda:0")
            if by_layer:
                h, strm = pool.handle, pool.stream()
                with pytest.raises(B.GpError):                       # no step begun
                    B.gp_step_end(h, ids.data_ptr(), n, acts[0].data_ptr(), strm)
                for t in range(T):
                    B.gp_step_begin(h, ids.data_ptr(), n, acts[t].data_ptr(), strm)
                    if t == 0:
                        with pytest.raises(B.GpError):               # a step is open
                            pool.decode_step(ids, qd[t], kd[t], vd[t], outs[t], acts[t])
                        with pytest.raises(B.GpError):               # not every layer done yet
                            B.gp_step_end(h, ids.data_ptr(), n, acts[t].data_ptr(), strm)
                    for layer in rng.permutation(s.n_layers):
                        layer = int(layer)
                        B.gp_attn_layer(h, layer, ids.data_ptr(), n, qd[t, layer].data_ptr(), kd[t, layer].data_ptr(),
                                        vd[t, layer].data_ptr(), outs[t, layer].data_ptr(), strm)
                    B.gp_step_end(h, ids.data_ptr(), n, acts[t].data_ptr(), strm)
            else:
                for t in range(T):
                    pool.decode_step(ids, qd[t], kd[t], vd[t], outs[t], acts[t])
            torch.cuda.synchronize()
            state = [B.gp_debug_request(pool.handle, i, 48)[:3] for i in range(n)]
            kept = [B.gp_debug_retained(pool.handle, i, s.n_layers - 1, 1, state[i][1]) for i in range(n)]
            summ = [B.gp_debug_summaries(pool.handle, i, s.n_layers, s.n_q_heads, s.head_dim) for i in range(n)]
            assert B.gp_debug_pool(pool.handle)[2][7] == 0
            results.append((outs.cpu().numpy(), acts.cpu().numpy(), state, kept, summ))
        finally:
            pool.close()
    whole, layered = results
    assert np.array_equal(whole[1], layered[1]) and whole[2] == layered[2]
    assert all(np.array_equal(a, b_) for a, b_ in zip(whole[3], layered[3]))
    assert all(np.array_equal(a, b_) for a, b_ in zip(whole[4], layered[4]))
    # the two entry points cut long requests into work items of different sizes, so the attention outputs agree
    # to the rounding of the order in which partial results are merged, not to the bit
    assert np.abs(whole[0] - layered[0]).max() <= 2e-6
    assert (whole[1] == B.GP_ACT_GROW).any() and (whole[1] == B.GP_ACT_COMPRESS).any()


def test_results_do_not_depend_on_batch_order_or_on_the_run():
    # The same steps three times: ids ascending, ids ascending again (run-to-run determinism: the histograms use
    # integer atomics only and every floating-point sum has a fixed order), and the batch in a different random
    # order every step (a request's result does not depend on its position in the batch or on its neighbours):
    # outputs, actions, page tables, retained sets and summaries must be equal bit for bit.
    import torch
    shape = W.Shape(2, 8, 2, 64)
    reqs = [W.RequestSpec(i, 90 + 53 * i, 70, 0.05) for i in range(7)]
    wl = W.Workload("order", 37, shape, reqs, n_resident=7, initial_pages=0, max_pages_per_req=40, n_pages=7 * 40)
    s, n, T = shape, 7, 70
    q = np.empty((T, s.n_layers, n, s.n_q_heads, s.head_dim), dtype=np.uint16)
    k = np.empty((T, s.n_layers, n, s.n_kv_heads, s.head_dim), dtype=np.uint16)
    v = np.empty_like(k)
    prompts = []
    for i in range(n):
        st = wl.stream(reqs[i])
        prompts.append(st.prompt_kv())
        q[:, :, i], k[:, :, i], v[:, :, i] = st.steps(0, T)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to("cuda:0")
    rng = np.random.default_rng(1)
    results = []
    for mode in ("sorted", "sorted", "shuffled"):
        pool = B.Pool(B.make_config(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, n_pages=wl.n_pages,
                                    max_pages_per_req=40, max_requests=8, tau=-0.05))
        try:
            for i in range(n):
                assert pool.request_add(-1, 0, prompts[i][0], prompts[i][1], reqs[i].prompt_len, 0)[0] == B.GP_OK
            outs = np.zeros((T, s.n_layers, n, s.n_q_heads, s.head_dim), dtype=np.float32)
            acts = np.zeros((T, n), dtype=np.int32)
            for t in range(T):
                perm = rng.permutation(n) if mode == "shuffled" else np.arange(n)
                ids = torch.tensor(perm, dtype=torch.int32, device="cuda:0")
                out = torch.zeros((s.n_layers, n, s.n_q_heads, s.head_dim), dtype=torch.float32, device="cuda:0")
                act = torch.zeros(n, dtype=torch.int32, device="cuda:0")
                pool.decode_step(ids, dev(q[t][:, perm]), dev(k[t][:, perm]), dev(v[t][:, perm]), out, act)
                outs[t][:, perm] = out.cpu().numpy()
                acts[t][perm] = act.cpu().numpy()
            state = [B.gp_debug_request(pool.handle, i, 40) for i in range(n)]
            kept = [B.gp_debug_retained(pool.handle, i, 1, 1, state[i][1]) for i in range(n)]
            summ = [B.gp_debug_summaries(pool.handle, i, s.n_layers, s.n_q_heads, s.head_dim) for i in range(n)]
            assert B.gp_debug_pool(pool.handle)[2][7] == 0
            results.append((outs, acts, state, kept, summ))
        finally:
            pool.close()
    first = results[0]
    assert (first[1] == B.GP_ACT_GROW).any() and (first[1] == B.GP_ACT_COMPRESS).any()
    for other in results[1:]:
        assert np.array_equal(first[1], other[1]) and first[2] == other[2]
        assert all(np.array_equal(a, b_) for a, b_ in zip(first[3], other[3]))
        assert all(np.array_equal(a, b_) for a, b_ in zip(first[4], other[4]))
        assert np.array_equal(first[0], other[0])


class _ScaledStream:
    """A request's inputs with queries and keys multiplied by a power of two (exact in bf16)."""

    def __init__(self, inner, q_scale, k_scale):
        self.inner, self.q_scale, self.k_scale = inner, q_scale, k_scale

    @staticmethod
    def _mul(bits, f):
        return W.f32_to_bf16_bits((W.bf16_bits_to_f64(bits) * f).astype(np.float32))

    def prompt_kv(self):
        k, v = self.inner.prompt_kv()
        return self._mul(k, self.k_scale), v

    def steps(self, t0, t1):
        q, k, v = self.inner.steps(t0, t1)
        return self._mul(q, self.q_scale), self._mul(k, self.k_scale), v


_ALWAYS_SHRINK = dict(policy=B.GP_POLICY_SHRINK, shrink_below=0.5, tau=1.0, min_capacity=48)


@pytest.mark.parametrize("config,q_scale,k_scale,steps,over", [
    (1, 16.0, 8.0, 256, {}), (1, 16.0, 1.0, 120, {}), (1, 64.0, 32.0, 120, {}), (1, 1.0 / 64, 1.0 / 64, 120, {}),
    (2, 8.0, 4.0, 40, {}), (1, 16.0, 8.0, 120, _ALWAYS_SHRINK), (5, 16.0, 4.0, 60, _ALWAYS_SHRINK)])
def test_saturated_and_flat_softmax(config, q_scale, k_scale, steps, over):
    # Logits in the tens, hundreds or thousands: the summary probabilities of a candidate set span far more than
    # the 2^64 range the one-pass selection handles (many underflow to denormals or exactly zero, a mass of equal
    # scores under a few large ones), so working sets and eviction lists come from the general radix descent;
    # softmaxes are one-hot up to rounding and working sets hold a few tokens.  And logits near zero: uniform
    # attention, working sets of about p |C|.  All against the oracle, ties by slot order.
    wl = W.parity_instance(config)
    plain = wl.stream
    object.__setattr__(wl, "stream", lambda spec: _ScaledStream(plain(spec), q_scale, k_scale))
    st = LS.run_lockstep(wl, max_steps=steps, **over)
    _report(f"config {config}, q x{q_scale}, k x{k_scale}", st)
    assert st.decisions["sel"] > 0
    if over:
        assert st.actions.get(B.GP_ACT_SHRINK, 0) > 0


@pytest.mark.parametrize("name,shape,n_prompt,over", [
    ("rope at the 8B shape, several chunks", (2, 32, 8, 128), 1530, dict(rope_theta=1e4, tau=-0.02)),
    ("rope, G = 8, d = 64", (2, 64, 8, 64), 700, dict(rope_theta=5e5, tau=-0.02)),
    ("beta_S = 0: the short summary is the current query", (1, 8, 2, 64), 300, dict(beta_s=0.0, tau=-0.02)),
    ("beta_S = beta_L: equal summaries, Delta = 0 at every boundary", (1, 8, 2, 64), 300, dict(beta_s=0.9, beta_l=0.9)),
    ("top_p close to one", (1, 8, 2, 64), 300, dict(top_p=0.999999, tau=-0.02)),
    ("top_p small", (1, 8, 2, 64), 300, dict(top_p=0.05, tau=-0.002)),
    ("tau above any Delta: fixed budget", (1, 8, 2, 64), 300, dict(tau=1.5)),
])
def test_setting_variants_on_one_request(name, shape, n_prompt, over):
    # the paper's ablation settings (Sec. 5, "Dual-Timescale Signal Ablation": beta_S = 0; fixed budget) and the
    # ends of the parameter ranges, each against the oracle over several capacity boundaries
    st = _single_request_case(W.Shape(*shape), n_prompt, 70, **over)
    _report(name, st)
    assert st.decisions["act"] >= 3
    if ("beta_l" in over and over["beta_l"] == over["beta_s"]) or over.get("tau", 0) > 1:
        assert st.actions.get(B.GP_ACT_GROW, 0) == 0


def test_sequence_lengths_around_chunk_and_page_edges():
    # a request is cut into chunks of 32 pages (512 tokens), boundary requests into chunks of 8 pages; every
    # length around those edges and around a page edge, a few steps each (the append crosses the edge), attention
    # and boundary decisions against the oracle
    lengths = list(range(505, 520)) + list(range(1018, 1030)) + [127, 128, 129, 255, 256, 257, 2047, 2048, 2049]
    for n_prompt in lengths:
        st = _single_request_case(W.Shape(1, 8, 2, 64), n_prompt, 3, seed=n_prompt, tau=-0.02)
        assert st.steps == 3 and st.attn_max_abs <= LS.ATTN_MAX_ABS


def test_host_entry_point_with_pageable_buffers_and_without_the_final_wait():
    # gp_decode_step_host fetches pinned inputs with one kernel over the bus (the ids fill whole 16-byte pieces
    # here: four requests) and writes pinned outputs over the bus as it runs; pageable buffers take copies.
    # gp_decode_step_host_async is the same without the synchronisation at the end: the loop below issues step t,
    # then waits for step t - 1 (gp_decode_step_host_wait) and reads its results from the other of two pairs of
    # result buffers.
    import torch
    cfg = B.make_config(1, 8, 2, 64, n_pages=32, max_pages_per_req=4, max_requests=8, host_staging=True)
    results = []
    for mode in ("pinned", "pageable", "pinned, one step behind"):
        pool = B.Pool(cfg)
        try:
            rng = np.random.default_rng(0)
            bits = lambda *shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
            kt, vt = bits(1, 20, 2, 64), bits(1, 20, 2, 64)
            for i in range(4):
                assert pool.request_add(-1, 0, kt, vt, 20, 0) == (B.GP_OK, i)
            fix = (lambda t: t) if mode == "pageable" else (lambda t: t.pin_memory())
            outs, pending, keep = [], None, []
            for t in range(14):                                   # crosses the boundary at n = 32
                q, k, v = bits(1, 4, 8, 64), bits(1, 4, 2, 64), bits(1, 4, 2, 64)
                out = fix(torch.zeros((1, 4, 8, 64), dtype=torch.float32))
                act = fix(torch.zeros(4, dtype=torch.int32))
                ids = fix(torch.arange(4, dtype=torch.int32))
                tq, tk, tv = (fix(torch.from_numpy(x.view(np.int16))) for x in (q, k, v))
                if mode.endswith("behind"):
                    keep.append((ids, tq, tk, tv))                # the inputs stay as they are until their step has run
                    pool.decode_step_host_async(ids, tq, tk, tv, out, act)
                    if pending is not None:
                        pool.host_wait()                          # the call before this one
                        outs.append((pending[1].clone().numpy(), pending[2].clone().numpy()))
                    pending = (None, out, act)
                else:
                    pool.decode_step_host(ids, tq, tk, tv, out, act)
                    outs.append((out.clone().numpy(), act.clone().numpy()))
            if pending is not None:
                pool.host_wait()
                outs.append((pending[1].clone().numpy(), pending[2].clone().numpy()))
                assert B.gp_pool_status(pool.handle) == (B.GP_OK, 0)
            results.append(outs)
            assert B.gp_debug_pool(pool.handle)[2][7] == 0
        finally:
            pool.close()
    for other in results[1:]:
        for (o1, a1), (o2, a2) in zip(results[0], other):
            assert np.array_equal(o1, o2) and np.array_equal(a1, a2)
    assert any((a != B.GP_ACT_NONE).any() for _, a in results[0])


def test_largest_page_cap_still_launches_the_selection_kernel():
    # the selection kernel's shared memory grows with the per-request page cap (one bit per candidate token);
    # at the largest cap the configuration check admits, the kernel must still launch and decide as the oracle
    wl = W.Workload("cap", 41, W.Shape(1, 4, 1, 64), [W.RequestSpec(0, 200, 40, 0.05)], n_resident=1, initial_pages=0,
                    max_pages_per_req=61000, n_pages=64)
    st = LS.run_lockstep(wl, tau=-0.02)
    _report("cap 61000", st)
    assert st.decisions["act"] >= 2


@pytest.mark.parametrize("seed,pol", [(2024, {}), (7, dict(policy=B.GP_POLICY_SHRINK, shrink_below=0.0, min_capacity=48)),
                                      (11, dict(policy=B.GP_POLICY_RANDOM, policy_seed=5, p_compress=0.5))])
def test_random_admissions_sharing_steps_and_releases(seed, pol):
    # a seeded random walk over the public calls: admissions with and without shared prompt pages (from donors at
    # any stage, with tails of any length, valid and invalid), decode steps on random subsets in random order,
    # releases; after every call the two sides must agree on statuses, ids, actions, page counts, token counts,
    # positions, free pages and the multiset of reference counts, and on the attention outputs
    import torch
    L, Hq, Hkv, d, b = 1, 4, 2, 64, 16
    kw = dict(n_pages=72, max_pages_per_req=9, max_requests=8, k_loc=2, tau=0.0)
    gpu = B.Pool(B.make_config(L, Hq, Hkv, d, **kw, **pol))
    ora = O.OraclePool(O.OracleConfig(L, Hq, Hkv, d, **kw, **pol))
    rng = np.random.default_rng(seed)
    bits = lambda *shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    o_map = {O.OK: B.GP_OK, O.ERR_INVALID: B.GP_ERR_INVALID, O.ERR_NO_SLOT: B.GP_ERR_NO_SLOT, O.ERR_NO_PAGES: B.GP_ERR_NO_PAGES}
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to("cuda:0")
    live = []
    counts = {"add": 0, "add_shared": 0, "add_refused": 0, "step": 0, "release": 0}
    actions_seen = {}

    def check_state():
        n_free, ref, counters = B.gp_debug_pool(gpu.handle, kw["n_pages"])
        assert counters[7] == 0 and n_free == ora.n_free()
        assert sorted(ref[ref > 0].tolist()) == sorted(ora.refcount[ora.refcount > 0].tolist())
        for rid in live:
            assert B.gp_debug_request(gpu.handle, rid, 9)[:3] == ora.request_state(rid)[:3], rid

    try:
        for it in range(420):
            u = rng.random()
            if u < 0.2 or not live:
                share = int(rng.choice(live)) if live and rng.random() < 0.6 else int(rng.integers(-1, 8))
                n_sh = int(rng.integers(0, 5)) if share >= 0 else 0
                n_tail = int(rng.integers(0, 45))
                init = int(rng.integers(0, 7))
                kt, vt = (bits(L, n_tail, Hkv, d), bits(L, n_tail, Hkv, d)) if n_tail else (None, None)
                g_st, g_rid = gpu.request_add(share, n_sh, kt, vt, n_tail, init)
                o_st, o_rid = ora.request_add(share, n_sh, None if kt is None else H.decode_bits(kt),
                                              None if vt is None else H.decode_bits(vt), n_tail, init)
                assert g_st == o_map[o_st], (it, "add", share, n_sh, n_tail, init, g_st, o_st)
                if g_st == B.GP_OK:
                    assert g_rid == o_rid
                    live.append(g_rid)
                    counts["add_shared" if n_sh else "add"] += 1
                else:
                    counts["add_refused"] += 1
            elif u < 0.94:
                k_sub = int(rng.integers(1, len(live) + 1))
                rids = [int(x) for x in rng.permutation(live)[:k_sub]]
                if rng.random() < 0.1 and len(rids) < 8:              # a batch holds at most max_requests ids
                    rids.append(int(rng.integers(0, 8)))              # a repeated, dead or live extra id
                Bn = len(rids)
                q, k, v = bits(L, Bn, Hq, d), bits(L, Bn, Hkv, d), bits(L, Bn, Hkv, d)
                out = torch.zeros((L, Bn, Hq, d), dtype=torch.float32, device="cuda:0")
                act = torch.zeros(Bn, dtype=torch.int32, device="cuda:0")
                gpu.decode_step(torch.tensor(rids, dtype=torch.int32, device="cuda:0"), dev(q), dev(k), dev(v), out, act)
                rec = ora.decode_step(rids, H.decode_bits(q), H.decode_bits(k), H.decode_bits(v))
                a = act.cpu().numpy()
                assert np.array_equal(a, rec.actions), (it, rids, a, rec.actions)
                stepped = [i for i in range(Bn) if a[i] >= 0]
                if stepped:
                    err = np.abs(out.cpu().numpy().astype(np.float64)[:, stepped] - rec.out[:, stepped]).max()
                    assert err <= LS.ATTN_MAX_ABS, (it, err)
                for x in a:
                    actions_seen[int(x)] = actions_seen.get(int(x), 0) + 1
                counts["step"] += 1
            else:
                rid = int(rng.choice(live))
                gpu.release(rid)
                assert ora.release(rid) == O.OK
                live.remove(rid)
                counts["release"] += 1
            check_state()
        print("\\nrandom walk:", counts, "actions", actions_seen)
        assert counts["add_shared"] >= 5 and counts["add_refused"] >= 3 and counts["release"] >= 5
        assert actions_seen.get(B.GP_ACT_COMPRESS, 0) + actions_seen.get(B.GP_ACT_COMPRESS_FALLBACK, 0) + actions_seen.get(B.GP_ACT_SHRINK, 0)
        assert actions_seen.get(B.GP_ACT_INVALID, 0)
        if pol.get("policy") == B.GP_POLICY_SHRINK:
            assert actions_seen.get(B.GP_ACT_SHRINK, 0)
        else:
            assert actions_seen.get(B.GP_ACT_GROW, 0)
    finally:
        gpu.close()


def test_random_shapes_and_settings():
    # a dozen seeded draws of geometry (layers, heads, group size, head dimension), prompt lengths, quota, coverage,
    # smoothing, threshold, RoPE and policy, each a short lockstep run of three requests
    rng = np.random.default_rng(99)
    for trial in range(12):
        G = int(rng.choice([1, 2, 4, 8]))
        Hkv = int(rng.choice([1, 2, 3, 4]))
        d = int(rng.choice([64, 128]))
        L = int(rng.integers(1, 4))
        shape = W.Shape(L, Hkv * G, Hkv, d)
        reqs = [W.RequestSpec(i, int(rng.integers(1, 330)), 44, float(rng.uniform(0.01, 0.2))) for i in range(3)]
        cap = max(r.prompt_len for r in reqs) // 16 + 3
        wl = W.Workload(f"draw{trial}", 1000 + trial, shape, reqs, n_resident=3, initial_pages=int(rng.integers(0, 4)),
                        max_pages_per_req=cap, n_pages=3 * cap - int(rng.integers(0, 4)))
        over = dict(k_loc=int(rng.integers(0, 9)), top_p=float(rng.choice([0.8, 0.95, 0.99, 0.999])),
                    beta_s=float(rng.choice([0.0, 0.5, 0.9])), beta_l=float(rng.choice([0.99, 0.999])),
                    tau=float(rng.choice([-0.05, -0.01, 0.0])), rope_theta=float(rng.choice([0.0, 1e4])))
        if rng.random() < 0.4:
            over.update(policy=B.GP_POLICY_SHRINK, shrink_below=float(rng.choice([-0.03, 0.5])), min_capacity=48)
        st = LS.run_lockstep(wl, **over)
        _report(f"draw {trial}: {shape} prompts {[r.prompt_len for r in reqs]} {over}", st)


def test_a_32k_token_request_at_the_32b_head_shape():
    # the longest sequence of the multi-layer configurations (32 768 tokens, 64 query heads over 8 KV heads): 64
    # work items per (layer, head), candidate sets five times the selection kernel's staging buffers, 2047
    # candidate pages; grows to its cap, then a fallback compression over 32k candidates
    st = _single_request_case(W.Shape(1, 64, 8, 128), 32760, 60)
    _report("32760-token request, 32B head shape", st)
    assert st.actions.get(B.GP_ACT_GROW, 0) == 3 and st.actions.get(B.GP_ACT_COMPRESS_FALLBACK, 0) == 1
    assert st.decisions["sel"] == 8


def test_overlapped_launches_equal_plain_launches():
    # In the normal mode the kernels of a step are chained with programmatic dependent launch; with early
    # planning on, the plan of a step also runs beside the compaction of the step before; in profiling mode every
    # kernel is launched the plain way, after the one before it has ended.  Same inputs, all three: outputs,
    # actions, page tables, retained sets and summaries must be equal bit for bit.
    import torch
    wl = W.layer8b(seed=5, n_requests=24, n_steps=200, prompt_range=(100, 700))
    s = wl.shape
    n, T = len(wl.requests), 200
    q = np.empty((T, s.n_layers, n, s.n_q_heads, s.head_dim), dtype=np.uint16)
    k = np.empty((T, s.n_layers, n, s.n_kv_heads, s.head_dim), dtype=np.uint16)
    v = np.empty_like(k)
    prompts = []
    for i in range(n):
        st = wl.stream(wl.requests[i])
        prompts.append(st.prompt_kv())
        q[:, :, i], k[:, :, i], v[:, :, i] = st.steps(0, T)
    dev = lambda a: torch.from_numpy(a.view(np.int16)).to("cuda:0")
    qd, kd, vd = dev(q), dev(k), dev(v)
    ids = torch.arange(n, dtype=torch.int32, device="cuda:0")
    results = []
    for plain, early in ((False, False), (True, False), (False, True)):
        pool = B.Pool(B.make_config(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, n_pages=wl.n_pages,
                                    max_pages_per_req=wl.max_pages_per_req, max_requests=n, tau=-0.003))
        try:
            for i in range(n):
                assert pool.request_add(-1, 0, prompts[i][0], prompts[i][1], wl.requests[i].prompt_len, 0)[0] == B.GP_OK
            B.gp_set_profiling(pool.handle, plain)
            B.gp_set_early_plan(pool.handle, early)
            outs = torch.zeros((T, s.n_layers, n, s.n_q_heads, s.head_dim), dtype=torch.float32, device="cuda:0")
            acts = torch.zeros((T, n), dtype=torch.int32, device="cuda:0")
            for t in range(T):
                pool.decode_step(ids, qd[t], kd[t], vd[t], outs[t], acts[t])
            torch.cuda.synchronize()
            state = [B.gp_debug_request(pool.handle, i, wl.max_pages_per_req) for i in range(n)]
            kept = [B.gp_debug_retained(pool.handle, i, 0, 3, state[i][1]) for i in range(n)]
            summ = [B.gp_debug_summaries(pool.handle, i, s.n_layers, s.n_q_heads, s.head_dim) for i in range(0, n, 5)]
            assert B.gp_debug_pool(pool.handle)[2][7] == 0
            results.append((outs.cpu().numpy(), acts.cpu().numpy(), state, kept, summ))
        finally:
            pool.close()
    a = results[0]
    for b_ in results[1:]:
        assert np.array_equal(a[1], b_[1]) and a[2] == b_[2]
        assert all(np.array_equal(x, y) for x, y in zip(a[3], b_[3])) and all(np.array_equal(x, y) for x, y in zip(a[4], b_[4]))
        assert np.array_equal(a[0], b_[0])
    assert (a[1] == B.GP_ACT_GROW).any() and (a[1] == B.GP_ACT_COMPRESS).any()


@pytest.mark.parametrize("config,over", [(1, {}), (1, dict(tau=-0.2)), (2, dict(tau=-0.02)), (5, dict(async_boundary=True))])
def test_entropy_as_the_working_set_metric(config, over):
    # the ablation's other demand metric: Delta_t from the views' entropies; selection and compaction unchanged
    st = LS.run_lockstep(W.parity_instance(config), demand_metric=B.GP_METRIC_ENTROPY, max_steps=200, **over)
    _report(f"entropy config{config} {over}", st)
    assert st.decisions["act"] > 0 and st.near_ties["act"] == 0
    if over.get("tau", 0.0) <= -0.2:
        assert st.actions.get(B.GP_ACT_GROW, 0) > 0


def test_preempted_request_is_readmitted_with_its_history_and_fresh_summaries():
    """The scheduler's preemption (App. D.1: a preempted request gives its slot and pages back and, when it is
    scheduled again, binds a slot anew and starts its summaries over): a request is released in mid-generation and
    admitted again with everything it has seen so far as its prompt.  Both sides do the same; the slot's stale
    summaries must not leak into the second life (the first step overwrites them), and the pages come back."""
    import torch
    L, Hq, Hkv, d, b = 2, 8, 2, 64, 16
    kw = dict(n_pages=40, max_pages_per_req=12, max_requests=4, k_loc=4, tau=-0.05)
    gpu = B.Pool(B.make_config(L, Hq, Hkv, d, **kw))
    ora = O.OraclePool(O.OracleConfig(L, Hq, Hkv, d, **kw))
    rng = np.random.default_rng(23)
    bits = lambda *shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to("cuda:0")
    f = W.bf16_bits_to_f64
    try:
        hist_k, hist_v = bits(L, 40, Hkv, d), bits(L, 40, Hkv, d)          # the prompt, then every decoded token
        other_k, other_v = bits(L, 25, Hkv, d), bits(L, 25, Hkv, d)
        for (k0, v0, n0) in ((hist_k, hist_v, 40), (other_k, other_v, 25)):
            g = gpu.request_add(-1, 0, k0, v0, n0, 0)
            o = ora.request_add(-1, 0, f(k0), f(v0), n0, 0)
            assert g == (B.GP_OK, o[1])

        def steps(n, rids):
            nonlocal hist_k, hist_v
            for _ in range(n):
                q, k, v = bits(L, len(rids), Hq, d), bits(L, len(rids), Hkv, d), bits(L, len(rids), Hkv, d)
                out = torch.zeros((L, len(rids), Hq, d), dtype=torch.float32, device="cuda:0")
                act = torch.zeros(len(rids), dtype=torch.int32, device="cuda:0")
                gpu.decode_step(torch.tensor(rids, dtype=torch.int32, device="cuda:0"), dev(q), dev(k), dev(v), out, act)
                rec = ora.decode_step(rids, f(q), f(k), f(v))
                assert act.cpu().tolist() == rec.actions.tolist()
                assert np.abs(out.cpu().numpy() - rec.out).max() <= LS.ATTN_MAX_ABS
                if 0 in rids:
                    i = rids.index(0)
                    hist_k = np.concatenate([hist_k, k[:, i:i + 1]], axis=1)
                    hist_v = np.concatenate([hist_v, v[:, i:i + 1]], axis=1)

        def same_state(rid):
            assert B.gp_debug_request(gpu.handle, rid, 12)[:3] == ora.request_state(rid)[:3]
            g, o = B.gp_debug_summaries(gpu.handle, rid, L, Hq, d), ora.summaries(rid)
            assert (np.linalg.norm(g - o, axis=-1) / np.linalg.norm(o, axis=-1)).max() <= LS.SUMMARY_REL
            for l in range(L):
                for h in range(Hkv):
                    n = ora.request_state(rid)[1]
                    assert np.array_equal(B.gp_debug_retained(gpu.handle, rid, l, h, n), ora.retained(rid, l, h))

        steps(37, [0, 1])                                   # past two boundaries of request 0 (48 and 64 or 48 again)
        same_state(0); same_state(1)
        stale = B.gp_debug_summaries(gpu.handle, 0, L, Hq, d)
        free_before = B.gp_debug_pool(gpu.handle)[0]
        held = B.gp_debug_request(gpu.handle, 0, 12)[0]
        gpu.release(0); assert ora.release(0) == O.OK                              # preempted
        assert B.gp_debug_pool(gpu.handle)[0] == free_before + held == ora.n_free()
        steps(5, [1])                                       # the other request goes on alone
        n_hist = hist_k.shape[1]
        g = gpu.request_add(-1, 0, hist_k, hist_v, n_hist, 0)                      # scheduled again: same slot, new life
        o = ora.request_add(-1, 0, f(hist_k), f(hist_v), n_hist, 0)
        assert g == (B.GP_OK, 0) and o == (O.OK, 0)
        assert B.gp_debug_request(gpu.handle, 0, 12)[:3] == (n_hist // b + 1, n_hist, n_hist)
        steps(1, [0, 1])
        fresh = B.gp_debug_summaries(gpu.handle, 0, L, Hq, d)
        assert np.array_equal(fresh[:, 0], fresh[:, 1]) and not np.allclose(fresh, stale)   # S = L = the first query again
        steps(40, [0, 1])
        same_state(0); same_state(1)
        n_free, ref, counters = B.gp_debug_pool(gpu.handle, 40)
        assert counters[7] == 0 and n_free == ora.n_free()
    finally:
        gpu.close()


@pytest.mark.parametrize("rope_theta,hq,hkv,d", [(0.0, 8, 2, 64), (1e4, 8, 2, 128), (1e6, 16, 2, 64)])
def test_layer_entry_with_fused_query_key_normalisation(rope_theta, hq, hkv, d):
    """gp_attn_layer_qknorm takes the projections' raw outputs; the oracle is fed what a plain implementation of
    the model's normalisation gives: per head x / sqrt(mean(x^2) + eps) * weight in float64, the key then rotated
    to its position, both rounded to bf16.  Everything downstream (attention, summaries taken after the
    normalisation and before the rotation, boundaries, retained sets) must agree as in the other lockstep tests."""
    import torch
    L, b, eps = 3, 16, 1e-6
    kw = dict(n_pages=48, max_pages_per_req=5, max_requests=4, k_loc=4, tau=-0.03, rope_theta=rope_theta)   # the cap forces compressions
    gpu = B.Pool(B.make_config(L, hq, hkv, d, **kw))
    ora = O.OraclePool(O.OracleConfig(L, hq, hkv, d, **kw))
    rng = np.random.default_rng(31)
    bits = lambda *shape: W.f32_to_bf16_bits((2.5 * rng.standard_normal(shape)).astype(np.float32))
    f = W.bf16_bits_to_f64
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to("cuda:0")
    wq = (1.0 + 0.3 * rng.standard_normal((L, d))).astype(np.float32)
    wk = (1.0 + 0.3 * rng.standard_normal((L, d))).astype(np.float32)
    wq_d, wk_d = torch.from_numpy(wq).cuda(), torch.from_numpy(wk).cuda()
    round_bf16 = lambda x: W.f32_to_bf16_bits(x.astype(np.float32))              # double -> float -> bf16

    def normalise(x_bits, w):                                                      # [.., heads, d] per head
        x = f(x_bits)
        return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * w.astype(np.float64)

    try:
        prompts = (21, 40, 13)
        for n0 in prompts:
            kp, vp = bits(L, n0, hkv, d), bits(L, n0, hkv, d)
            assert gpu.request_add(-1, 0, kp, vp, n0, 0)[0] == B.GP_OK
            assert ora.request_add(-1, 0, f(kp), f(vp), n0, 0)[0] == O.OK
        n_req = len(prompts)
        ids = torch.arange(n_req, dtype=torch.int32, device="cuda:0")
        seen = {}
        for t in range(60):
            q_raw, k_raw, v = bits(L, n_req, hq, d), bits(L, n_req, hkv, d), bits(L, n_req, hkv, d)
            pos = [ora.request_state(r)[2] for r in range(n_req)]
            q_n = np.stack([round_bf16(normalise(q_raw[l], wq[l])) for l in range(L)])
            k_n = np.stack([np.stack([round_bf16(O.rope(normalise(k_raw[l, r], wk[l]), pos[r], rope_theta)) for r in range(n_req)])
                            for l in range(L)])
            rec = ora.decode_step(list(range(n_req)), f(q_n), f(k_n), f(v))
            out = torch.zeros((L, n_req, hq, d), dtype=torch.float32, device="cuda:0")
            act = torch.zeros(n_req, dtype=torch.int32, device="cuda:0")
            qd, kd, vd = dev(q_raw), dev(k_raw), dev(v)
            s_ = gpu.stream()
            B.gp_step_begin(gpu.handle, ids.data_ptr(), n_req, act.data_ptr(), s_)
            for l in rng.permutation(L):
                l = int(l)
                B.gp_attn_layer_qknorm(gpu.handle, l, ids.data_ptr(), n_req, qd[l].data_ptr(), kd[l].data_ptr(), vd[l].data_ptr(),
                                       wq_d[l].data_ptr(), wk_d[l].data_ptr(), eps, out[l].data_ptr(), s_)
            B.gp_step_end(gpu.handle, ids.data_ptr(), n_req, act.data_ptr(), s_)
            assert act.cpu().tolist() == rec.actions.tolist(), t
            assert np.abs(out.cpu().numpy() - rec.out).max() <= LS.ATTN_MAX_ABS, t
            for a in rec.actions.tolist():
                seen[a] = seen.get(a, 0) + 1
        assert seen.get(B.GP_ACT_GROW, 0) > 0 and seen.get(B.GP_ACT_COMPRESS, 0) + seen.get(B.GP_ACT_COMPRESS_FALLBACK, 0) > 0, seen
        for r in range(n_req):
            assert B.gp_debug_request(gpu.handle, r, 5)[:3] == ora.request_state(r)[:3]
            g, o = B.gp_debug_summaries(gpu.handle, r, L, hq, d), ora.summaries(r)
            assert (np.linalg.norm(g - o, axis=-1) / np.linalg.norm(o, axis=-1)).max() <= LS.SUMMARY_REL
            n = ora.request_state(r)[1]
            for l in range(L):
                for h in range(hkv):
                    assert np.array_equal(B.gp_debug_retained(gpu.handle, r, l, h, n), ora.retained(r, l, h))
                    kk, _ = B.gp_debug_kv(gpu.handle, r, l, h, n, d)
                    assert np.array_equal(f(kk), ora.requests[r].K[l, h, :n]), "the cached keys are not the normalised, rotated ones"
        assert B.gp_debug_pool(gpu.handle)[2][7] == 0
    finally:
        gpu.close()
