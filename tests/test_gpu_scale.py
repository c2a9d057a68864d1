"""Properties that hold at any size, checked on mid-sized instances of the multi-layer configurations.

The float64 oracle follows the reduced instances of these configurations element by element (test_gpu_parity);
here the instances are an order of magnitude larger (tens of resident requests, several layers, continuous
batching with admissions and releases, a pool under pressure, shared prompts), too large for the oracle, and the
C-ABI path is checked against what the method fixes whatever the inputs:

  * a capacity boundary is reached exactly when the appended token fills the last page, and only there is an
    action other than "none" reported; a grant adds one page and one token, a compression leaves the page count
    and sets the token count to (P - 1) * b;
  * page accounting: free pages + distinct pages held = pool size, every page's reference count equals the
    number of page tables that hold it, and a request that has compacted holds no shared page any more
    (copy-on-write is complete);
  * the retained token ids of a (layer, head) are strictly increasing, end at the newest token, and the newest
    page worth of tokens is always retained (the protected recent window);
  * the attention output of a request is the softmax-weighted mean of the values it retains, recomputed here in
    float64 numpy from the keys and values read back from the pool;
  * step and token counters, no kernel error bit, and an empty pool after every request is released.
"""
import numpy as np
import pytest

from paper_2609_03494_b200 import binding as B
from paper_2609_03494_b200 import harness as H
from paper_2609_03494_b200 import workload as W

pytestmark = pytest.mark.gpu

ATTN_MAX_ABS = 1e-2


def _instance(name: str, tau: float) -> W.Workload:
    if name == "stack8b":
        wl = W.stack8b(n_layers=8, n_resident=40, n_total=72, out_range=(48, 224), prompt_range=(128, 1024))
        wl.n_pages = 40 * 39                    # under what 40 residents ask for: fallbacks and stalls happen
        return wl
    if name == "stack32b":
        wl = W.stack32b(n_layers=4, n_requests=24, out_range=(96, 256), prompt_range=(128, 1024))
        wl.n_pages = 24 * 80
        return wl
    if name == "prefix":
        wl = W.prefix_stress(n_groups=6, group_size=8, prompt_len=1024, n_steps=160, initial_pages=8, extra_pages=3)
        if tau < 0:
            # Every request may grow by five pages (its cap), and the pool holds the shared prompts once, every
            # request at its cap, and 640 pages more.  At the cap a request that asks for a page compresses instead
            # (fallback), which needs 64 pages for its copies-on-write: ten requests get them, the others stall
            # and are released by the scheduler.
            wl.max_pages_per_req = 65 + 5
            wl.n_pages = 6 * 64 + 48 * 6 + 640
        return wl
    if name == "many":
        # the most requests a pool takes (512), short sequences, dozens of boundaries in every step, a pool that
        # runs dry: the planning, decision and compaction bookkeeping at their widest
        g = np.random.default_rng(5)
        reqs = [W.RequestSpec(i, int(g.integers(1, 61)), int(g.integers(24, 57)), 0.05) for i in range(640)]
        return W.Workload("many", 5, W.Shape(2, 8, 2, 64), reqs, n_resident=512, initial_pages=0,
                          max_pages_per_req=6, n_pages=512 * 3 + 100)
    raise ValueError(name)


def _pool_accounting(gpu, cfg, live):
    """live: request ids.  Returns the reference counts."""
    n_free, ref, counters = B.gp_debug_pool(gpu.handle, cfg.n_pages)
    assert counters[7] == 0, f"kernel error bits {counters[7]:#x}"
    held = np.zeros(cfg.n_pages, dtype=np.int64)
    for rid in live:
        P, n, pos, table = B.gp_debug_request(gpu.handle, rid, cfg.max_pages_per_req)
        assert len(set(table)) == P, f"request {rid} holds a page twice"
        held[table] += 1
    assert np.array_equal(held, ref.astype(np.int64)), "reference counts differ from the page tables"
    assert int((held > 0).sum()) + n_free == cfg.n_pages, "free pages + pages held != pool size"
    return ref


# tau below zero makes part of the boundaries ask for a page (with the synthetic streams Delta_t is seldom
# positive), so that grants, fallbacks under an empty free list and stalls all occur
@pytest.mark.parametrize("name,tau,shrink_below", [("stack8b", -0.05, None), ("stack32b", -0.03, None),
                                                  ("prefix", 0.0, None), ("prefix", -0.05, None),
                                                  ("stack8b", -0.04, -0.06), ("prefix", 0.0, -0.005),
                                                  ("many", -0.05, None), ("many", -0.03, -0.06)])
def test_invariants_under_continuous_batching(name, tau, shrink_below):
    """shrink_below set: the three-way Shrink policy (Eq. 13) with a 256-token minimum capacity."""
    import torch

    wl = _instance(name, tau)
    s = wl.shape
    b = s.page_size
    G = s.n_q_heads // s.n_kv_heads
    dev = "cuda:0"
    cfg = B.make_config(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, n_pages=wl.n_pages,
                        max_pages_per_req=wl.max_pages_per_req, max_requests=max(4, wl.n_resident), k_loc=wl.k_loc, tau=tau,
                        **(dict(policy=B.GP_POLICY_SHRINK, shrink_below=shrink_below, min_capacity=48 if name == "many" else 256)
                           if shrink_below is not None else {}),
                        # shared prompt pages count once in the pool but once per request in a batch
                        max_batch_tokens=wl.n_resident * wl.max_pages_per_req * b)
    gpu = B.Pool(cfg, 0)
    sch = H.Scheduler(wl)
    rng = np.random.default_rng(7)
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(dev)
    steps = tokens = 0
    seen = {k: 0 for k in ("none", "grow", "compress", "fallback", "shrink", "stalled", "attn", "retained")}
    compacted = set()
    try:
        while not sch.done():
            while True:
                op = sch.next_admission()
                if op is None:
                    break
                sf = sch.rid_of(op.share_from_spec) if op.share_from_spec >= 0 else -1
                st, rid = gpu.request_add(sf, op.n_shared_pages, op.k_tail, op.v_tail, op.n_tail, op.initial_pages)
                if st != B.GP_OK:
                    assert st == B.GP_ERR_NO_PAGES and sch.resident, f"admission failed with {st}"
                    break
                sch.admitted(op, rid)
                compacted.discard(rid)
            specs, rids, q, k, v = sch.batch()
            Bn = len(rids)
            before = {rid: B.gp_debug_request(gpu.handle, rid, cfg.max_pages_per_req) for rid in rids}
            ids_t = torch.tensor(rids, dtype=torch.int32, device=dev)
            out_t = torch.zeros((s.n_layers, Bn, s.n_q_heads, s.head_dim), dtype=torch.float32, device=dev)
            act_t = torch.zeros(Bn, dtype=torch.int32, device=dev)
            gpu.decode_step(ids_t, to_dev(q), to_dev(k), to_dev(v), out_t, act_t)
            act = act_t.cpu().numpy()
            steps += 1
            tokens += Bn

            # ---- actions and state transitions ---------------------------------------------------------------
            quiet = []
            for i, rid in enumerate(rids):
                P0, n0, pos0, _ = before[rid]
                P1, n1, pos1, table = B.gp_debug_request(gpu.handle, rid, cfg.max_pages_per_req)
                a = int(act[i])
                at_boundary = n0 + 1 == P0 * b
                if not at_boundary:
                    assert a == B.GP_ACT_NONE and (P1, n1, pos1) == (P0, n0 + 1, pos0 + 1), (steps, rid, a)
                    seen["none"] += 1
                    quiet.append(i)
                elif a == B.GP_ACT_GROW:
                    assert (P1, n1, pos1) == (P0 + 1, n0 + 1, pos0 + 1) and P1 <= cfg.max_pages_per_req
                    seen["grow"] += 1
                    quiet.append(i)
                elif a in (B.GP_ACT_COMPRESS, B.GP_ACT_COMPRESS_FALLBACK):
                    assert (P1, n1, pos1) == (P0, (P0 - 1) * b, pos0 + 1), (steps, rid, a, P0, n0, P1, n1)
                    seen["compress" if a == B.GP_ACT_COMPRESS else "fallback"] += 1
                    compacted.add(rid)
                elif a == B.GP_ACT_SHRINK:
                    assert shrink_below is not None and (P0 - 1) * b >= cfg.min_capacity
                    assert (P1, n1, pos1) == (P0 - 1, (P0 - 2) * b, pos0 + 1), (steps, rid, P0, n0, P1, n1)
                    seen["shrink"] += 1
                    compacted.add(rid)
                else:
                    assert a == B.GP_ACT_STALLED, f"step {steps} request {rid}: action {a} at a boundary"
                    seen["stalled"] += 1

            # ---- retained ids and attention of a few requests -------------------------------------------------
            for i in rng.choice(Bn, size=min(3, Bn), replace=False):
                rid = rids[i]
                a = int(act[i])
                if a == B.GP_ACT_STALLED:
                    continue
                P1, n1, pos1, _ = B.gp_debug_request(gpu.handle, rid, cfg.max_pages_per_req)
                l, h = int(rng.integers(s.n_layers)), int(rng.integers(s.n_kv_heads))
                tok = B.gp_debug_retained(gpu.handle, rid, l, h, n1).astype(np.int64)
                assert (np.diff(tok) > 0).all() and tok[-1] == pos1 - 1 and tok[0] >= 0
                w = min(b, n1)
                assert np.array_equal(tok[-w:], np.arange(pos1 - w, pos1)), "the newest page worth of tokens is not retained"
                seen["retained"] += 1
                if i in quiet:
                    kk, vv = B.gp_debug_kv(gpu.handle, rid, l, h, n1, s.head_dim)
                    kk, vv = H.decode_bits(kk), H.decode_bits(vv)
                    qq = H.decode_bits(q[l, i, h * G:(h + 1) * G])                     # [G][d]
                    z = qq @ kk.T / np.sqrt(s.head_dim)
                    p = np.exp(z - z.max(axis=1, keepdims=True))
                    want = (p / p.sum(axis=1, keepdims=True)) @ vv
                    got = out_t[l, i, h * G:(h + 1) * G].cpu().numpy().astype(np.float64)
                    assert np.abs(got - want).max() <= ATTN_MAX_ABS, f"step {steps} request {rid} ({l},{h})"
                    seen["attn"] += 1

            if steps % 16 == 0:
                ref = _pool_accounting(gpu, cfg, rids)
                for rid in compacted & set(rids):
                    _, _, _, table = B.gp_debug_request(gpu.handle, rid, cfg.max_pages_per_req)
                    assert (ref[table] == 1).all(), f"request {rid} compacted but still holds a shared page"
            for idx, rid in sch.after_step(specs, act):
                gpu.release(rid)
                compacted.discard(rid)

        n_free, ref, counters = B.gp_debug_pool(gpu.handle, cfg.n_pages)
        assert counters[7] == 0 and counters[5] == steps and counters[6] == tokens
        assert n_free == cfg.n_pages and not ref.any(), "pages leaked after every request was released"
        print(f"\n{name} tau={tau} shrink_below={shrink_below}: {steps} steps, {tokens} tokens, {seen}, cow pages {counters[4]}")
        assert seen["attn"] > 100
        if tau < 0:
            assert seen["grow"] > 0
        else:
            assert seen["compress"] + seen["shrink"] > 0
        if shrink_below is not None:
            assert seen["shrink"] > 0 and counters[10] == seen["shrink"]
        if (name == "stack8b" and shrink_below is None) or (name == "prefix" and tau < 0):
            assert seen["fallback"] + seen["stalled"] > 0, "the pool never ran dry: no pressure in this instance"
        if name == "prefix":
            assert counters[4] > 0, "no copy-on-write happened"
        if name == "prefix" and tau < 0:
            assert seen["fallback"] > 0 and seen["stalled"] > 0
    finally:
        gpu.close()


def test_pool_larger_than_four_giga_elements():
    """36 layers x 4300 pages of the 8B shape: 11 GB of K/V, element offsets beyond 2^32 (the full multi-layer
    configuration is ten times this).  Eight requests with 8192-token prompts fill 4096 pages; the prompts are
    drawn on the device.  Checked: the pool holds, bit for bit, what was ingested, at the highest offsets too;
    attention outputs equal the float64 softmax-weighted mean of what the pool holds; the boundary step (8192
    candidates per unit, 288 units per request) leaves a valid state."""
    import torch

    L, Hq, Hkv, d, b = 36, 32, 8, 128, 16
    n_req, n_prompt = 8, 8192
    P0 = n_prompt // b + 1
    cfg = B.make_config(L, Hq, Hkv, d, n_pages=4300, max_pages_per_req=P0 + 2, max_requests=n_req, tau=-1.0)
    gpu = B.Pool(cfg, 0)
    dev = "cuda:0"
    gen = torch.Generator(device=dev)
    gen.manual_seed(17)
    try:
        keep = {}
        for i in range(n_req):
            k = torch.randn((L, n_prompt, Hkv, d), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
            v = torch.randn((L, n_prompt, Hkv, d), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
            assert gpu.request_add(-1, 0, k, v, n_prompt, 0) == (B.GP_OK, i)
            # what the checks below need of this prompt: the last layer, both end heads
            keep[i] = {(l, h): (k[l, :, h].view(torch.int16).cpu().numpy().view(np.uint16),
                                v[l, :, h].view(torch.int16).cpu().numpy().view(np.uint16))
                       for (l, h) in ((0, 0), (L - 1, Hkv - 1))}
            del k, v
        P, n, pos, table = B.gp_debug_request(gpu.handle, n_req - 1, cfg.max_pages_per_req)
        assert (P, n, pos) == (P0, n_prompt, n_prompt) and max(table) >= 4000
        for i in (0, n_req - 1):
            for (l, h), (k_src, v_src) in keep[i].items():
                kk, vv = B.gp_debug_kv(gpu.handle, i, l, h, n_prompt, d)
                assert np.array_equal(kk, k_src) and np.array_equal(vv, v_src), f"request {i} ({l},{h}): pool differs from the prompt"
        ids = torch.arange(n_req, dtype=torch.int32, device=dev)
        G = Hq // Hkv
        out = torch.zeros((L, n_req, Hq, d), dtype=torch.float32, device=dev)
        act = torch.zeros(n_req, dtype=torch.int32, device=dev)
        for t in range(b + 2):
            q = torch.randn((L, n_req, Hq, d), generator=gen, device=dev).to(torch.bfloat16)
            k = torch.randn((L, n_req, Hkv, d), generator=gen, device=dev).to(torch.bfloat16)
            v = torch.randn((L, n_req, Hkv, d), generator=gen, device=dev).to(torch.bfloat16)
            gpu.decode_step(ids, q, k, v, out, act)
            a = act.cpu().numpy()
            at_boundary = t == b - 1
            assert ((a == B.GP_ACT_GROW).all() if at_boundary else (a == B.GP_ACT_NONE).all()), (t, a)
            if t in (0, b - 1, b + 1):
                for i, l, h in ((0, 0, 0), (n_req - 1, L - 1, Hkv - 1), (3, 17, 4)):
                    n1 = n_prompt + t + 1
                    kk, vv = B.gp_debug_kv(gpu.handle, i, l, h, n1, d)
                    kk, vv = H.decode_bits(kk), H.decode_bits(vv)
                    qq = q[l, i, h * G:(h + 1) * G].to(torch.float64).cpu().numpy()
                    z = qq @ kk.T / np.sqrt(d)
                    p = np.exp(z - z.max(axis=1, keepdims=True))
                    want = (p / p.sum(axis=1, keepdims=True)) @ vv
                    got = out[l, i, h * G:(h + 1) * G].cpu().numpy().astype(np.float64)
                    assert np.abs(got - want).max() <= ATTN_MAX_ABS, f"step {t} request {i} ({l},{h})"
        _pool_accounting(gpu, cfg, list(range(n_req)))
        for i in range(n_req):
            P, n, pos, _ = B.gp_debug_request(gpu.handle, i, cfg.max_pages_per_req)
            assert (P, n, pos) == (P0 + 1, n_prompt + b + 2, n_prompt + b + 2)
        # a second boundary under pressure: the pool has 4300 - 8 * 514 = 188 pages left, the cap is P0 + 2
        for t in range(b + 2, 3 * b + 2):
            q = torch.randn((L, n_req, Hq, d), generator=gen, device=dev).to(torch.bfloat16)
            k = torch.randn((L, n_req, Hkv, d), generator=gen, device=dev).to(torch.bfloat16)
            v = torch.randn((L, n_req, Hkv, d), generator=gen, device=dev).to(torch.bfloat16)
            gpu.decode_step(ids, q, k, v, out, act)
            a = act.cpu().numpy()
            if t == 2 * b - 1:
                assert (a == B.GP_ACT_GROW).all(), a                     # second boundary: up to the cap
            elif t == 3 * b - 1:
                assert (a == B.GP_ACT_COMPRESS_FALLBACK).all(), a        # third boundary, at the cap: compresses
            else:
                assert (a == B.GP_ACT_NONE).all(), (t, a)
        _pool_accounting(gpu, cfg, list(range(n_req)))
        for i in (0, n_req - 1):
            P, n, pos, _ = B.gp_debug_request(gpu.handle, i, cfg.max_pages_per_req)
            assert (P, n) == (P0 + 2, (P0 + 1) * b + 2)                  # two steps after the compression
            tok = B.gp_debug_retained(gpu.handle, i, L - 1, Hkv - 1, n).astype(np.int64)
            assert (np.diff(tok) > 0).all() and np.array_equal(tok[-b:], np.arange(pos - b, pos))
    finally:
        gpu.close()


@pytest.mark.parametrize("async_boundary", [False, True])
def test_36_layers_64_residents_with_device_side_inputs_and_continuous_batching(async_boundary):
    """The full 36-layer stack with 64 resident requests (a quarter of the configuration's residents on a pool
    scaled to the same pressure), inputs drawn on the device, requests finishing, stalling and being replaced:
    the scheduler loop and checks that the full-size runs of the benchmark use (`synth.run_at_size`)."""
    from paper_2609_03494_b200 import synth
    sc = synth.config3(n_layers=36, n_resident=64)
    sc.n_pages = 64 * 44                       # under what 64 residents of up to 1024 + 300 tokens ask for
    sc.cap_pages = 90
    res = synth.run_at_size(sc, n_steps=160, chunk=8, async_boundary=async_boundary, tau=-0.05, life_fraction=0.02,
                            check_every=4, boundary_tokens_div=2)
    print("\n", res)
    assert res["layers"] == 36 and res["steps"] == 160 and res["tokens"] > 160 * 40
    assert res["checked"]["attention"] >= 20 and res["checked"]["retained"] >= 30
    assert res["scheduler"]["finished"] > 0 and res["scheduler"]["admitted"] > 64        # continuous batching happened
    assert res["events"]["grow"] > 0 and res["events"]["compress"] + res["events"]["fallback"] > 0
