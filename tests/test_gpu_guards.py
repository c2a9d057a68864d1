"""Refusals of the C ABI that protect the pool and the GPU: misaligned tensors are turned away before any
launch, the pool cannot be changed between gp_step_begin and gp_step_end, an open step can be abandoned,
and the kernels' error word reaches the caller."""
import numpy as np
import pytest

from paper_2609_03494_b200 import binding as B
from paper_2609_03494_b200 import workload as W

pytestmark = pytest.mark.gpu

L, HQ, HKV, D = 2, 8, 2, 64


def _pool(**kw):
    cfg = B.make_config(L, HQ, HKV, D, n_pages=40, max_pages_per_req=6, max_requests=8, **kw)
    return B.Pool(cfg)


def _bits(rng, *shape):
    return W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))


def _dev(torch, a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()


def _invariants(pool, live):
    n_free, ref, counters = B.gp_debug_pool(pool.handle, 40)
    assert counters[7] == 0
    assert int((ref > 0).sum()) + n_free == 40
    held = 0
    for r in live:
        P, n, pos, table = B.gp_debug_request(pool.handle, r, 6)
        assert len(set(table)) == P and n <= P * 16
        held += P
    assert int(ref.sum()) == held
    return n_free


def test_misaligned_tensors_are_refused_before_any_launch():
    import torch
    rng = np.random.default_rng(3)
    pool = _pool()
    try:
        assert pool.request_add(-1, 0, _bits(rng, L, 20, HKV, D), _bits(rng, L, 20, HKV, D), 20, 0) == (B.GP_OK, 0)
        ids = torch.zeros(1, dtype=torch.int32, device="cuda")
        act = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = torch.zeros((L, 1, HQ, D), dtype=torch.float32, device="cuda")
        big = torch.zeros(L * HQ * D + 64, dtype=torch.int16, device="cuda")
        q = big.data_ptr()
        launches = B.gp_launch_count(pool.handle)
        s = pool.stream()
        for bad in (dict(q=q + 2), dict(k=q + 8), dict(v=q + 4), dict(out=out.data_ptr() + 4),
                    dict(ids=ids.data_ptr() + 2), dict(act=act.data_ptr() + 1)):
            a = dict(ids=ids.data_ptr(), q=q, k=q, v=q, out=out.data_ptr(), act=act.data_ptr())
            a.update(bad)
            with pytest.raises(B.GpError) as e:
                B.gp_decode_step(pool.handle, a["ids"], 1, a["q"], a["k"], a["v"], a["out"], a["act"], s)
            assert e.value.status == B.GP_ERR_INVALID, bad
        B.gp_step_begin(pool.handle, ids.data_ptr(), 1, act.data_ptr(), s)
        with pytest.raises(B.GpError) as e:
            B.gp_attn_layer(pool.handle, 0, ids.data_ptr(), 1, q + 2, q, q, out.data_ptr(), s)
        assert e.value.status == B.GP_ERR_INVALID
        B.gp_step_abort(pool.handle)
        assert B.gp_launch_count(pool.handle) == launches + 1           # only the plan of gp_step_begin ran
        torch.cuda.synchronize()
        assert B.gp_pool_status(pool.handle) == (B.GP_OK, 0)
    finally:
        pool.close()


def test_pool_is_closed_to_admissions_and_releases_inside_an_open_step_and_a_step_can_be_abandoned():
    import torch
    rng = np.random.default_rng(5)
    prompts = [(_bits(rng, L, n, HKV, D), _bits(rng, L, n, HKV, D), n) for n in (31, 20, 47)]
    q, k, v = _bits(rng, L, 3, HQ, D), _bits(rng, L, 3, HKV, D), _bits(rng, L, 3, HKV, D)

    def fresh():
        p = _pool(host_staging=True, tau=-1.0)
        for kt, vt, n in prompts:
            assert p.request_add(-1, 0, kt, vt, n, 0)[0] == B.GP_OK
        return p

    ids = torch.arange(3, dtype=torch.int32, device="cuda")
    qd, kd, vd = _dev(torch, q), _dev(torch, k), _dev(torch, v)
    results = []
    for disturb in (False, True):
        pool = fresh()
        try:
            out = torch.zeros((L, 3, HQ, D), dtype=torch.float32, device="cuda")
            act = torch.zeros(3, dtype=torch.int32, device="cuda")
            s = pool.stream()
            if disturb:
                free0 = _invariants(pool, [0, 1, 2])
                B.gp_step_begin(pool.handle, ids.data_ptr(), 3, act.data_ptr(), s)
                B.gp_attn_layer(pool.handle, 1, ids.data_ptr(), 3, qd[1].data_ptr(), kd[1].data_ptr(), vd[1].data_ptr(),
                                out[1].data_ptr(), s)
                # nothing that touches the free list or the slots may pass while the step is open
                with pytest.raises(B.GpError) as e:
                    pool.release(1)
                assert e.value.status == B.GP_ERR_STATE
                assert pool.request_add(-1, 0, prompts[0][0], prompts[0][1], 31, 0)[0] == B.GP_ERR_STATE
                with pytest.raises(B.GpError) as e:
                    pool.decode_step(ids, qd, kd, vd, out, act)
                assert e.value.status == B.GP_ERR_STATE
                ph = lambda t: t.cpu().pin_memory()
                with pytest.raises(B.GpError) as e:
                    pool.decode_step_host(ph(ids), ph(qd), ph(kd), ph(vd), ph(out), ph(act))
                assert e.value.status == B.GP_ERR_STATE
                with pytest.raises(B.GpError) as e:              # the same layer twice
                    B.gp_attn_layer(pool.handle, 1, ids.data_ptr(), 3, qd[1].data_ptr(), kd[1].data_ptr(),
                                    vd[1].data_ptr(), out[1].data_ptr(), s)
                assert e.value.status == B.GP_ERR_STATE
                with pytest.raises(B.GpError) as e:              # a layer is missing
                    B.gp_step_end(pool.handle, ids.data_ptr(), 3, act.data_ptr(), s)
                assert e.value.status == B.GP_ERR_STATE
                B.gp_step_abort(pool.handle)
                with pytest.raises(B.GpError) as e:
                    B.gp_step_abort(pool.handle)
                assert e.value.status == B.GP_ERR_STATE
                assert _invariants(pool, [0, 1, 2]) == free0
                assert [B.gp_debug_request(pool.handle, r, 6)[1] for r in range(3)] == [31, 20, 47]
                out.zero_()
            # the abandoned step left nothing behind: the same step now gives what an undisturbed pool gives
            pool.decode_step(ids, qd, kd, vd, out, act)
            torch.cuda.synchronize()
            summ = [B.gp_debug_summaries(pool.handle, r, L, HQ, D) for r in range(3)]
            results.append((out.cpu().numpy(), act.cpu().numpy(), summ, _invariants(pool, [0, 1, 2])))
            assert B.gp_pool_status(pool.handle) == (B.GP_OK, 0)
        finally:
            pool.close()
    (o1, a1, s1, f1), (o2, a2, s2, f2) = results
    assert np.array_equal(o1, o2) and np.array_equal(a1, a2) and f1 == f2
    assert all(np.array_equal(x, y) for x, y in zip(s1, s2))
    assert a1.tolist() == [B.GP_ACT_GROW, B.GP_ACT_NONE, B.GP_ACT_GROW]      # 32 and 48 tokens fill two and three pages


# ----------------------------------------------------------------------------------------------------------------
# bounded waits that run out: the kernel gives up, says so, and ends; nothing hangs, nothing faults
# ----------------------------------------------------------------------------------------------------------------
def _accounting_intact(pool, n_pages, live, cap):
    n_free, ref, _ = B.gp_debug_pool(pool.handle, n_pages)
    held = 0
    for r in live:
        P, n, pos, table = B.gp_debug_request(pool.handle, r, cap)
        assert len(set(table)) == P and 0 < n <= P * 16
        held += P
    assert int((ref > 0).sum()) + n_free == n_pages and int(ref.sum()) == held


def _one_step(pool, torch, rng, n_req, hq, hkv, d, host=False):
    q, k, v = _bits(rng, 1, n_req, hq, d), _bits(rng, 1, n_req, hkv, d), _bits(rng, 1, n_req, hkv, d)
    out = torch.zeros((1, n_req, hq, d), dtype=torch.float32, device="cuda")
    act = torch.zeros(n_req, dtype=torch.int32, device="cuda")
    ids = torch.arange(n_req, dtype=torch.int32, device="cuda")
    if host:
        ph = lambda t: t.cpu().pin_memory()
        args = [ph(ids), ph(_dev(torch, q)), ph(_dev(torch, k)), ph(_dev(torch, v)), ph(out), ph(act)]
        pool.decode_step_host(*args)
        return args[4].numpy().copy(), args[5].numpy().copy()
    pool.decode_step(ids, _dev(torch, q), _dev(torch, k), _dev(torch, v), out, act)
    torch.cuda.synchronize()
    return out.cpu().numpy(), act.cpu().numpy()


def test_attention_wait_that_runs_out_is_reported_and_the_kernel_drains():
    import torch
    # 80 requests x 8 heads = 640 work items on 296 thread blocks: the first block has a second item, which the test
    # withholds from its consumer warps; their wait gives up after 3000 tries
    n_req, hq, hkv, d, cap = 80, 8, 8, 64, 4
    cfg = B.make_config(1, hq, hkv, d, n_pages=n_req * cap, max_pages_per_req=cap, max_requests=n_req, host_staging=True)
    results = []
    for withhold in (0, 1):
        rng = np.random.default_rng(11)
        pool = B.Pool(cfg)
        try:
            for _ in range(n_req):
                assert pool.request_add(-1, 0, _bits(rng, 1, 20, hkv, d), _bits(rng, 1, 20, hkv, d), 20, 0)[0] == B.GP_OK
            B.gp_test_withhold(pool.handle, withhold, 3000)
            if withhold:
                with pytest.raises(B.GpError) as e:              # the host entry point looks at the error word itself
                    _one_step(pool, torch, rng, n_req, hq, hkv, d, host=True)
                assert e.value.status == B.GP_ERR_CUDA
                st, bits = B.gp_pool_status(pool.handle)
                assert st == B.GP_ERR_CUDA and (bits & 1) and (bits >> 7), bits      # a wait gave up, and which one
                _accounting_intact(pool, n_req * cap, range(n_req), cap)
                assert B.gp_debug_pool(pool.handle)[2][7] == bits
            else:
                results.append(_one_step(pool, torch, rng, n_req, hq, hkv, d, host=True))
                assert B.gp_pool_status(pool.handle) == (B.GP_OK, 0)
        finally:
            pool.close()
    # the device is as usable as before: an ordinary pool gives the ordinary result
    rng = np.random.default_rng(11)
    pool = B.Pool(cfg)
    try:
        for _ in range(n_req):
            pool.request_add(-1, 0, _bits(rng, 1, 20, hkv, d), _bits(rng, 1, 20, hkv, d), 20, 0)
        out, act = _one_step(pool, torch, rng, n_req, hq, hkv, d, host=True)
        diff = np.abs(out - results[0][0])
        assert np.array_equal(act, results[0][1]) and diff.max() == 0.0, (float(diff.max()), np.argwhere(diff > 0)[:4].tolist(), int((diff > 0).sum()))
    finally:
        pool.close()


@pytest.mark.parametrize("async_boundary,what,bit", [(False, 2, 8), (True, 2, 8), (True, 4, 8), (False, 4, 8), (False, 8, 16)])
def test_compaction_and_decision_waits_that_run_out_are_reported(async_boundary, what, bit):
    import torch
    # one request of eight pages that fills its last slot with the first step and compresses: two chunks per unit
    n_req, hq, hkv, d, cap = 3, 8, 2, 64, 9
    cfg = B.make_config(1, hq, hkv, d, n_pages=n_req * cap, max_pages_per_req=cap, max_requests=4, async_boundary=async_boundary)
    rng = np.random.default_rng(13)
    pool = B.Pool(cfg)
    try:
        for _ in range(n_req):
            assert pool.request_add(-1, 0, _bits(rng, 1, 127, hkv, d), _bits(rng, 1, 127, hkv, d), 127, 0)[0] == B.GP_OK
        B.gp_test_withhold(pool.handle, what, 2000)
        out, act = _one_step(pool, torch, rng, n_req, hq, hkv, d)
        assert act.tolist() == [B.GP_ACT_PENDING if async_boundary else B.GP_ACT_COMPRESS] * n_req
        B.gp_async_join(pool.handle, pool.stream())
        torch.cuda.synchronize()
        st, bits = B.gp_pool_status(pool.handle)
        assert st == B.GP_ERR_CUDA and (bits & bit), bits
        _accounting_intact(pool, n_req * cap, range(n_req), cap)
        assert [B.gp_debug_request(pool.handle, r, cap)[:2] for r in range(n_req)] == [(8, 112)] * n_req
        B.gp_test_withhold(pool.handle, 0, 0)
        out, act = _one_step(pool, torch, rng, n_req, hq, hkv, d)        # the pool still steps
        assert np.isfinite(out).all() and act.tolist() == [B.GP_ACT_HELD if async_boundary else B.GP_ACT_NONE] * n_req
    finally:
        pool.close()
