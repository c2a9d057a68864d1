"""The allocation-free attention entry point against the pool's own decode step and against the float64 oracle.

Some callers cannot give the library scratch memory or let it allocate (all device memory is committed to
the KV pool, or the host forbids allocator calls from plug-ins); `gp_attention_noalloc` serves them from a
fixed array inside the library.  This test feeds it the same keys and values the pool holds after a decode
step and expects the same attention output, on two consecutive calls (the array keeps the first call's
contents, which must not leak into the second), and compares it with the oracle's dense attention on
requests of ragged lengths, one of them empty.  It is collected last on purpose."""
import numpy as np
import pytest

from oracle import growpage_oracle as O
from paper_2609_03494_b200 import binding as B
from paper_2609_03494_b200 import workload as W

pytestmark = pytest.mark.gpu

ATTN_MAX_ABS = 1e-2      # same bound as the other attention parity tests
ATTN_MEAN_ABS = 1e-3


@pytest.mark.parametrize("hq,hkv,d,prompts", [(8, 2, 64, (37, 130, 300)), (32, 8, 128, (513, 16, 95, 1))])
def test_noalloc_attention_matches_the_pool_on_two_calls(hq, hkv, d, prompts):
    import torch
    rng = np.random.default_rng(7)
    n_req = len(prompts)
    cap = max(prompts) // 16 + 3
    cfg = B.make_config(1, hq, hkv, d, n_pages=n_req * cap, max_pages_per_req=cap, max_requests=8, tau=-1.0)
    pool = B.Pool(cfg)
    bits = lambda *shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()
    try:
        for n in prompts:
            st, _ = pool.request_add(-1, 0, bits(1, n, hkv, d), bits(1, n, hkv, d), n, 0)
            assert st == B.GP_OK
        ids = torch.arange(n_req, dtype=torch.int32, device="cuda")
        max_len = max(prompts) + 2
        for step in range(2):
            q, k, v = bits(1, n_req, hq, d), bits(1, n_req, hkv, d), bits(1, n_req, hkv, d)
            out = torch.zeros((1, n_req, hq, d), dtype=torch.float32, device="cuda")
            act = torch.zeros(n_req, dtype=torch.int32, device="cuda")
            qd = dev(q)
            pool.decode_step(ids, qd, dev(k), dev(v), out, act)
            # the pool's keys and values after the step (the new token included), as plain dense tensors
            K = np.zeros((n_req, hkv, max_len, d), dtype=np.uint16)
            V = np.zeros((n_req, hkv, max_len, d), dtype=np.uint16)
            lens = np.zeros(n_req, dtype=np.int32)
            for r in range(n_req):
                _, n, _, _ = B.gp_debug_request(pool.handle, r, cap)
                lens[r] = n
                for h in range(hkv):
                    K[r, h, :n], V[r, h, :n] = B.gp_debug_kv(pool.handle, r, 0, h, n, d)
            assert lens.tolist() == [p + step + 1 for p in prompts]
            out2 = torch.full((n_req, hq, d), float("nan"), dtype=torch.float32, device="cuda")
            Kd, Vd, lens_d = dev(K), dev(V), torch.from_numpy(lens).cuda()      # the caller owns every buffer
            B.gp_attention_noalloc(qd.data_ptr(), Kd.data_ptr(), Vd.data_ptr(), lens_d.data_ptr(), n_req, hq, hkv, d,
                                   max_len, out2.data_ptr(), pool.stream())
            torch.cuda.synchronize()
            err = (out2 - out[0]).abs()
            assert float(err.max()) <= ATTN_MAX_ABS and float(err.mean()) <= ATTN_MEAN_ABS, (step, float(err.max()))
    finally:
        pool.close()


@pytest.mark.parametrize("hq,hkv,d,lens", [(8, 2, 64, (37, 0, 300, 1)), (32, 8, 128, (513, 16, 0, 95)), (16, 2, 128, (129,))])
def test_noalloc_attention_matches_the_oracle_and_an_empty_request_gives_zeros(hq, hkv, d, lens):
    import torch
    rng = np.random.default_rng(19)
    n_req, max_len = len(lens), max(lens) + 5
    bits = lambda *shape: W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    q, K, V = bits(n_req, hq, d), bits(n_req, hkv, max_len, d), bits(n_req, hkv, max_len, d)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()
    qd, Kd, Vd = dev(q), dev(K), dev(V)
    lens_d = torch.tensor(lens, dtype=torch.int32, device="cuda")
    f = W.bf16_bits_to_f64
    for call in range(2):                                    # the second call finds the first one's partials in the array
        out = torch.full((n_req, hq, d), float("nan"), dtype=torch.float32, device="cuda")
        B.gp_attention_noalloc(qd.data_ptr(), Kd.data_ptr(), Vd.data_ptr(), lens_d.data_ptr(), n_req, hq, hkv, d,
                               max_len, out.data_ptr(), 0)
        torch.cuda.synchronize()
        got = out.cpu().numpy().astype(np.float64)
        for r, n in enumerate(lens):
            if n == 0:
                assert np.array_equal(got[r], np.zeros((hq, d))), "an empty request must give a row of zeros"
                continue
            want = O.attention_decode(f(q[r]), f(K[r, :, :n]), f(V[r, :, :n]))
            err = np.abs(got[r] - want)
            assert err.max() <= ATTN_MAX_ABS and err.mean() <= ATTN_MEAN_ABS, (call, r, err.max())


def test_noalloc_rejects_what_does_not_fit():
    import torch
    z = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.GpError) as e:
        B.gp_attention_noalloc(z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(), 128, 32, 8, 128, 4, z.data_ptr(), 0)
    assert e.value.status == B.GP_ERR_TOO_LARGE and "fixed scratch" in str(e.value)
    with pytest.raises(B.GpError) as e:
        B.gp_attention_noalloc(z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(), 1, 8, 2, 96, 4, z.data_ptr(), 0)
    assert e.value.status == B.GP_ERR_INVALID
