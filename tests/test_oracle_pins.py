"""Pins of the CPU oracle against things it did not compute itself: closed forms, library
routines, brute force over all subsets, and invariants the paper states.  A dropped term, a wrong
sign or index, or a transposed operand in the oracle fails at least one of these."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import growpage_oracle as O

RNG = np.random.default_rng(1234)


# ----------------------------------------------------------------------------- defaults
def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_defaults.txt")
    vals = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            key, val = line.split("=")
            vals[key.strip()] = float(val)
    return vals


def test_defaults_match_the_paper():
    g = _golden()
    c = O.OracleConfig(1, 8, 2, 64, n_pages=8, max_pages_per_req=4)
    assert c.beta_s == g["beta_S"] and c.beta_l == g["beta_L"]
    assert c.top_p == g["p"] and c.tau == g["tau"]
    assert c.max_requests == g["M"]
    # quota is the paper's fraction of a block: 64 of 256 tokens
    assert c.k_loc / c.page_size == g["k_loc"] / g["b"]
    # the ablation's policies
    assert c.p_compress == g["p_compress"] and c.shrink_below == g["shrink_below"] and c.min_capacity == g["min_capacity"]


# ----------------------------------------------------------------------------- attention
def test_attention_single_token_returns_its_value():
    q = RNG.standard_normal((8, 64))
    K = RNG.standard_normal((2, 1, 64))
    V = RNG.standard_normal((2, 1, 64))
    out = O.attention_decode(q, K, V)
    for g in range(8):
        np.testing.assert_allclose(out[g], V[g // 4, 0], rtol=0, atol=1e-15)


def test_attention_equal_keys_average_the_values():
    q = RNG.standard_normal((4, 32))
    K = np.repeat(RNG.standard_normal((2, 1, 32)), 7, axis=1)
    V = RNG.standard_normal((2, 7, 32))
    out = O.attention_decode(q, K, V)
    for g in range(4):
        np.testing.assert_allclose(out[g], V[g // 2].mean(axis=0), atol=1e-14)


def test_attention_two_tokens_is_a_logistic_mix():
    d = 16
    q = RNG.standard_normal((1, d))
    K = RNG.standard_normal((1, 2, d))
    V = RNG.standard_normal((1, 2, d))
    gap = (K[0, 0] - K[0, 1]) @ q[0] / math.sqrt(d)
    w0 = 1.0 / (1.0 + math.exp(-gap))
    np.testing.assert_allclose(O.attention_decode(q, K, V)[0], w0 * V[0, 0] + (1 - w0) * V[0, 1], atol=1e-14)


def test_attention_is_permutation_invariant_and_matches_torch_sdpa():
    torch = pytest.importorskip("torch")
    h_q, h_kv, n, d = 8, 2, 37, 64
    q = RNG.standard_normal((h_q, d))
    K = RNG.standard_normal((h_kv, n, d))
    V = RNG.standard_normal((h_kv, n, d))
    out = O.attention_decode(q, K, V)
    perm = RNG.permutation(n)
    np.testing.assert_allclose(O.attention_decode(q, K[:, perm], V[:, perm]), out, atol=1e-13)
    G = h_q // h_kv
    tq = torch.from_numpy(q)[None, :, None, :]
    tk = torch.from_numpy(K).repeat_interleave(G, dim=0)[None]
    tv = torch.from_numpy(V).repeat_interleave(G, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0, :, 0].numpy()
    np.testing.assert_allclose(out, ref, atol=1e-12)


# ----------------------------------------------------------------------------- Eq. 6
def test_ema_closed_form_and_special_cases():
    T, d = 40, 8
    qs = RNG.standard_normal((T, 1, d))
    bs, bl = 0.9, 0.999
    S = L = np.zeros((1, d))
    started = False
    for t in range(T):
        S, L = O.ema_update(S, L, qs[t], started, bs, bl)
        started = True
        if t == 0:                      # first decode step of a slot: both states are the query
            assert np.array_equal(S, qs[0]) and np.array_equal(L, qs[0])
    for beta, got in ((bs, S), (bl, L)):
        want = beta ** (T - 1) * qs[0]
        for j in range(1, T):
            want = want + (1 - beta) * beta ** (T - 1 - j) * qs[j]
        np.testing.assert_allclose(got, want, rtol=1e-12)
    # a constant query is a fixed point
    c = RNG.standard_normal((1, d))
    S = L = np.zeros((1, d)); started = False
    for _ in range(10):
        S, L = O.ema_update(S, L, c, started, bs, bl); started = True
    np.testing.assert_allclose(S, c, rtol=1e-14); np.testing.assert_allclose(L, c, rtol=1e-14)
    # beta_S = 0: the short summary is the current query (the paper's beta ablation)
    S, L = O.ema_update(RNG.standard_normal((1, d)), RNG.standard_normal((1, d)), c, True, 0.0, bl)
    assert np.array_equal(S, c)


def test_stale_slot_contents_do_not_leak_into_a_new_request():
    stale = 1e6 * np.ones((2, 4))
    q = RNG.standard_normal((2, 4))
    S, L = O.ema_update(stale, stale, q, False, 0.9, 0.999)
    assert np.array_equal(S, q) and np.array_equal(L, q)


# ----------------------------------------------------------------------------- Eq. 12, RoPE
def test_rms_calibration_identities():
    q = RNG.standard_normal((6, 32))
    qb = RNG.standard_normal((6, 32)) * RNG.uniform(0.01, 30, (6, 1))
    qt = O.rms_calibrate(qb, q)
    np.testing.assert_allclose(O.rms(qt), O.rms(q), rtol=1e-13)            # scales are matched
    cos = np.sum(qt * qb, -1) / np.linalg.norm(qt, axis=-1) / np.linalg.norm(qb, axis=-1)
    np.testing.assert_allclose(cos, 1.0, rtol=1e-13)                       # direction is kept
    np.testing.assert_allclose(O.rms_calibrate(3.7 * q, q), q, rtol=1e-13)  # collinear: the query itself
    z = np.zeros((1, 8))
    assert np.array_equal(O.rms_calibrate(z, RNG.standard_normal((1, 8))), z)
    x = np.array([[3.0, 4.0]])
    assert O.rms(x)[0] == pytest.approx(math.sqrt(12.5))


def test_rope_is_a_position_dependent_rotation():
    d, theta = 16, 10000.0
    x = RNG.standard_normal((3, d)); y = RNG.standard_normal((3, d))
    assert np.array_equal(O.rope(x, 5, 0.0), x)                            # switched off
    np.testing.assert_allclose(O.rope(x, 0, theta), x, atol=0)             # position 0
    np.testing.assert_allclose(np.linalg.norm(O.rope(x, 123, theta), axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)
    # scores depend on the position difference only
    a = np.sum(O.rope(x, 40, theta) * O.rope(y, 33, theta), -1)
    b_ = np.sum(O.rope(x, 107, theta) * O.rope(y, 100, theta), -1)
    np.testing.assert_allclose(a, b_, rtol=1e-10)
    # d = 2: a plain plane rotation by `pos` radians (frequency theta^0 = 1), counter-clockwise
    v = np.array([[1.0, 0.0]])
    np.testing.assert_allclose(O.rope(v, 1, theta), [[math.cos(1.0), math.sin(1.0)]], atol=1e-15)
    # pairing is (i, i + d/2): rotating a vector that lives in one pair leaves the others zero
    e = np.zeros((1, d)); e[0, 2] = 1.0
    r = O.rope(e, 7, theta)
    assert set(np.nonzero(np.abs(r[0]) > 1e-12)[0]) <= {2, 2 + d // 2}
    ang = 7 * theta ** (-2.0 * 2 / d)
    np.testing.assert_allclose([r[0, 2], r[0, 2 + d // 2]], [math.cos(ang), math.sin(ang)], atol=1e-14)


def test_rope_matches_transformers_rotate_half():
    torch = pytest.importorskip("torch")
    mod = pytest.importorskip("transformers.models.llama.modeling_llama")
    d, theta, pos = 32, 1e6, 77
    x = RNG.standard_normal((4, d))
    inv = 1.0 / (theta ** (torch.arange(0, d, 2, dtype=torch.float64) / d))
    ang = pos * inv
    emb = torch.cat([ang, ang])
    cos, sin = emb.cos()[None, None], emb.sin()[None, None]
    tx = torch.from_numpy(x)[None]
    ref, _ = mod.apply_rotary_pos_emb(tx, tx, cos, sin, unsqueeze_dim=1)
    np.testing.assert_allclose(O.rope(x, pos, theta), ref.reshape(4, d).numpy(), atol=1e-12)


# ----------------------------------------------------------------------------- Eq. 2, Eq. 5, Theorem 1
def test_p_coverage_closed_forms():
    n = 50
    assert O.p_coverage_demand(np.full(n, 1.0 / n), 0.5) == 25
    assert O.p_coverage_demand(np.full(n, 1.0 / n), 0.503) == 26
    one = np.zeros(n); one[17] = 1.0
    assert O.p_coverage_demand(one, 0.99) == 1
    # geometric weights: the top-k mass is 1 - r^k up to the normaliser
    r = 0.8
    a = (1 - r) * r ** np.arange(200)
    a = RNG.permutation(a / a.sum())
    k = O.p_coverage_demand(a, 0.99)
    assert k == math.ceil(math.log(1 - 0.99 * (1 - r ** 200)) / math.log(r))
    # order of the input does not matter; never reached -> everything
    assert O.p_coverage_demand(np.array([0.2, 0.5, 0.3]), 0.75) == 2
    assert O.p_coverage_demand(np.array([0.25, 0.25]), 0.99) == 2


def test_worst_case_error_is_attained_and_theorem_1_by_brute_force():
    for trial in range(20):
        n = int(RNG.integers(4, 12))
        a = RNG.dirichlet(np.full(n, RNG.uniform(0.2, 2.0)))
        v_max = float(RNG.uniform(0.5, 3.0))
        # Eq. 5: the bound is met by opposite directions of norm Vmax on and off S
        S = sorted(RNG.choice(n, size=int(RNG.integers(1, n)), replace=False).tolist())
        u = RNG.standard_normal(5); u /= np.linalg.norm(u)
        v = np.array([(-v_max if i in S else v_max) * u for i in range(n)])
        o = a @ v
        o_hat, m = O.subset_output(a, v, S)
        assert np.linalg.norm(o - o_hat) == pytest.approx(2 * v_max * (1 - m), rel=1e-10)
        assert O.worst_case_error(a, S, v_max) == pytest.approx(2 * v_max * (1 - m), rel=1e-12)
        # random values never exceed it
        w = RNG.standard_normal((n, 5)); w *= v_max / np.linalg.norm(w, axis=1, keepdims=True)
        o_hat2, _ = O.subset_output(a, w, S)
        assert np.linalg.norm(a @ w - o_hat2) <= 2 * v_max * (1 - m) + 1e-12
        # Theorem 1: min |S| with worst-case error <= delta equals D_{1 - delta / (2 Vmax)}
        delta = float(RNG.uniform(0.05, 1.9)) * v_max
        best = None
        for size in range(1, n + 1):
            if any(O.worst_case_error(a, comb, v_max) <= delta for comb in itertools.combinations(range(n), size)):
                best = size
                break
        assert best == O.p_coverage_demand(a, 1 - delta / (2 * v_max))


def test_summary_attention_is_the_group_mean_of_softmaxes():
    sp = pytest.importorskip("scipy.special")
    G, n, d = 4, 33, 16
    qt = RNG.standard_normal((G, d)); Kc = RNG.standard_normal((n, d))
    a = O.summary_attention(qt, Kc)
    assert a.sum() == pytest.approx(1.0, abs=1e-14)
    ref = np.mean([sp.softmax(Kc @ qt[g] / math.sqrt(d)) for g in range(G)], axis=0)
    np.testing.assert_allclose(a, ref, rtol=1e-12)
    # a calibrated summary collinear with the query reproduces the query's own attention over C
    q = RNG.standard_normal((1, d))
    np.testing.assert_allclose(O.summary_attention(O.rms_calibrate(0.2 * q, q), Kc),
                               sp.softmax(Kc @ q[0] / math.sqrt(d)), rtol=1e-12)


# ----------------------------------------------------------------------------- Eq. 9, Eq. 10
def test_token_score_is_the_larger_view():
    a = RNG.random(9); c = RNG.random(9)
    s = O.token_scores(a, c)
    assert np.all(s >= a) and np.all(s >= c) and np.all((s == a) | (s == c))


def _best_subset(s, n_blocks, b, K_t, k_prime):
    best, best_val = None, -1.0
    for comb in itertools.combinations(range(n_blocks * b), K_t):
        cnt = np.bincount(np.asarray(comb) // b, minlength=n_blocks)
        if np.all(cnt >= k_prime):
            val = s[list(comb)].sum()
            if val > best_val:
                best, best_val = comb, val
    return np.asarray(best)


@pytest.mark.parametrize("n_blocks,b,k_loc", [(3, 4, 1), (3, 4, 2), (4, 3, 1), (2, 6, 2), (3, 4, 0)])
def test_selection_is_the_constrained_optimum(n_blocks, b, k_loc):
    for _ in range(6):
        s = RNG.random(n_blocks * b) ** 3
        K_t = n_blocks * b - b
        keep, _ = O.select_retained(s, n_blocks, b, K_t, k_loc)
        assert keep.size == K_t and np.all(np.diff(keep) > 0)
        k_prime = min(k_loc, K_t // n_blocks)
        np.testing.assert_array_equal(keep, _best_subset(s, n_blocks, b, K_t, k_prime))
        if n_blocks >= 3:                                        # the Shrink target of Eq. 13: two pages go
            K_t = n_blocks * b - 2 * b
            keep, _ = O.select_retained(s, n_blocks, b, K_t, k_loc)
            np.testing.assert_array_equal(keep, _best_subset(s, n_blocks, b, K_t, min(k_loc, K_t // n_blocks)))


def test_selection_special_cases_and_ties():
    b, n_blocks = 16, 5
    s = RNG.random(n_blocks * b)
    K_t = (n_blocks - 1) * b
    keep, _ = O.select_retained(s, n_blocks, b, K_t, 0)          # no quota: plain top-K_t
    np.testing.assert_array_equal(keep, np.sort(np.argpartition(-s, K_t - 1)[:K_t]))
    # quota large enough that the local picks fill the budget: floor(K_t / n_blocks) from each block
    keep, _ = O.select_retained(s[:16], 4, 4, 12, 3)
    assert np.all(np.bincount(keep // 4, minlength=4) == 3)
    # exact duplicates: the older (lower) slot wins, in the local and in the global cut
    s = np.array([0.5, 0.5, 0.5, 0.5, 0.1, 0.1, 0.1, 0.1])
    keep, margin = O.select_retained(s, 2, 4, 4, 1)
    np.testing.assert_array_equal(keep, [0, 1, 2, 4])
    assert margin == 0.0
    # block quota overrides global rank: the worst block still keeps its best k'
    s = np.concatenate([np.full(4, 0.9), np.full(4, 0.8), np.array([0.01, 0.04, 0.02, 0.03])])
    keep, _ = O.select_retained(s, 3, 4, 8, 1)
    assert 9 in keep and np.bincount(keep // 4, minlength=3).tolist() == [4, 3, 1]


# ----------------------------------------------------------------------------- state machine
def _cfg(**kw):
    base = dict(n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=8, n_pages=12, max_pages_per_req=6, page_size=4,
                recent_window=4, k_loc=1, max_requests=4)
    base.update(kw)
    return O.OracleConfig(**base)


def _rand_step(c, B):
    return (RNG.standard_normal((c.n_layers, B, c.n_q_heads, c.head_dim)),
            RNG.standard_normal((c.n_layers, B, c.n_kv_heads, c.head_dim)),
            RNG.standard_normal((c.n_layers, B, c.n_kv_heads, c.head_dim)))


def _check_invariants(pool: O.OraclePool):
    c = pool.cfg
    b = c.page_size
    refs = np.zeros(c.n_pages, dtype=np.int64)
    for rid, r in pool.requests.items():
        assert len(r.table) == r.P and r.n <= r.P * b
        for page in r.table:
            refs[page] += 1
        for l in range(c.n_layers):
            for h in range(c.n_kv_heads):
                tok = r.tok[l, h, :r.n]
                assert np.all(np.diff(tok) > 0)                       # slot order is token order
                assert np.all(tok[-min(r.n, 1):] == r.pos - 1) or r.n == 0 or not r.started
                assert np.all(r.tok[l, h, r.n:r.P * b] == -1) or not r.started
    assert np.array_equal(refs, pool.refcount)                        # references are conserved
    assert len(set(pool.free)) == len(pool.free)
    assert len(pool.free) + int((pool.refcount > 0).sum()) == c.n_pages
    assert all(pool.refcount[p] == 0 for p in pool.free)


def test_capacity_moves_only_at_boundaries_and_only_up_by_one():
    c = _cfg()
    pool = O.OraclePool(c)
    kt = RNG.standard_normal((c.n_layers, 6, c.n_kv_heads, c.head_dim))
    st, rid = pool.request_add(-1, 0, kt, kt.copy(), 6, 2)
    assert st == O.OK and rid == 0
    P, n, pos, table = pool.request_state(rid)
    assert (P, n, pos) == (2, 6, 6)                                   # floor(6/4)+1 = 2 pages
    seen = set()
    for step in range(60):
        q, k, v = _rand_step(c, 1)
        P0, n0, _, _ = pool.request_state(rid)
        rec = pool.decode_step([rid], q, k, v)
        P1, n1, pos1, _ = pool.request_state(rid)
        act = int(rec.actions[0]); seen.add(act)
        assert pos1 == 7 + step
        if n0 + 1 < P0 * c.page_size:
            assert act == O.ACT_NONE and P1 == P0 and n1 == n0 + 1
        elif act == O.ACT_GROW:
            assert P1 == P0 + 1 and n1 == n0 + 1
        else:
            assert act in (O.ACT_COMPRESS, O.ACT_COMPRESS_FALLBACK)
            assert P1 == P0 and n1 == (P0 - 1) * c.page_size          # exactly one page of slots freed
            info = rec.boundary[rid]
            for l in range(c.n_layers):
                for h in range(c.n_kv_heads):
                    tok = pool.retained(rid, l, h)
                    assert np.array_equal(tok[-c.page_size:], np.arange(pos1 - c.page_size, pos1))  # newest survive
                    assert info.keep[(l, h)].size == (P0 - 2) * c.page_size
        assert P1 <= c.max_pages_per_req
        _check_invariants(pool)
    assert O.ACT_COMPRESS in seen or O.ACT_COMPRESS_FALLBACK in seen


def test_first_boundary_with_equal_summaries_compresses():
    # one free slot at admission: the first decode step is a boundary with S == L, so Delta = 0
    c = _cfg()
    pool = O.OraclePool(c)
    kt = RNG.standard_normal((c.n_layers, 7, c.n_kv_heads, c.head_dim))
    _, rid = pool.request_add(-1, 0, kt, kt.copy(), 7, 0)
    q, k, v = _rand_step(c, 1)
    rec = pool.decode_step([rid], q, k, v)
    info = rec.boundary[rid]
    assert info.delta == 0.0 and np.array_equal(info.K_s, info.K_l)
    assert int(rec.actions[0]) == O.ACT_COMPRESS
    # and the attention output of that step saw all 8 tokens (append precedes attention)
    r = pool.requests[rid]
    assert r.n == 4


def test_grow_fallback_and_stall_under_a_small_pool():
    c = _cfg(n_pages=3, max_pages_per_req=3)
    pool = O.OraclePool(c)
    kt = RNG.standard_normal((c.n_layers, 3, c.n_kv_heads, c.head_dim))
    _, a = pool.request_add(-1, 0, kt, kt.copy(), 3, 0)              # P = 1
    q, k, v = _rand_step(c, 1)
    rec = pool.decode_step([a], q, k, v)                              # n = 4 = P b, C empty -> grow
    assert int(rec.actions[0]) == O.ACT_GROW and pool.request_state(a)[0] == 2
    st, b_id = pool.request_add(-1, 0, kt, kt.copy(), 3, 0)
    assert st == O.OK and pool.n_free() == 0
    rec = pool.decode_step([b_id], *_rand_step(c, 1))                 # P = 1, no page: nothing to evict
    assert int(rec.actions[0]) == O.ACT_STALLED
    rec = pool.decode_step([b_id], *_rand_step(c, 1))                 # stays stalled, untouched
    assert int(rec.actions[0]) == O.ACT_STALLED and pool.request_state(b_id)[1] == 4
    assert pool.request_add(-1, 0, kt, kt.copy(), 3, 0)[0] == O.ERR_NO_PAGES
    # force "wants to grow" on a full pool: falls back to compression
    for _ in range(3):
        pool.decode_step([a], *_rand_step(c, 1))
    rec = pool.step_compute([a], *_rand_step(c, 1))
    pool.step_apply(rec, {a: {"want_grow": True}})
    assert int(rec.actions[0]) == O.ACT_COMPRESS_FALLBACK
    assert pool.release(b_id) == O.OK and pool.n_free() == 1
    _check_invariants(pool)


def test_prefix_sharing_copy_on_write_and_release():
    c = _cfg(n_pages=16, max_pages_per_req=5)
    pool = O.OraclePool(c)
    kt = RNG.standard_normal((c.n_layers, 8, c.n_kv_heads, c.head_dim))   # two full pages
    _, a = pool.request_add(-1, 0, kt, kt.copy(), 8, 0)                   # P = 3
    _, b_id = pool.request_add(a, 2, None, None, 0, 0)
    _, c_id = pool.request_add(a, 2, None, None, 0, 0)
    shared = pool.request_state(a)[3][:2]
    assert pool.request_state(b_id)[3][:2] == shared and all(pool.refcount[p] == 3 for p in shared)
    assert pool.request_add(a, 3, None, None, 0, 0)[0] == O.ERR_INVALID   # page 2 is not a full prompt page
    snapshot = pool.requests[b_id].K[:, :, :8].copy()
    free0 = pool.n_free()
    # run a and b to their first boundary together, forcing compression for both
    for step in range(4):
        rec = pool.step_compute([a, b_id], *_rand_step(c, 2))
        pool.step_apply(rec, {a: {"want_grow": False}, b_id: {"want_grow": False}})
        _check_invariants(pool)
    assert [int(x) for x in rec.actions] == [O.ACT_COMPRESS, O.ACT_COMPRESS]
    assert rec.boundary[a].cow_pages == 2 and rec.boundary[b_id].cow_pages == 2
    # both replaced both shared pages; the third sharer still holds them, untouched
    assert all(pool.refcount[p] == 1 for p in shared)
    assert pool.request_state(c_id)[3][:2] == shared
    assert not set(pool.request_state(a)[3]) & set(pool.request_state(b_id)[3])
    assert pool.n_free() == free0 - 4
    np.testing.assert_array_equal(pool.requests[c_id].K[:, :, :8], snapshot)
    assert pool.request_add(a, 1, None, None, 0, 0)[0] == O.ERR_INVALID   # a's prefix is no longer pristine
    # last sharer compresses alone: it is the only owner now and keeps its pages
    for step in range(4):
        rec = pool.step_compute([c_id], *_rand_step(c, 1))
        pool.step_apply(rec, {c_id: {"want_grow": False}})
    assert rec.boundary[c_id].cow_pages == 0 and pool.request_state(c_id)[3][:2] == shared
    for rid in (a, b_id, c_id):
        assert pool.release(rid) == O.OK
    assert pool.n_free() == c.n_pages and not pool.refcount.any()


def test_simultaneous_last_sharers_both_copy_and_the_page_is_freed_afterwards():
    c = _cfg(n_pages=10, max_pages_per_req=4)
    pool = O.OraclePool(c)
    kt = RNG.standard_normal((c.n_layers, 4, c.n_kv_heads, c.head_dim))
    _, a = pool.request_add(-1, 0, kt, kt.copy(), 4, 3)                   # P = 3 (budget above the prompt)
    _, b_id = pool.request_add(a, 1, None, None, 0, 3)
    page = pool.request_state(a)[3][0]
    for step in range(8):
        rec = pool.step_compute([a, b_id], *_rand_step(c, 2))
        pool.step_apply(rec, {a: {"want_grow": False}, b_id: {"want_grow": False}})
    assert pool.refcount[page] == 0 and page in pool.free
    _check_invariants(pool)


def test_stall_when_copy_on_write_targets_are_missing_leaves_the_request_unchanged():
    c = _cfg(n_pages=5, max_pages_per_req=3)
    pool = O.OraclePool(c)
    kt = RNG.standard_normal((c.n_layers, 8, c.n_kv_heads, c.head_dim))
    _, a = pool.request_add(-1, 0, kt, kt.copy(), 8, 0)                   # 3 pages
    _, b_id = pool.request_add(a, 2, None, None, 0, 0)                    # 1 private page; pool: 1 free
    for step in range(4):
        before = pool.request_state(b_id)
        rec = pool.step_compute([b_id], *_rand_step(c, 1))
        pool.step_apply(rec, {b_id: {"want_grow": False}})
    assert int(rec.actions[0]) == O.ACT_STALLED                       # needs 2 targets, 1 free
    P, n, pos, table = pool.request_state(b_id)
    assert n == P * c.page_size and table == before[3]
    _check_invariants(pool)


def test_invalid_ids_and_duplicates_are_reported_per_request():
    c = _cfg()
    pool = O.OraclePool(c)
    kt = RNG.standard_normal((c.n_layers, 2, c.n_kv_heads, c.head_dim))
    _, a = pool.request_add(-1, 0, kt, kt.copy(), 2, 0)
    rec = pool.decode_step([a, 3, a], *_rand_step(c, 3))
    assert [int(x) for x in rec.actions] == [O.ACT_NONE, O.ACT_INVALID, O.ACT_INVALID]
    assert pool.request_state(a)[1] == 3
    # the same at a capacity boundary (page size 4, one page: the fourth token fills it): the action belongs to the
    # first batch slot that names the request, the repeat stays invalid
    rec = pool.decode_step([a, a], *_rand_step(c, 2))
    assert int(rec.actions[0]) in (O.ACT_GROW, O.ACT_COMPRESS_FALLBACK, O.ACT_STALLED) and int(rec.actions[1]) == O.ACT_INVALID
    assert pool.request_state(a)[2] == 4
    assert pool.release(2) == O.ERR_INVALID
    for i in range(3):
        assert pool.request_add(-1, 0, kt, kt.copy(), 2, 0)[0] == O.OK
    assert pool.request_add(-1, 0, kt, kt.copy(), 2, 0)[0] == O.ERR_NO_SLOT


def test_retained_output_error_respects_the_worst_case_bound():
    # after a compression with retained set S, the view's own output error is bounded by Eq. 5
    c = _cfg(n_layers=1, n_q_heads=2, n_kv_heads=2, n_pages=8, max_pages_per_req=4)
    pool = O.OraclePool(c)
    kt = RNG.standard_normal((1, 11, 2, 8))
    _, a = pool.request_add(-1, 0, kt, RNG.standard_normal((1, 11, 2, 8)), 11, 0)
    r = pool.requests[a]
    rec = pool.step_compute([a], *_rand_step(c, 1))
    V_c = r.V[0, 0, :8].copy()
    pool.step_apply(rec, {a: {"want_grow": False}})
    info = rec.boundary[a]
    S = info.keep[(0, 0)]
    a_s = info.a_s[0, 0]
    o_hat, m = O.subset_output(a_s, V_c, S)
    v_max = np.linalg.norm(V_c, axis=1).max()
    assert np.linalg.norm(a_s @ V_c - o_hat) <= 2 * v_max * (1 - m) + 1e-12


def test_random_policy_draws_are_splitmix64_and_uniform():
    # golden: the first two outputs of SplitMix64 seeded with 0 (published with the generator) are what the
    # draw's mixing function gives for (seed 0, request 0, position 0) and (seed 0, request 1, position 0)
    assert O.random_draw(0, 0, 0) == (0xE220A8397B1DCDAF >> 11) / 2.0 ** 53
    assert O.random_draw(0, 1, 0) == (0x6E789E6AA1B965F4 >> 11) / 2.0 ** 53
    u = np.array([O.random_draw(9, r, p) for r in range(40) for p in range(250)])
    assert 0.0 <= u.min() and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 4 * (1 / 12) ** 0.5 / len(u) ** 0.5
    assert abs((u < 0.7).mean() - 0.7) < 4 * (0.21 / len(u)) ** 0.5
    # position and request both matter
    assert len({O.random_draw(9, 3, p) for p in range(100)}) == 100
    assert len({O.random_draw(9, r, 5) for r in range(100)}) == 100


def test_inverse_and_random_policies_only_change_the_decision():
    # same request, same inputs: the three policies see the same Delta at the first boundary that has history
    # (the one after 16 more steps; the very first has S == L) and turn it into their own action
    outs = {}
    for policy, kw in ((0, {}), (1, {}), (2, dict(p_compress=1.0)), (3, dict(p_compress=0.0))):
        c = _cfg(n_pages=16, max_pages_per_req=8)
        c.policy = min(policy, 2)
        for k_, v_ in kw.items():
            setattr(c, k_, v_)
        pool = O.OraclePool(c)
        g = np.random.default_rng(3)
        kt = g.standard_normal((c.n_layers, 20, c.n_kv_heads, c.head_dim))
        _, rid = pool.request_add(-1, 0, kt, kt.copy(), 20, 0)
        acts, deltas = [], []
        for t in range(12):
            shp_q = (c.n_layers, 1, c.n_q_heads, c.head_dim)
            shp_k = (c.n_layers, 1, c.n_kv_heads, c.head_dim)
            rec = pool.decode_step([rid], g.standard_normal(shp_q), g.standard_normal(shp_k), g.standard_normal(shp_k))
            if rid in rec.boundary:
                acts.append(int(rec.actions[0]))
                deltas.append(rec.boundary[rid].delta)
                break
        outs[policy] = (acts, deltas)
    assert outs[0][1] == outs[1][1] == outs[2][1] == outs[3][1]          # same Delta, whatever the policy
    d = outs[0][1][0]
    assert outs[0][0][0] == (O.ACT_GROW if d > 0 else O.ACT_COMPRESS)
    assert outs[1][0][0] == (O.ACT_COMPRESS if d > 0 else O.ACT_GROW)
    assert outs[2][0][0] == O.ACT_COMPRESS                               # p_compress = 1: always Compress & Hold
    assert outs[3][0][0] == O.ACT_GROW                                   # p_compress = 0: always grows


def test_eq13_regions_of_the_shrink_policy():
    # Eq. 13 with the paper's thresholds: Shrink under -0.005, Compress & Hold on [-0.005, 0], Grow above 0
    assert O.shrink_policy(-0.0051) == O.ACT_SHRINK and O.shrink_policy(-1.0) == O.ACT_SHRINK
    assert O.shrink_policy(-0.005) == O.ACT_COMPRESS          # both ends of the middle interval are closed
    assert O.shrink_policy(-0.001) == O.ACT_COMPRESS and O.shrink_policy(0.0) == O.ACT_COMPRESS
    assert O.shrink_policy(1e-12) == O.ACT_GROW and O.shrink_policy(1.0) == O.ACT_GROW
    assert O.OracleConfig(1, 1, 1, 8, 1, 1).shrink_below == -0.005 and O.OracleConfig(1, 1, 1, 8, 1, 1).min_capacity == 1024


def test_shrink_returns_one_page_evicts_two_and_respects_the_floor():
    c = _cfg(n_pages=16, max_pages_per_req=6)                        # at most 20 candidates: brute force stays small
    c.policy, c.min_capacity, c.shrink_below, c.tau = 3, 12, -0.005, 0.01
    pool = O.OraclePool(c)
    b = c.page_size
    g = np.random.default_rng(11)
    kt = g.standard_normal((c.n_layers, 14, c.n_kv_heads, c.head_dim))
    _, rid = pool.request_add(-1, 0, kt, kt.copy(), 14, 0)
    seen = {}
    for step in range(160):
        shp_q, shp_k = (c.n_layers, 1, c.n_q_heads, c.head_dim), (c.n_layers, 1, c.n_kv_heads, c.head_dim)
        P0, n0, _, _ = pool.request_state(rid)
        free0 = pool.n_free()
        rec = pool.decode_step([rid], g.standard_normal(shp_q), g.standard_normal(shp_k), g.standard_normal(shp_k))
        P1, n1, pos1, _ = pool.request_state(rid)
        act = int(rec.actions[0])
        seen[act] = seen.get(act, 0) + 1
        if rid in rec.boundary:
            info = rec.boundary[rid]
            want = O.shrink_policy(info.delta, c.tau, c.shrink_below)
            if want == O.ACT_SHRINK and (P0 - 1) * b < c.min_capacity:
                want = O.ACT_COMPRESS                                  # the floor: capacity left would be under 12
            if want == O.ACT_GROW and act != O.ACT_GROW:
                assert act == O.ACT_COMPRESS_FALLBACK and (P0 == c.max_pages_per_req or free0 == 0)
            else:
                assert act == want
        if act == O.ACT_SHRINK:
            assert (P1, n1) == (P0 - 1, (P0 - 2) * b) and pool.n_free() == free0 + 1
            assert P1 * b >= c.min_capacity
            for l in range(c.n_layers):
                for h in range(c.n_kv_heads):
                    assert info.keep[(l, h)].size == (P0 - 3) * b
                    s_tok = O.token_scores(info.a_s[l, h], info.a_l[l, h])
                    np.testing.assert_array_equal(
                        info.keep[(l, h)], _best_subset(s_tok, P0 - 1, b, (P0 - 3) * b, min(c.k_loc, ((P0 - 3) * b) // (P0 - 1))))
                    tok = pool.retained(rid, l, h)
                    assert np.array_equal(tok[-b:], np.arange(pos1 - b, pos1))       # the newest page survives
        _check_invariants(pool)
    assert seen.get(O.ACT_SHRINK, 0) > 0 and seen.get(O.ACT_GROW, 0) > 0 and seen.get(O.ACT_COMPRESS, 0) > 0, seen


def test_shrink_with_shared_prompt_pages_copies_before_it_writes():
    c = _cfg(n_pages=40, max_pages_per_req=12)
    c.policy, c.min_capacity, c.shrink_below, c.tau = 3, 8, 0.5, 2.0     # every admissible boundary shrinks
    pool = O.OraclePool(c)
    g = np.random.default_rng(12)
    kt = g.standard_normal((c.n_layers, 24, c.n_kv_heads, c.head_dim))
    _, a = pool.request_add(-1, 0, kt, kt.copy(), 24, 0)
    _, b_ = pool.request_add(a, 6, None, None, 0, 0)
    K_before = pool.requests[b_].K[:, :, :24].copy()
    for step in range(40):
        shp_q, shp_k = (c.n_layers, 1, c.n_q_heads, c.head_dim), (c.n_layers, 1, c.n_kv_heads, c.head_dim)
        rec = pool.decode_step([a], g.standard_normal(shp_q), g.standard_normal(shp_k), g.standard_normal(shp_k))
        _check_invariants(pool)
    assert pool.counters["shrink"] > 0 and pool.counters["cow_pages"] == 6
    # the sharer's prompt is untouched by the other request's shrinking
    np.testing.assert_array_equal(pool.requests[b_].K[:, :, :24], K_before)
    pool.release(a); pool.release(b_)
    assert pool.n_free() == c.n_pages


# ----------------------------------------------------------------------------- near-tie margins and moved rows
def test_working_set_margin_is_the_distance_of_the_running_sum_from_p_at_the_crossing():
    # dyadic weights: every cumulative sum is exact, so the margins below are hand arithmetic
    a = np.array([0.125, 0.5, 0.125, 0.25])                 # descending: 0.5, 0.25, 0.125, 0.125 -> sums 0.5, 0.75, 0.875, 1
    k, m = O.p_coverage_demand_with_margin(a, 0.7)           # crossing at k = 2: above by 0.05, the sum before is 0.2 short
    assert k == 2 and abs(m - (0.75 - 0.7) / 0.7) < 1e-15
    k, m = O.p_coverage_demand_with_margin(a, 0.52)          # same k, but now the sum before (0.5) is the closer one
    assert k == 2 and abs(m - (0.52 - 0.5) / 0.52) < 1e-15
    k, m = O.p_coverage_demand_with_margin(a, 0.4)           # k = 1: the sum before is the empty sum
    assert k == 1 and abs(m - (0.5 - 0.4) / 0.4) < 1e-15
    k, m = O.p_coverage_demand_with_margin(a, 0.875)         # hits p exactly: a tie in the sense of the protocol
    assert k == 3 and m == 0.0
    k, m = O.p_coverage_demand_with_margin(a, 0.875 * (1 + 1e-7))
    assert k == 4 and 0.9e-7 < m < 1.1e-7                    # just missed: a near-tie (< 1e-6)
    assert O.p_coverage_demand(a, 0.7) == 2


def test_selection_margin_is_the_smallest_relative_gap_at_any_local_or_global_cut():
    # two blocks of four, one local pick each, two global picks
    s = np.array([8.0, 4.0, 2.0, 1.0, 16.0, 3.0, 0.5, 0.25])
    keep, margin = O.select_retained(s, 2, 4, 4, 1)
    np.testing.assert_array_equal(keep, [0, 1, 4, 5])        # locals 0 and 4; of the rest {4, 2, 1, 3, .5, .25} the best two
    # local cuts: (8 - 4) / 8 and (16 - 3) / 16; global cut between 3 (kept) and 2 (dropped)
    assert abs(margin - (3.0 - 2.0) / 3.0) < 1e-15
    # now the tightest cut is a local one: block 0's best two are 8 and 7.75 with a quota of one
    s = np.array([8.0, 7.75, 2.0, 1.0, 16.0, 3.0, 0.5, 0.25])
    keep, margin = O.select_retained(s, 2, 4, 4, 1)
    np.testing.assert_array_equal(keep, [0, 1, 4, 5])
    assert abs(margin - 0.25 / 8.0) < 1e-15
    # no cut at all (everything kept): the margin is infinite; _top on its own
    keep, gap = O._top(np.arange(4), np.array([1.0, 4.0, 2.0, 3.0]), 4)
    assert gap == math.inf and sorted(keep.tolist()) == [0, 1, 2, 3]
    keep, gap = O._top(np.arange(4), np.array([1.0, 4.0, 2.0, 3.0]), 2)
    assert keep.tolist() == [1, 3] and abs(gap - (3.0 - 2.0) / 3.0) < 1e-15


def _boundary_with_forced_working_sets(monkeypatch, k_s, k_l, margins, **cfg_over):
    """Runs one request into its first boundary with Eq. 7's results replaced by the given ones, so that the
    bookkeeping around them (Eq. 8, the decision, the near-tie flag) can be checked by hand."""
    c = _cfg(n_layers=1, n_kv_heads=2, n_q_heads=4, **cfg_over)
    pool = O.OraclePool(c)
    n0 = 3 * c.page_size - 1                                  # three pages, one slot free
    kt = RNG.standard_normal((1, n0, 2, c.head_dim))
    assert pool.request_add(-1, 0, kt, kt.copy(), n0, 0) == (O.OK, 0)
    seq = iter([(k_s[0], margins[0]), (k_l[0], margins[1]), (k_s[1], margins[2]), (k_l[1], margins[3])])
    monkeypatch.setattr(O, "p_coverage_demand_with_margin", lambda a, p: next(seq))
    rec = pool.step_compute([0], *_rand_step(c, 1))
    return rec.boundary[0], c


def test_action_near_tie_flag_says_whether_a_near_tied_working_set_could_flip_the_decision(monkeypatch):
    # |C| = 8, two KV heads: Delta = (sum K^S - sum K^L) / (2 * 8)
    info, c = _boundary_with_forced_working_sets(monkeypatch, (3, 4), (3, 4), (1e-9, 0.1, 0.1, 0.1))
    assert info.delta == 0.0 and not info.want_grow           # Delta = 0 compresses
    assert info.action_near_tie                               # one size off by one makes Delta = +1/16 > tau: it could grow
    info, c = _boundary_with_forced_working_sets(monkeypatch, (6, 5), (3, 3), (1e-9, 0.1, 0.1, 0.1))
    assert info.delta == 5 / 16 and info.want_grow
    assert not info.action_near_tie                           # 4/16 and 6/16 are on the same side of tau
    info, c = _boundary_with_forced_working_sets(monkeypatch, (3, 4), (3, 4), (1e-5, 0.1, 0.1, 0.1))
    assert not info.action_near_tie                           # a margin of 1e-5 is not a near-tie
    info, c = _boundary_with_forced_working_sets(monkeypatch, (4, 4), (3, 3), (1e-9, 1e-9, 0.1, 0.1), tau=0.0)
    assert info.want_grow and info.action_near_tie            # two near-ties: 2/16 could become 0/16


def _compress_with_keep(keep_slots, shared_pages):
    """One request of three 16-token pages at its boundary, compressed with a prescribed keep set; when
    shared_pages > 0 its leading prompt pages are shared with a donor.  Returns the boundary record."""
    c = O.OracleConfig(1, 2, 1, 8, n_pages=16, max_pages_per_req=4, k_loc=0, max_requests=4)
    pool = O.OraclePool(c)
    kt = RNG.standard_normal((1, 47, 1, 8))
    assert pool.request_add(-1, 0, kt, kt.copy(), 47, 0) == (O.OK, 0)
    rid = 0
    if shared_pages:
        tail = 47 - 16 * shared_pages
        kt2 = RNG.standard_normal((1, tail, 1, 8))
        assert pool.request_add(0, shared_pages, kt2, kt2.copy(), tail, 0) == (O.OK, 1)
        rid = 1
    q, k, v = RNG.standard_normal((1, 1, 2, 8)), RNG.standard_normal((1, 1, 1, 8)), RNG.standard_normal((1, 1, 1, 8))
    rec = pool.decode_step([rid], q, k, v, overrides={rid: {"keep": {(0, 0): np.asarray(keep_slots)}}})
    info = rec.boundary[rid]
    assert info.action == O.ACT_COMPRESS and pool.requests[rid].n == 32
    assert pool.counters["moved_rows"] == info.moved_tokens
    return info


def test_moved_rows_counts_the_slots_that_change_place_and_whole_copied_pages():
    # |C| = 32, 16 go.  Keep slots 0..7 and 16..23: 0..7 stay where they are, 16..23 move to 8..15, the 16 protected
    # slots 32..47 move to 16..31
    keep = list(range(0, 8)) + list(range(16, 24))
    assert _compress_with_keep(keep, 0).moved_tokens == 8 + 16
    # keep the whole first page: only the protected page moves (slots 32..47 -> 16..31)
    assert _compress_with_keep(list(range(16)), 0).moved_tokens == 16
    # keep the whole second page: it moves down one page, and so does the protected page
    assert _compress_with_keep(list(range(16, 32)), 0).moved_tokens == 32
    # the first page is shared with a donor: it is copied to a fresh page, so its kept slots count although
    # their slot numbers do not change
    info = _compress_with_keep(keep, 1)
    assert info.cow_pages == 1 and info.moved_tokens == 8 + 8 + 16
    info = _compress_with_keep(list(range(16)), 1)
    assert info.cow_pages == 1 and info.moved_tokens == 16 + 16
    # both candidate pages shared: every kept slot is written to a fresh page
    info = _compress_with_keep(list(range(4, 20)), 2)
    assert info.cow_pages == 2 and info.moved_tokens == 16 + 16


# ----------------------------------------------------------------------------- asynchronous boundary work
def _run_oracle_job(async_boundary, n_req=3, n_tokens=40, seed=5):
    """Feeds every request its own fixed token stream; a request that is held keeps its token for the next step.
    Returns per request the list of (token index, output, retained ids after the step) and the step log."""
    c = _cfg(n_layers=1, n_pages=40, max_pages_per_req=8, async_boundary=async_boundary, tau=-0.03)
    rng = np.random.default_rng(seed)
    pool = O.OraclePool(c)
    streams = []
    for r in range(n_req):
        n0 = 5 + 3 * r
        kt = rng.standard_normal((1, n0, c.n_kv_heads, c.head_dim))
        assert pool.request_add(-1, 0, kt, kt + 1.0, n0, 0) == (O.OK, r)
        streams.append([(rng.standard_normal((1, c.n_q_heads, c.head_dim)), rng.standard_normal((1, c.n_kv_heads, c.head_dim)),
                         rng.standard_normal((1, c.n_kv_heads, c.head_dim))) for _ in range(n_tokens)])
    done = [0] * n_req
    per_token = [[] for _ in range(n_req)]
    log = []
    while min(done) < n_tokens:
        rids = [r for r in range(n_req) if done[r] < n_tokens]
        q = np.stack([streams[r][done[r]][0] for r in rids], axis=1)
        k = np.stack([streams[r][done[r]][1] for r in rids], axis=1)
        v = np.stack([streams[r][done[r]][2] for r in rids], axis=1)
        before = {r: pool.request_state(r)[:3] for r in rids}
        rec = pool.decode_step(rids, q, k, v)
        for i, r in enumerate(rids):
            a = int(rec.actions[i])
            log.append((pool.serial - 1, r, a))
            if a == O.ACT_HELD:
                assert pool.request_state(r)[2] == before[r][2]            # the position does not move while sitting out
                continue
            assert a >= 0
            per_token[r].append((done[r], rec.out[:, i].copy(), pool.requests[r].pos))
            done[r] += 1
        _check_invariants(pool)
    final = {r: (pool.request_state(r)[:3], [pool.retained(r, 0, h).tolist() for h in range(c.n_kv_heads)],
                 pool.summaries(r)) for r in range(n_req)}
    return per_token, log, final, pool


def test_sitting_out_changes_when_a_token_is_decoded_not_what_it_sees():
    sync_tok, sync_log, sync_final, sp = _run_oracle_job(False)
    asyn_tok, asyn_log, asyn_final, ap = _run_oracle_job(True)
    # the pool never runs short here, so a request's own history decides everything: token for token the same
    # outputs, and the same pages, retained tokens and summaries at the end; no token lost or decoded twice
    for r in range(3):
        assert [t for t, _, _ in asyn_tok[r]] == list(range(40))
        for (t1, o1, p1), (t2, o2, p2) in zip(sync_tok[r], asyn_tok[r]):
            assert t1 == t2 and p1 == p2 and np.array_equal(o1, o2)
        assert sync_final[r][0] == asyn_final[r][0] and sync_final[r][1] == asyn_final[r][1]
        assert np.array_equal(sync_final[r][2], asyn_final[r][2])
    for name in ("grow", "compress", "fallback", "moved_rows", "scored_tokens"):
        assert sp.counters[name] == ap.counters[name]
    assert sp.counters["grow"] > 0 and sp.counters["compress"] > 0
    # every boundary is reported as pending, is followed by exactly one step out, and costs exactly that step
    pend = [(s, r) for s, r, a in asyn_log if a == O.ACT_PENDING]
    held = [(s, r) for s, r, a in asyn_log if a == O.ACT_HELD]
    assert len(pend) > 0 and sorted((s + 1, r) for s, r in pend if (s + 1, r) in held) == sorted(held)
    assert all(a not in (O.ACT_PENDING, O.ACT_HELD) for _, _, a in sync_log)
    n_b = {r: sum(1 for _, rr in pend if rr == r) for r in range(3)}
    last_async = {r: max(s for s, rr, a in asyn_log if rr == r and a != O.ACT_HELD) for r in range(3)}
    assert all(last_async[r] == 39 + n_b[r] - (1 if (last_async[r], r) in pend else 0) for r in range(3))
    # the decision is remembered with the step it belongs to
    for r in range(3):
        act, at = ap.boundary_outcome(r)
        assert at == max(s for s, rr in pend if rr == r) and act in (O.ACT_GROW, O.ACT_COMPRESS, O.ACT_COMPRESS_FALLBACK)


# ----------------------------------------------------------------------------- protected window smaller than a block
def _best_subset_ragged(s, b, K_t, k_prime):
    """Exhaustive optimum of Eq. 10 over len(s) candidates in blocks of b, the last one short: the K_t slots of
    largest total score among the choices that keep at least min(k', block size) slots of every block."""
    n = len(s)
    n_blocks = -(-n // b)
    size = np.bincount(np.arange(n) // b, minlength=n_blocks)
    best, best_val = None, -1.0
    for comb in itertools.combinations(range(n), K_t):
        cnt = np.bincount(np.asarray(comb) // b, minlength=n_blocks)
        if np.all(cnt >= np.minimum(k_prime, size)):
            val = s[list(comb)].sum()
            if val > best_val:
                best, best_val = comb, val
    return np.asarray(best)


@pytest.mark.parametrize("P,b,R,k_loc", [(3, 4, 2, 1), (2, 6, 2, 2), (3, 4, 1, 1), (4, 3, 1, 0)])
def test_selection_with_a_short_last_block_is_the_constrained_optimum(P, b, R, k_loc):
    # the paper's geometry in small: blocks of b slots, a protected window of R < b newest tokens; the candidates
    # are all P b - R others, the target (P - 1) b - R of them, so exactly one block worth of slots goes
    n_e, K_t = P * b - R, (P - 1) * b - R
    for _ in range(5):
        s = RNG.random(n_e) ** 3
        keep, _ = O.select_retained(s, P, b, K_t, k_loc)
        assert keep.size == K_t == n_e - b and np.all(np.diff(keep) > 0)
        np.testing.assert_array_equal(keep, _best_subset_ragged(s, b, K_t, min(k_loc, K_t // P)))


def test_two_supports_demand_leaves_out_the_newest_block_eviction_only_the_protected_window():
    b, R = 8, 2
    c = O.OracleConfig(2, 4, 2, 8, n_pages=12, max_pages_per_req=4, page_size=b, recent_window=R, k_loc=2, max_requests=2)
    pool = O.OraclePool(c)
    n0 = 3 * b - 1
    kt = RNG.standard_normal((2, n0, 2, 8))
    assert pool.request_add(-1, 0, kt, kt * 0.5, n0, 0) == (O.OK, 0)
    r = pool.requests[0]
    q, k, v = _rand_step(c, 1)
    rec = pool.step_compute([0], q, k, v)
    info = rec.boundary[0]
    assert (info.n_c, info.n_e) == (2 * b, 3 * b - R)             # |C_t| of Eq. 7 and the candidates of Eq. 10
    assert info.a_s.shape[-1] == 2 * b and info.e_s.shape[-1] == 3 * b - R
    for a in (info.a_s, info.a_l, info.e_s, info.e_l):               # each support has its own normalisation
        np.testing.assert_allclose(a.sum(axis=-1), 1.0, rtol=1e-12)
    # the demand views do not see the newest block: changing its keys changes neither K^S nor K^L nor Delta ...
    ks, kl, delta = info.K_s.copy(), info.K_l.copy(), info.delta
    saved = r.K[:, :, 2 * b:3 * b - R].copy()
    r.K[:, :, 2 * b:3 * b - R] *= 3.0
    info2 = pool._demand(0, r, q[:, 0], r.pos - 1)
    assert np.array_equal(info2.K_s, ks) and np.array_equal(info2.K_l, kl) and info2.delta == delta
    assert not np.allclose(info2.e_s, info.e_s)                   # ... but the eviction scores do
    r.K[:, :, 2 * b:3 * b - R] = saved
    tok_before = r.tok[:, :, :3 * b].copy()
    pool.step_apply(rec)
    assert info.action == O.ACT_COMPRESS                          # first boundary: both summaries equal, Delta = 0
    assert r.n == 2 * b and r.P == 3                              # exactly one block of slots is free again
    for l in range(2):
        for h in range(2):
            kept = r.tok[l, h, :r.n]
            assert np.all(np.diff(kept) > 0) and kept.size == 2 * b
            assert np.array_equal(kept[-R:], tok_before[l, h, 3 * b - R:3 * b])      # the R newest tokens survive
            assert np.isin(kept[:-R], tok_before[l, h, :3 * b - R]).all()
            # tokens of the newest block outside the window are ordinary candidates: some may go, some stay
            assert info.keep[(l, h)].size == 2 * b - R
            # every block, the short last one included, keeps its quota
            cnt = np.bincount(info.keep[(l, h)] // b, minlength=3)
            assert (cnt >= min(c.k_loc, (2 * b - R) // 3)).all()
    _check_invariants(pool)


def test_paper_geometry_runs_and_keeps_its_invariants():
    # b = 256, |R| = 16, k_loc = 64 (Sec. 5.1, App. B.2) on a small head shape: boundaries every 256 tokens
    c = O.OracleConfig(1, 2, 1, 8, n_pages=8, max_pages_per_req=3, page_size=256, recent_window=16, k_loc=64, max_requests=2,
                       tau=-1.0)
    pool = O.OraclePool(c)
    n0 = 300
    kt = RNG.standard_normal((1, n0, 1, 8))
    assert pool.request_add(-1, 0, kt, kt.copy(), n0, 0) == (O.OK, 0)
    r = pool.requests[0]
    assert r.P == 2
    acts = []
    for t in range(600):
        rec = pool.decode_step([0], *_rand_step(c, 1))
        if rec.actions[0] != O.ACT_NONE:
            acts.append((t, int(rec.actions[0]), r.P, r.n))
            info = rec.boundary[0]
            if rec.actions[0] == O.ACT_COMPRESS_FALLBACK:
                assert info.n_c == 2 * 256 and info.n_e == 3 * 256 - 16 and info.keep[(0, 0)].size == 2 * 256 - 16
                assert r.n == 2 * 256 and np.array_equal(r.tok[0, 0, r.n - 16:r.n], np.arange(r.pos - 16, r.pos))
    # 300 + 212 tokens fill two blocks: grant; 256 more fill three: at the cap, compress; then every 256 tokens
    assert [a[:2] for a in acts] == [(211, O.ACT_GROW), (467, O.ACT_COMPRESS_FALLBACK)], acts
    _check_invariants(pool)


# ----------------------------------------------------------------------------- entropy as the working-set metric
def test_entropy_metric_closed_forms_and_its_use_in_the_decision():
    n = 64
    H, r = O.entropy_ratio(np.full(n, 1.0 / n))
    assert abs(H - math.log(n)) < 1e-12 and abs(r - 1.0) < 1e-12            # flat view: the whole set
    one_hot = np.zeros(n); one_hot[17] = 1.0
    assert O.entropy_ratio(one_hot) == (0.0, 0.0)                           # one token: nothing to spread over
    a = np.array([0.5, 0.25, 0.25])
    assert abs(O.entropy_ratio(a)[0] - 1.5 * math.log(2.0)) < 1e-15          # 0.5 ln 2 + 2 * 0.25 ln 4
    two = np.zeros(n); two[:2] = 0.5
    assert abs(O.entropy_ratio(two)[1] - math.log(2) / math.log(n)) < 1e-15
    # like K / |C|, the ratio grows when mass spreads: the sign convention of Delta_t carries over
    g = np.exp(-0.3 * np.arange(n)); g /= g.sum()
    w = np.exp(-0.05 * np.arange(n)); w /= w.sum()
    assert O.entropy_ratio(w)[1] > O.entropy_ratio(g)[1] and O.p_coverage_demand(w, 0.99) > O.p_coverage_demand(g, 0.99)
    # in the state machine: Delta_t from entropies, same decision rule, same compression afterwards
    c = _cfg(n_layers=2, demand_metric=1, tau=0.0)
    pool = O.OraclePool(c)
    n0 = 3 * c.page_size - 1
    kt = RNG.standard_normal((2, n0, 2, c.head_dim))
    assert pool.request_add(-1, 0, kt, kt.copy(), n0, 0) == (O.OK, 0)
    rec = pool.decode_step([0], *_rand_step(c, 1))
    info = rec.boundary[0]
    assert info.delta == 0.0 and info.action == O.ACT_COMPRESS              # first step: both summaries are the query
    for t in range(3 * c.page_size):
        rec = pool.decode_step([0], *_rand_step(c, 1))
        if 0 in rec.boundary:
            info = rec.boundary[0]
            want = sum(O.entropy_ratio(info.a_s[l, h])[1] - O.entropy_ratio(info.a_l[l, h])[1]
                       for l in range(2) for h in range(2)) / 4.0             # Eq. 8 with the entropy ratios
            assert abs(info.delta - want) < 1e-12 and info.want_grow == (info.delta > 0.0)
            assert not info.K_s.any()
    _check_invariants(pool)
