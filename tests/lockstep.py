"""Runs a synthetic workload through the CUDA pool and the float64 oracle in lockstep and compares
them after every decode step.  Helper for the GPU parity tests and the smoke check.

Tolerances (stated by the benchmark spec):
  attention outputs        max |err| <= 1e-2 and mean |err| <= 1e-3 (bf16 inputs, fp32 accumulation)
  query summaries          ||gpu - oracle||_2 / ||oracle||_2 <= 1e-4 per (layer, view, head) vector
  working-set sizes, retained-index sets, grow / compress actions, page counts
                           bit-exact, except inside near-ties whose oracle margin is < 1e-6
                           relative; those are counted, must stay below 0.1 % of decisions, and the
                           oracle then adopts the GPU's choice so that the two stay comparable.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, Optional

import numpy as np

from oracle import growpage_oracle as O
from paper_2609_03494_b200 import binding as B
from paper_2609_03494_b200 import harness as H
from paper_2609_03494_b200 import workload as W

ATTN_MAX_ABS = 1e-2
ATTN_MEAN_ABS = 1e-3
SUMMARY_REL = 1e-4
NEAR_TIE = 1e-6
NEAR_TIE_FRACTION = 1e-3


@dataclasses.dataclass
class Stats:
    steps: int = 0
    tokens: int = 0
    attn_max_abs: float = 0.0
    attn_sum_abs: float = 0.0
    attn_count: int = 0
    summary_max_rel: float = 0.0
    decisions: Dict[str, int] = dataclasses.field(default_factory=lambda: {"ws": 0, "sel": 0, "act": 0})
    near_ties: Dict[str, int] = dataclasses.field(default_factory=lambda: {"ws": 0, "sel": 0, "act": 0})
    actions: Dict[int, int] = dataclasses.field(default_factory=dict)
    counters: Optional[np.ndarray] = None

    @property
    def attn_mean_abs(self) -> float:
        return self.attn_sum_abs / max(self.attn_count, 1)


def make_pools(wl: W.Workload, device: int = 0, **over):
    s = wl.shape
    kw = dict(n_pages=wl.n_pages, max_pages_per_req=wl.max_pages_per_req,
              max_requests=max(4, wl.n_resident), k_loc=wl.k_loc)
    tun = {k: over[k] for k in ("beta_s", "beta_l", "top_p", "tau", "rope_theta", "policy", "policy_seed", "p_compress",
                                    "shrink_below", "min_capacity", "async_boundary", "demand_metric")
           if k in over}
    for k in ("n_pages", "max_pages_per_req", "k_loc", "max_requests"):
        if k in over:
            kw[k] = over[k]
    ocfg = O.OracleConfig(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, page_size=s.page_size, recent_window=16, **kw, **tun)
    gcfg = B.make_config(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, page_size=s.page_size, **kw, **tun,
                         max_batch_tokens=over.get("max_batch_tokens", 0), async_slots=over.get("async_slots", 0),
                         overlap_slots=over.get("overlap_slots", 0),
                         max_boundary_tokens=over.get("max_boundary_tokens", 0))
    pool = B.Pool(gcfg, device)
    if over.get("compact_by_unit"):
        B.gp_test_withhold(pool.handle, 16, 0)          # the compaction claims whole units whatever their number
    return pool, O.OraclePool(ocfg)


def _to_dev(torch, arr: np.ndarray, device: int):
    return torch.from_numpy(np.ascontiguousarray(arr).view(np.int16)).to(f"cuda:{device}")


def run_lockstep(wl: W.Workload, max_steps: Optional[int] = None, summary_every: int = 16, device: int = 0,
                 check_pool_every: int = 8, **over) -> Stats:
    import torch
    gpu, ora = make_pools(wl, device, **over)
    s = wl.shape
    b = s.page_size
    sch = H.Scheduler(wl)
    st = Stats()
    try:
        while not sch.done():
            # ---- admissions, mirrored on both sides --------------------------------------------------
            while True:
                op = sch.next_admission()
                if op is None:
                    break
                sf = sch.rid_of(op.share_from_spec) if op.share_from_spec >= 0 else -1
                g_st, g_rid = gpu.request_add(sf, op.n_shared_pages, op.k_tail, op.v_tail, op.n_tail, op.initial_pages)
                o_st, o_rid = ora.request_add(sf, op.n_shared_pages,
                                              None if op.k_tail is None else H.decode_bits(op.k_tail),
                                              None if op.v_tail is None else H.decode_bits(op.v_tail),
                                              op.n_tail, op.initial_pages)
                o_map = {O.OK: B.GP_OK, O.ERR_INVALID: B.GP_ERR_INVALID, O.ERR_NO_SLOT: B.GP_ERR_NO_SLOT,
                         O.ERR_NO_PAGES: B.GP_ERR_NO_PAGES}
                assert g_st == o_map[o_st], f"admission status gpu {g_st} oracle {o_st}"
                if g_st != B.GP_OK:
                    break
                assert g_rid == o_rid
                sch.admitted(op, g_rid)
            if not sch.resident:
                raise AssertionError("nothing resident and nothing admissible: pool too small for the workload")
            if max_steps is not None and st.steps >= max_steps:
                break
            specs, rids, q, k, v = sch.batch()
            Bn = len(rids)
            ids_t = torch.tensor(rids, dtype=torch.int32, device=f"cuda:{device}")
            out_t = torch.zeros((s.n_layers, Bn, s.n_q_heads, s.head_dim), dtype=torch.float32, device=f"cuda:{device}")
            act_t = torch.zeros(Bn, dtype=torch.int32, device=f"cuda:{device}")
            gpu.decode_step(ids_t, _to_dev(torch, q, device), _to_dev(torch, k, device), _to_dev(torch, v, device),
                            out_t, act_t)
            rec = ora.step_compute(rids, H.decode_bits(q), H.decode_bits(k), H.decode_bits(v))
            g_out = out_t.cpu().numpy().astype(np.float64)
            g_act = act_t.cpu().numpy()

            # ---- attention outputs --------------------------------------------------------------------------
            stepped = [i for i in range(Bn) if rec.actions[i] in (O.ACT_NONE, O.ACT_PENDING)]
            # what the GPU decided at this step's boundaries: in the step's actions, or, with asynchronous boundary
            # work, asked for afterwards (the call waits for the boundary chain)
            is_async = bool(over.get("async_boundary", False))
            g_dec = {}
            for rid in rec.boundary:
                i = rids.index(rid)
                if is_async:
                    assert int(g_act[i]) == B.GP_ACT_PENDING, f"step {st.steps} req {rid}: action {g_act[i]}, expected pending"
                    g_dec[rid], at = B.gp_boundary_outcome(gpu.handle, rid)
                    assert at == ora.serial - 1, f"step {st.steps} req {rid}: boundary step gpu {at} oracle {ora.serial - 1}"
                else:
                    g_dec[rid] = int(g_act[i])
            if stepped:
                err = np.abs(g_out[:, stepped] - rec.out[:, stepped])
                st.attn_max_abs = max(st.attn_max_abs, float(err.max()))
                st.attn_sum_abs += float(err.sum())
                st.attn_count += err.size
                assert err.max() <= ATTN_MAX_ABS, f"step {st.steps}: attention max abs err {err.max()}"

            # ---- boundary decisions ---------------------------------------------------------------------------
            overrides = {}
            for rid, info in rec.boundary.items():
                i = rids.index(rid)
                if info.n_c > 0:
                    ks, kl, delta = B.gp_debug_boundary(gpu.handle, rid, s.n_layers, s.n_kv_heads)
                    for name, gk, ok, col in (("S", ks, info.K_s, 0), ("L", kl, info.K_l, 1)):
                        st.decisions["ws"] += ok.size
                        bad = np.argwhere(gk != ok)
                        for (l, h) in bad:
                            assert info.ws_margin[l, h, col] < NEAR_TIE and abs(int(gk[l, h]) - int(ok[l, h])) == 1, (
                                f"step {st.steps} req {rid} K^{name}[{l},{h}] gpu {gk[l, h]} oracle {ok[l, h]} "
                                f"margin {info.ws_margin[l, h, col]}")
                            st.near_ties["ws"] += 1
                    if over.get("demand_metric", 0) == 1:
                        # entropy metric: floating-point sums of logarithms on both sides, compared to rounding
                        hs, hl = B.gp_debug_entropy(gpu.handle, rid, s.n_layers, s.n_kv_heads)
                        assert np.allclose(hs, info.H_s, rtol=1e-11, atol=1e-13) and np.allclose(hl, info.H_l, rtol=1e-11, atol=1e-13)
                        assert abs(delta - info.delta) <= 1e-12, f"Delta gpu {delta} oracle {info.delta}"
                    elif np.array_equal(ks, info.K_s) and np.array_equal(kl, info.K_l):
                        assert delta == info.delta, f"Delta gpu {delta} oracle {info.delta}"
                st.decisions["act"] += 1
                g_want = g_dec[rid] in (B.GP_ACT_GROW, B.GP_ACT_COMPRESS_FALLBACK) or \
                    (g_dec[rid] == B.GP_ACT_STALLED and info.n_c == 0)
                if info.n_c > 0 and g_dec[rid] != B.GP_ACT_STALLED and g_want != info.want_grow:
                    assert info.action_near_tie, f"step {st.steps} req {rid}: grow decision differs outside a near-tie"
                    st.near_ties["act"] += 1
                    overrides.setdefault(rid, {})["want_grow"] = g_want
                g_shrink = g_dec[rid] == B.GP_ACT_SHRINK
                if g_dec[rid] in (B.GP_ACT_COMPRESS, B.GP_ACT_SHRINK) and g_shrink != info.want_shrink:
                    assert info.action_near_tie, f"step {st.steps} req {rid}: shrink decision differs outside a near-tie"
                    st.near_ties["act"] += 1
                    overrides.setdefault(rid, {})["want_shrink"] = g_shrink
            # ---- retained sets of the requests the GPU compressed -----------------------------------------------
            for rid, info in rec.boundary.items():
                if g_dec[rid] not in (B.GP_ACT_COMPRESS, B.GP_ACT_COMPRESS_FALLBACK, B.GP_ACT_SHRINK):
                    continue
                r = ora.requests[rid]
                R = ora.cfg.recent_window
                # the candidates of Eq. 10 are everything but the protected window; a page worth of them goes (Eq. 13:
                # a Shrink evicts two pages)
                K_t = info.n_e - (2 * b if g_dec[rid] == B.GP_ACT_SHRINK else b)
                for l in range(s.n_layers):
                    for h in range(s.n_kv_heads):
                        st.decisions["sel"] += 1
                        keep, margin = O.select_retained(O.token_scores(info.e_s[l, h], info.e_l[l, h]),
                                                         -(-info.n_e // b), b, K_t, ora.cfg.k_loc)
                        want_tok = r.tok[l, h, keep]
                        got = B.gp_debug_retained(gpu.handle, rid, l, h, K_t + R)
                        got_hist, got_prot = got[:K_t], got[K_t:]
                        assert np.array_equal(got_prot, r.tok[l, h, info.n_e:info.n_e + R]), "protected window lost"
                        if not np.array_equal(got_hist, want_tok):
                            assert margin < NEAR_TIE, (f"step {st.steps} req {rid} ({l},{h}): retained set differs, "
                                                       f"margin {margin}")
                            assert np.all(np.diff(got_hist) > 0) and np.isin(got_hist, r.tok[l, h, :info.n_e]).all()
                            st.near_ties["sel"] += 1
                            slots = np.searchsorted(r.tok[l, h, :info.n_e], got_hist)
                            overrides.setdefault(rid, {}).setdefault("keep", {})[(l, h)] = slots
            ora.step_apply(rec, overrides)

            # ---- actions and page state ---------------------------------------------------------------------------
            for i, rid in enumerate(rids):
                a_g, a_o = int(g_act[i]), int(rec.actions[i])
                assert a_g == a_o, f"step {st.steps} req {rid}: action gpu {a_g} oracle {a_o}"
                st.actions[a_g] = st.actions.get(a_g, 0) + 1
            for rid, info in rec.boundary.items():          # the decisions themselves (asynchronous mode: not in the actions)
                assert g_dec[rid] == info.action, f"step {st.steps} req {rid}: decision gpu {g_dec[rid]} oracle {info.action}"
                if is_async:
                    st.actions[g_dec[rid]] = st.actions.get(g_dec[rid], 0) + 1
            if check_pool_every and (st.steps % check_pool_every == 0 or rec.boundary):
                for rid in rids:
                    if rid not in ora.requests:
                        continue
                    P, n, pos, table = B.gp_debug_request(gpu.handle, rid, gpu.cfg.max_pages_per_req)
                    oP, on, opos, otable = ora.request_state(rid)
                    assert (P, n, pos) == (oP, on, opos), f"step {st.steps} req {rid}: state gpu {(P, n, pos)} oracle {(oP, on, opos)}"
                    assert len(set(table)) == P
                n_free, ref, counters = B.gp_debug_pool(gpu.handle, gpu.cfg.n_pages)
                assert n_free == ora.n_free(), f"step {st.steps}: free pages gpu {n_free} oracle {ora.n_free()}"
                assert counters[7] == 0, f"kernel error bits {counters[7]}"
                assert int((ref > 0).sum()) + n_free == gpu.cfg.n_pages
                assert sorted(ref[ref > 0].tolist()) == sorted(ora.refcount[ora.refcount > 0].tolist())
            if summary_every and st.steps % summary_every == 0:
                _check_summaries(gpu, ora, rids, s, st)
            st.steps += 1
            st.tokens += len(stepped)
            for idx, rid in sch.after_step(specs, g_act):
                gpu.release(rid)
                assert ora.release(rid) == O.OK
        _check_summaries(gpu, ora, [r.rid for r in sch.resident.values()], s, st)
        _, _, st.counters = B.gp_debug_pool(gpu.handle)
        assert st.counters[7] == 0
        for kind in st.decisions:
            if st.decisions[kind]:
                frac = st.near_ties[kind] / st.decisions[kind]
                assert frac < NEAR_TIE_FRACTION, f"{kind}: near-tie fraction {frac}"
        assert st.attn_mean_abs <= ATTN_MEAN_ABS, f"attention mean abs err {st.attn_mean_abs}"
        assert st.summary_max_rel <= SUMMARY_REL
        for name, gi in (("grow", 0), ("compress", 1), ("fallback", 2), ("stalled", 3), ("cow_pages", 4),
                         ("moved_rows", 8), ("scored_tokens", 9), ("shrink", 10)):
            assert int(st.counters[gi]) == ora.counters[name], f"counter {name}: gpu {st.counters[gi]} oracle {ora.counters[name]}"
    finally:
        gpu.close()
    return st


def _check_summaries(gpu, ora, rids, s, st: Stats) -> None:
    for rid in rids:
        if rid not in ora.requests or not ora.requests[rid].started:
            continue
        g = B.gp_debug_summaries(gpu.handle, rid, s.n_layers, s.n_q_heads, s.head_dim)
        o = ora.summaries(rid)
        num = np.linalg.norm(g - o, axis=-1)
        den = np.linalg.norm(o, axis=-1)
        rel = float((num / np.where(den > 0, den, 1.0)).max())
        st.summary_max_rel = max(st.summary_max_rel, rel)
        assert rel <= SUMMARY_REL, f"req {rid}: summary relative error {rel}"
