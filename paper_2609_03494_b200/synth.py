"""Device-side synthetic inputs and a scheduler loop for the multi-layer configurations at their stated sizes.

The seeded CPU generator in `workload.py` feeds both the CUDA path and the CPU checker and is what every parity
test uses; at the full sizes (36 or 64 layers, hundreds of resident requests, a pool of 120 GB) a step's inputs are
75 to 150 MB and the host cannot produce them at the rate the GPU consumes them.  This module draws inputs of the
same law on the device with torch's generator (throughput mode: same recipe, other numbers), plays the scheduler
(admission, release of finished and stalled requests, re-admission into the freed slots) and checks, on the
state read back through the C ABI, the properties that hold at any size.  It holds none of the method's
arithmetic apart from the float64 restatement of dense attention used as a spot check.

Recipe (as `workload.py`): per (layer, KV head) a unit direction u; a token is a heavy hitter with the request's
probability f_r (log-uniform in [0.5 %, 20 %]); heavy key = 4 u + 0.1 N(0, I), other keys and all values N(0, I);
query = 2 u + N(0, I) per query head; everything rounded to bf16.  A request with a direction shift gets a fresh
u of its own at a random step in [25 %, 75 %] of its output.
"""
from __future__ import annotations

import dataclasses
import math
import time
from typing import Dict, List, Optional

import numpy as np

from . import binding as B
from . import workload as W


@dataclasses.dataclass
class SizeConfig:
    name: str
    shape: W.Shape
    n_resident: int
    n_pages: int
    prompt_range: tuple
    out_range: tuple              # log-uniform output lengths
    cap_pages: int
    initial_pages: int = 0
    groups: int = 0               # > 0: residents form this many groups that share a prompt of prompt_range[1] tokens
    shift: bool = False           # mid-generation direction shift
    fixed_frac: Optional[float] = None


def config3(n_layers: int = 36, n_resident: int = 256, pool_bytes: float = 120e9) -> SizeConfig:
    """36-layer Qwen3-8B-shaped stack, 256 residents, outputs log-uniform in [1k, 16k], pool of 120 GB."""
    s = W.Shape(n_layers, 32, 8, 128)
    page_bytes = s.n_layers * s.token_bytes * s.page_size
    return SizeConfig("qwen3-8b-stack", s, n_resident, int(pool_bytes // page_bytes), (128, 1024), (1024, 16384),
                      cap_pages=(1024 + 16384) // 16 + 2)


def config4(n_layers: int = 64, n_resident: int = 128, pool_bytes: float = 120e9) -> SizeConfig:
    """64-layer Qwen3-32B-shaped stack (64 query / 8 KV heads), 128 requests, outputs up to 32k, direction shift."""
    s = W.Shape(n_layers, 64, 8, 128)
    page_bytes = s.n_layers * s.token_bytes * s.page_size
    return SizeConfig("qwen3-32b-stack", s, n_resident, int(pool_bytes // page_bytes), (128, 1024), (2048, 32768),
                      cap_pages=(1024 + 32768) // 16 + 2, shift=True)


def config5(n_groups: int = 16, group_size: int = 16, prompt_len: int = 2048, n_steps: int = 8192) -> SizeConfig:
    """Prefix stress on the 8B layer shape: groups sharing a 2048-token prompt in refcounted pages."""
    s = W.Shape(1, 32, 8, 128)
    n_req = n_groups * group_size
    p0 = max(8, prompt_len // 16 + 1)
    return SizeConfig("prefix-stress", s, n_req, n_groups * (prompt_len // 16) + n_req * (p0 + 8), (prompt_len, prompt_len),
                      (n_steps, n_steps), cap_pages=p0 + n_steps // 16 + 1, initial_pages=8, groups=n_groups, fixed_frac=0.05)


class DeviceInputs:
    def __init__(self, torch, device: int, shape: W.Shape, n_slots: int, seed: int):
        self.torch, self.dev, self.s, self.n = torch, f"cuda:{device}", shape, n_slots
        self.gen = torch.Generator(device=self.dev)
        self.gen.manual_seed(seed)
        u = torch.randn((shape.n_layers, shape.n_kv_heads, shape.head_dim), generator=self.gen, device=self.dev)
        self.u = u / u.norm(dim=-1, keepdim=True)
        # direction of every slot's queries and heavy keys: the common one until a request's shift
        self.u_slot = self.u[:, None].expand(-1, n_slots, -1, -1).contiguous()            # [L][B][H_kv][d]
        self.frac = torch.full((n_slots,), 0.05, device=self.dev)

    def fresh_direction(self, slot: int) -> None:
        s = self.s
        u2 = self.torch.randn((s.n_layers, s.n_kv_heads, s.head_dim), generator=self.gen, device=self.dev)
        self.u_slot[:, slot] = u2 / u2.norm(dim=-1, keepdim=True)

    def reset_slot(self, slot: int, frac: float) -> None:
        self.u_slot[:, slot] = self.u
        self.frac[slot] = frac

    def prompt(self, n: int, frac: float):
        """K, V of a prompt in cache form, bf16 [L][n][H_kv][d]."""
        t, s = self.torch, self.s
        k = t.randn((s.n_layers, n, s.n_kv_heads, s.head_dim), generator=self.gen, device=self.dev)
        heavy = t.rand((n,), generator=self.gen, device=self.dev) < frac
        k = t.where(heavy[None, :, None, None], 4.0 * self.u[:, None] + 0.1 * k, k)
        v = t.randn((s.n_layers, n, s.n_kv_heads, s.head_dim), generator=self.gen, device=self.dev)
        return k.to(t.bfloat16), v.to(t.bfloat16)

    def step(self):
        """q bf16 [L][B][H_q][d], k, v bf16 [L][B][H_kv][d] for all slots."""
        t, s = self.torch, self.s
        G = s.n_q_heads // s.n_kv_heads
        q = t.randn((s.n_layers, self.n, s.n_q_heads, s.head_dim), generator=self.gen, device=self.dev)
        q += 2.0 * self.u_slot.repeat_interleave(G, dim=2)
        k = t.randn((s.n_layers, self.n, s.n_kv_heads, s.head_dim), generator=self.gen, device=self.dev)
        heavy = t.rand((self.n,), generator=self.gen, device=self.dev) < self.frac
        k = t.where(heavy[None, :, None, None], 4.0 * self.u_slot + 0.1 * k, k)
        v = t.randn((s.n_layers, self.n, s.n_kv_heads, s.head_dim), generator=self.gen, device=self.dev)
        return q.to(t.bfloat16), k.to(t.bfloat16), v.to(t.bfloat16)


def check_invariants(pool: B.Pool, cfg, live: List[int], rng, last=None, n_samples: int = 6) -> Dict[str, int]:
    """Properties that hold at any size, on the state read back through the C ABI: page accounting and reference
    counts, token counts within the allocation, retained ids increasing with the newest page worth present, and
    (with `last` = (ids, q, out, actions) of the last step) sampled attention rows against float64 dense attention
    over the keys and values the pool holds."""
    b = 16
    n_free, ref, counters = B.gp_debug_pool(pool.handle, cfg.n_pages)
    assert counters[7] == 0, f"kernel error bits {counters[7]:#x}"
    held = np.zeros(cfg.n_pages, dtype=np.int64)
    state = {}
    for rid in live:
        P, n, pos, table = B.gp_debug_request(pool.handle, rid, cfg.max_pages_per_req)
        assert len(set(table)) == P and 0 < n <= P * b and P <= cfg.max_pages_per_req, (rid, P, n)
        held[table] += 1
        state[rid] = (P, n, pos)
    assert np.array_equal(held, ref.astype(np.int64)), "reference counts differ from the page tables"
    assert int((held > 0).sum()) + n_free == cfg.n_pages, "free pages + pages held != pool size"
    done = {"retained": 0, "attention": 0}
    L, Hkv, d = cfg.n_layers, cfg.n_kv_heads, cfg.head_dim
    G = cfg.n_q_heads // Hkv
    for rid in rng.choice(live, size=min(n_samples, len(live)), replace=False):
        rid = int(rid)
        P, n, pos = state[rid]
        l, h = int(rng.integers(L)), int(rng.integers(Hkv))
        tok = B.gp_debug_retained(pool.handle, rid, l, h, n).astype(np.int64)
        assert (np.diff(tok) > 0).all() and tok[0] >= 0 and tok[-1] == pos - 1, (rid, l, h)
        w = min(b, n)
        assert np.array_equal(tok[-w:], np.arange(pos - w, pos)), "the newest page worth of tokens is not retained"
        done["retained"] += 1
        if last is not None:
            ids, q, out, act = last
            i = ids.index(rid) if rid in ids else -1
            if i >= 0 and int(act[i]) == B.GP_ACT_NONE:
                kk, vv = B.gp_debug_kv(pool.handle, rid, l, h, n, d)
                kk, vv = W.bf16_bits_to_f64(kk), W.bf16_bits_to_f64(vv)
                qq = q[l, i, h * G:(h + 1) * G].double().cpu().numpy()
                z = qq @ kk.T / math.sqrt(d)
                p = np.exp(z - z.max(axis=1, keepdims=True))
                want = (p / p.sum(axis=1, keepdims=True)) @ vv
                got = out[l, i, h * G:(h + 1) * G].double().cpu().numpy()
                assert np.abs(got - want).max() <= 1e-2, f"request {rid} ({l},{h}): attention differs from dense attention"
                done["attention"] += 1
    return done


def run_at_size(sc: SizeConfig, n_steps: int, device: int = 0, seed: int = 2, chunk: int = 8, async_boundary: bool = False,
                tau: float = 0.0, boundary_tokens_div: int = 8, life_fraction: float = 1.0, check_every: int = 0,
                verbose: bool = False) -> Dict:
    """Runs `n_steps` decode steps of a configuration at its size with continuous batching: residents start at a
    random point of their life (a steady-state snapshot; `life_fraction` < 1 shortens all outputs so that more of
    them end inside a short run), finished and stalled requests are released after every chunk of steps and their
    slots re-admitted.  Device time is measured with CUDA events around the chunks' decode steps only (input
    generation and the scheduler's calls lie between chunks).  Returns throughput, bytes and what was checked."""
    import torch
    s = sc.shape
    b = s.page_size
    rng = np.random.default_rng(seed)
    M = sc.n_resident
    max_batch_tokens = sc.n_pages * b if not sc.groups else M * sc.cap_pages * b
    cfg = B.make_config(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, n_pages=sc.n_pages, max_pages_per_req=sc.cap_pages,
                        max_requests=max(4, M), tau=tau, async_boundary=async_boundary, max_batch_tokens=max_batch_tokens,
                        max_boundary_tokens=max(max_batch_tokens // boundary_tokens_div, sc.cap_pages * b))
    pool = B.Pool(cfg, device)
    inp = DeviceInputs(torch, device, s, M, seed)
    dev = f"cuda:{device}"
    remaining = np.zeros(M, dtype=np.int64)
    shift_at = np.full(M, -1, dtype=np.int64)
    live = np.zeros(M, dtype=bool)
    stats = {"admitted": 0, "finished": 0, "stalled": 0, "refused": 0, "shared_admissions": 0}
    group_donor: Dict[int, int] = {}

    def admit(slot: int, snapshot: bool) -> bool:
        frac = sc.fixed_frac if sc.fixed_frac is not None else float(np.exp(rng.uniform(math.log(0.005), math.log(0.2))))
        n_prompt = int(rng.integers(sc.prompt_range[0], sc.prompt_range[1] + 1))
        out_len = max(8, int(life_fraction * np.exp(rng.uniform(math.log(sc.out_range[0]), math.log(sc.out_range[1])))))
        donor, n_shared = -1, 0
        if sc.groups:
            g = slot % sc.groups
            if g in group_donor and live[group_donor[g]] and pristine[group_donor[g]]:
                donor, n_shared = group_donor[g], n_prompt // b
        n_tail = n_prompt - n_shared * b
        k = v = None
        if n_tail:
            k, v = inp.prompt(n_tail, frac)
        st, rid = pool.request_add(donor, n_shared, k, v, n_tail, sc.initial_pages)
        if st != B.GP_OK:
            assert st in (B.GP_ERR_NO_PAGES, B.GP_ERR_INVALID), st
            stats["refused"] += 1
            return False
        assert rid == slot, (rid, slot)
        inp.reset_slot(slot, frac)
        live[slot] = True
        pristine[slot] = True
        remaining[slot] = max(1, int(out_len * rng.uniform(0.02, 1.0))) if snapshot else out_len
        shift_at[slot] = int(remaining[slot] * rng.uniform(0.25, 0.75)) if sc.shift else -1
        if sc.groups and donor < 0:
            group_donor[slot % sc.groups] = slot
        stats["admitted"] += 1
        stats["shared_admissions"] += donor >= 0
        return True

    pristine = np.zeros(M, dtype=bool)
    try:
        # slots are filled in order: the lowest free slot is the one request_add hands out
        for slot in range(M):
            if not admit(slot, snapshot=not sc.groups):
                break
        ids_all = torch.arange(M, dtype=torch.int32, device=dev)
        out = torch.zeros((s.n_layers, M, s.n_q_heads, s.head_dim), dtype=torch.float32, device=dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        stream = torch.cuda.current_stream(device)
        ms = 0.0
        bytes_attn = 0.0
        tok0 = int(B.gp_debug_pool(pool.handle)[2][6])
        steps = 0
        last = None
        checked = {"retained": 0, "attention": 0, "rounds": 0}
        seen_actions: Dict[int, int] = {}
        t_wall = time.time()
        while steps < n_steps:
            c = min(chunk, n_steps - steps)
            ins = [inp.step() for _ in range(c)]
            acts = [torch.zeros(M, dtype=torch.int32, device=dev) for _ in range(c)]
            P, n = B.gp_debug_state(pool.handle, max(4, M))
            n_live = n[:M][live].astype(np.float64)
            bytes_attn += float(s.n_layers * s.token_bytes * (c * n_live.sum() + len(n_live) * c * (c + 1) / 2))
            # dead slots stay in the batch and are flagged invalid by the step (their rows are not touched)
            torch.cuda.synchronize(device)
            e0.record(stream)
            for j in range(c):
                q, k, v = ins[j]
                pool.decode_step(ids_all, q, k, v, out, acts[j])
            B.gp_async_join(pool.handle, pool.stream())
            e1.record(stream)
            torch.cuda.synchronize(device)
            ms += e0.elapsed_time(e1)
            steps += c
            a_all = torch.stack(acts).cpu().numpy()
            for a in np.unique(a_all):
                seen_actions[int(a)] = seen_actions.get(int(a), 0) + int((a_all == a).sum())
            stepped = np.isin(a_all, (B.GP_ACT_NONE, B.GP_ACT_GROW, B.GP_ACT_COMPRESS, B.GP_ACT_COMPRESS_FALLBACK, B.GP_ACT_SHRINK,
                                      B.GP_ACT_PENDING)).sum(axis=0)
            boundary = np.isin(a_all, (B.GP_ACT_GROW, B.GP_ACT_COMPRESS, B.GP_ACT_COMPRESS_FALLBACK, B.GP_ACT_SHRINK, B.GP_ACT_PENDING,
                                       B.GP_ACT_STALLED)).any(axis=0)
            pristine &= ~boundary
            last = (list(range(M)), ins[-1][0], out, a_all[-1])
            if check_every and (steps // chunk) % check_every == 0:
                got = check_invariants(pool, cfg, [int(x) for x in np.nonzero(live)[0]], rng, last)
                checked["retained"] += got["retained"]; checked["attention"] += got["attention"]; checked["rounds"] += 1
            # the scheduler: shifts, then releases and re-admissions
            remaining[live] -= stepped[live]
            if sc.shift:
                for slot in np.nonzero(live & (shift_at >= 0) & (remaining <= shift_at))[0]:
                    inp.fresh_direction(int(slot))
                    shift_at[slot] = -1
            stalled = live & (a_all[-1] == B.GP_ACT_STALLED)
            finished = live & (remaining <= 0) & ~stalled
            for slot in np.nonzero(stalled | finished)[0]:
                pool.release(int(slot))
                live[slot] = False
                stats["stalled" if stalled[slot] else "finished"] += 1
            for slot in np.nonzero(~live)[0]:          # lowest slots first, as request_add hands them out
                if not admit(int(slot), snapshot=False):
                    break
        got = check_invariants(pool, cfg, [int(x) for x in np.nonzero(live)[0]], rng, last, n_samples=12)
        checked["retained"] += got["retained"]; checked["attention"] += got["attention"]; checked["rounds"] += 1
        counters = B.gp_debug_pool(pool.handle)[2]
        tokens = int(counters[6]) - tok0
        P, n = B.gp_debug_state(pool.handle, max(4, M))
        res = {
            "config": sc.name, "layers": s.n_layers, "residents": int(live.sum()), "pool_pages": sc.n_pages,
            "pool_kv_gb": round(sc.n_pages * s.n_layers * s.token_bytes * b / 1e9, 1), "blob_gb": round(pool.nbytes / 1e9, 1),
            "steps": steps, "tokens": tokens, "device_ms": round(ms, 2), "ms_per_step": round(ms / steps, 4),
            "tokens_per_s": round(tokens / (ms * 1e-3), 1), "attention_gb_per_step": round(bytes_attn / steps / 1e9, 3),
            "attention_bytes_over_step_time_gbs": round(bytes_attn / (ms * 1e-3) / 1e9, 1),
            "mean_tokens_per_resident": round(float(n[:M][live].mean()), 1), "pages_in_use": int(P[:M][live].sum()),
            "events": {"grow": int(counters[0]), "compress": int(counters[1]), "fallback": int(counters[2]), "stalled": int(counters[3]),
                       "cow_pages": int(counters[4])},
            "scheduler": stats, "actions": seen_actions, "checked": checked, "async_boundary": async_boundary,
            "wall_s": round(time.time() - t_wall, 1),
        }
        if verbose:
            print(res)
        return res
    finally:
        pool.close()
