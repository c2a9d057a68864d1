"""Seeded synthetic inputs for the GrowPage decode path.

This module only draws random numbers and shapes them; it contains none of the
method's arithmetic (no attention, no summaries, no scoring).  Both the CUDA
path and the CPU checker consume its arrays as plain data, so the two sides see
bit-identical bf16 inputs.

The inputs stand in for the paper's reasoning workloads (long outputs, budgets
of a few thousand tokens, demand that differs between requests and drifts inside
a request; Sec. 2, Fig. 2, Fig. 3, Tab. 5).  Only that shape is reproduced:

* per (layer, KV head) a fixed unit direction ``u``;
* token ``j`` of a request is a heavy hitter with probability ``f_r``; a heavy
  key is ``4*u + 0.1*N(0,I)``, any other key is ``N(0,I)``; values are ``N(0,I)``;
* the query of a decode step is ``2*u + N(0,I)`` with independent noise per
  query head (KV head ``g // G``);
* everything is rounded to bf16 (round to nearest even) before anyone sees it.

Random numbers come from a counter-based generator (Philox) keyed by
``(seed, stream kind, request, block)``, so the inputs of one request, or of one
block of its decode steps, can be regenerated without touching the others.

Arrays are returned as ``uint16`` holding raw bf16 bit patterns.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Tuple

import numpy as np

STEP_BLOCK = 64  # decode steps generated per Philox key

_KIND_DIRECTION = 1
_KIND_REQUEST = 2
_KIND_PROMPT = 3
_KIND_STEPS = 4
_KIND_SHIFT = 5


# ----------------------------------------------------------------------------
# bf16 helpers (storage format only)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """bf16 values are exactly representable in float64."""
    return bf16_bits_to_f32(b).astype(np.float64)


def _rng(seed: int, kind: int, a: int = 0, b: int = 0) -> np.random.Generator:
    key = ((seed & 0xFFFFFFFF) << 96) | ((kind & 0xFF) << 88) | ((a & 0xFFFFFFFF) << 40) | (b & 0xFFFFFFFFFF)
    return np.random.Generator(np.random.Philox(key=key))


# ----------------------------------------------------------------------------
# workload description
# ----------------------------------------------------------------------------
@dataclasses.dataclass
class Shape:
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int = 16

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def token_bytes(self) -> int:
        """bf16 K and V of one token over all KV heads of one layer."""
        return 2 * self.n_kv_heads * self.head_dim * 2


@dataclasses.dataclass
class RequestSpec:
    index: int               # position in the workload's request list
    prompt_len: int
    n_steps: int             # decode steps (output tokens)
    heavy_frac: float        # f_r
    share_group: int = -1    # requests with the same group >= 0 share their prompt
    shift_step: int = -1     # decode step at which the query direction rotates (-1: never)


@dataclasses.dataclass
class Workload:
    name: str
    seed: int
    shape: Shape
    requests: List[RequestSpec]
    n_resident: int               # concurrent requests
    initial_pages: int            # the config's initial budget, 0 = prompt pages + 1
    max_pages_per_req: int        # per-request cap (also the page-table stride)
    n_pages: int                  # physical pages in the pool
    k_loc: int = 4
    note: str = ""

    def stream(self, req: RequestSpec) -> "RequestStream":
        return RequestStream(self, req)

    def directions(self) -> np.ndarray:
        """u[l][h_kv][d] float32 unit vectors, fixed per workload."""
        s = self.shape
        g = _rng(self.seed, _KIND_DIRECTION)
        u = g.standard_normal((s.n_layers, s.n_kv_heads, s.head_dim), dtype=np.float32)
        u /= np.linalg.norm(u, axis=-1, keepdims=True)
        return u


class RequestStream:
    """All inputs of one request, regenerable on their own."""

    def __init__(self, wl: Workload, req: RequestSpec):
        self.wl = wl
        self.req = req
        self.shape = wl.shape
        self._u = wl.directions()
        if req.shift_step >= 0:
            s = wl.shape
            g = _rng(wl.seed, _KIND_SHIFT, req.index)
            u2 = g.standard_normal((s.n_layers, s.n_kv_heads, s.head_dim), dtype=np.float32)
            u2 /= np.linalg.norm(u2, axis=-1, keepdims=True)
            self._u_shifted = u2
        else:
            self._u_shifted = None
        self._prompt_owner = req.index
        if req.share_group >= 0:
            # every member of a sharing group reads the prompt of the group's first request
            first = min(r.index for r in wl.requests if r.share_group == req.share_group)
            self._prompt_owner = first

    # -- prompt ---------------------------------------------------------------
    def prompt_kv(self) -> Tuple[np.ndarray, np.ndarray]:
        """K, V of the prompt in cache form: uint16 [L][n_prompt][H_kv][d]."""
        s = self.shape
        n = self.req.prompt_len
        owner = self._prompt_owner
        g = _rng(self.wl.seed, _KIND_PROMPT, owner)
        f = self.wl.requests[owner].heavy_frac
        heavy = g.random(n) < f
        k = g.standard_normal((s.n_layers, n, s.n_kv_heads, s.head_dim), dtype=np.float32)
        v = g.standard_normal((s.n_layers, n, s.n_kv_heads, s.head_dim), dtype=np.float32)
        if heavy.any():
            k[:, heavy] = 4.0 * self._u[:, None, :, :] + 0.1 * k[:, heavy]
        return f32_to_bf16_bits(k), f32_to_bf16_bits(v)

    # -- decode steps -----------------------------------------------------------
    def _block(self, blk: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        s = self.shape
        t0 = blk * STEP_BLOCK
        g = _rng(self.wl.seed, _KIND_STEPS, self.req.index, blk)
        heavy = g.random(STEP_BLOCK) < self.req.heavy_frac
        q = g.standard_normal((STEP_BLOCK, s.n_layers, s.n_q_heads, s.head_dim), dtype=np.float32)
        k = g.standard_normal((STEP_BLOCK, s.n_layers, s.n_kv_heads, s.head_dim), dtype=np.float32)
        v = g.standard_normal((STEP_BLOCK, s.n_layers, s.n_kv_heads, s.head_dim), dtype=np.float32)
        steps = np.arange(t0, t0 + STEP_BLOCK)
        shifted = (steps >= self.req.shift_step) if self.req.shift_step >= 0 else np.zeros(STEP_BLOCK, bool)
        for sel, u in ((~shifted, self._u), (shifted, self._u_shifted)):
            if u is None or not sel.any():
                continue
            uq = np.repeat(u, s.group, axis=1)                       # [L][H_q][d]
            q[sel] += 2.0 * uq[None]
            hs = sel & heavy
            if hs.any():
                k[hs] = 4.0 * u[None] + 0.1 * k[hs]
        return f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v)

    def steps(self, t0: int, t1: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """q uint16 [t1-t0][L][H_q][d]; k, v uint16 [t1-t0][L][H_kv][d] for decode steps t0..t1-1."""
        assert 0 <= t0 <= t1
        qs, ks, vs = [], [], []
        for blk in range(t0 // STEP_BLOCK, (max(t1, t0 + 1) - 1) // STEP_BLOCK + 1):
            q, k, v = self._block(blk)
            lo = max(t0 - blk * STEP_BLOCK, 0)
            hi = min(t1 - blk * STEP_BLOCK, STEP_BLOCK)
            if hi > lo:
                qs.append(q[lo:hi]); ks.append(k[lo:hi]); vs.append(v[lo:hi])
        if not qs:
            s = self.shape
            z = lambda h: np.zeros((0, s.n_layers, h, s.head_dim), np.uint16)
            return z(s.n_q_heads), z(s.n_kv_heads), z(s.n_kv_heads)
        return np.concatenate(qs), np.concatenate(ks), np.concatenate(vs)


# ----------------------------------------------------------------------------
# the five configurations (full size and reduced "parity" size)
# ----------------------------------------------------------------------------
def _log_uniform(g: np.random.Generator, lo: float, hi: float, size=None):
    return np.exp(g.uniform(math.log(lo), math.log(hi), size))


def _pages(tokens: int, b: int) -> int:
    return -(-tokens // b)


def tiny(seed: int = 0) -> Workload:
    """Config 1: 1 layer, 4 requests, 8/2 heads, d 64, prompt 64, 256 steps, budget 4, cap 16."""
    shape = Shape(1, 8, 2, 64)
    reqs = [RequestSpec(i, 64, 256, 0.05) for i in range(4)]
    return Workload("tiny", seed, shape, reqs, n_resident=4, initial_pages=4,
                    max_pages_per_req=16, n_pages=4 * 16 + 8)


def layer8b(seed: int = 1, n_requests: int = 64, n_steps: int = 4096,
            prompt_range: Tuple[int, int] = (128, 1024)) -> Workload:
    """Config 2: one Qwen3-8B-shaped layer, 64 requests, prompts U[128,1024], 4096 steps,
    heavy-hitter fraction log-uniform in [0.5%, 20%]."""
    shape = Shape(1, 32, 8, 128)
    g = _rng(seed, _KIND_REQUEST)
    plen = g.integers(prompt_range[0], prompt_range[1] + 1, n_requests)
    frac = _log_uniform(g, 0.005, 0.2, n_requests)
    reqs = [RequestSpec(i, int(plen[i]), n_steps, float(frac[i])) for i in range(n_requests)]
    cap = _pages(prompt_range[1], 16) + 1 + _pages(n_steps, 16)
    cap = -(-cap // 64) * 64
    return Workload("qwen3-8b-layer", seed, shape, reqs, n_resident=n_requests, initial_pages=0,
                    max_pages_per_req=cap, n_pages=n_requests * cap,
                    note="cap never binds: prompt pages + 1 + one page per boundary")


def stack8b_resident(seed: int = 2, n_layers: int = 36, n_requests: int = 16, n_steps: int = 96,
                     prompt_range: Tuple[int, int] = (400, 1000)) -> Workload:
    """The config-3 shape (36 Qwen3-8B-shaped layers) with every request resident from the first step and a
    pool that never runs dry: the multi-layer shape without the continuous batching, for measurements."""
    shape = Shape(n_layers, 32, 8, 128)
    g = _rng(seed, _KIND_REQUEST)
    plen = g.integers(prompt_range[0], prompt_range[1] + 1, n_requests)
    frac = _log_uniform(g, 0.005, 0.2, n_requests)
    reqs = [RequestSpec(i, int(plen[i]), n_steps, float(frac[i])) for i in range(n_requests)]
    cap = _pages(prompt_range[1], 16) + 1 + _pages(n_steps, 16)
    return Workload("qwen3-8b-stack-resident", seed, shape, reqs, n_resident=n_requests, initial_pages=0,
                    max_pages_per_req=cap, n_pages=n_requests * cap, note="cap never binds")


def stack8b(seed: int = 2, n_layers: int = 36, n_resident: int = 256, n_total: int = 1024,
            out_range: Tuple[int, int] = (1024, 16384), pool_bytes: float = 120e9,
            prompt_range: Tuple[int, int] = (128, 1024)) -> Workload:
    """Config 3: 36-layer Qwen3-8B-shaped stack, continuous batching under pool pressure."""
    shape = Shape(n_layers, 32, 8, 128)
    g = _rng(seed, _KIND_REQUEST)
    plen = g.integers(prompt_range[0], prompt_range[1] + 1, n_total)
    outs = _log_uniform(g, out_range[0], out_range[1], n_total).astype(np.int64)
    frac = _log_uniform(g, 0.005, 0.2, n_total)
    reqs = [RequestSpec(i, int(plen[i]), int(outs[i]), float(frac[i])) for i in range(n_total)]
    page_bytes = shape.n_layers * shape.token_bytes * shape.page_size
    n_pages = int(pool_bytes // page_bytes)
    cap = _pages(prompt_range[1] + out_range[1], 16) + 1
    return Workload("qwen3-8b-stack", seed, shape, reqs, n_resident=n_resident, initial_pages=0,
                    max_pages_per_req=cap, n_pages=n_pages,
                    note="no per-request cap below the longest possible sequence; the pool is the limit")


def stack32b(seed: int = 3, n_layers: int = 64, n_requests: int = 128,
             out_range: Tuple[int, int] = (2048, 32768), pool_bytes: float = 120e9,
             prompt_range: Tuple[int, int] = (128, 1024)) -> Workload:
    """Config 4: Qwen3-32B-shaped stack (64 q / 8 kv heads) with a mid-generation demand shift."""
    shape = Shape(n_layers, 64, 8, 128)
    g = _rng(seed, _KIND_REQUEST)
    plen = g.integers(prompt_range[0], prompt_range[1] + 1, n_requests)
    outs = _log_uniform(g, out_range[0], out_range[1], n_requests).astype(np.int64)
    frac = _log_uniform(g, 0.005, 0.2, n_requests)
    where = g.uniform(0.25, 0.75, n_requests)
    reqs = [RequestSpec(i, int(plen[i]), int(outs[i]), float(frac[i]),
                        shift_step=int(where[i] * outs[i])) for i in range(n_requests)]
    page_bytes = shape.n_layers * shape.token_bytes * shape.page_size
    n_pages = int(pool_bytes // page_bytes)
    cap = _pages(prompt_range[1] + out_range[1], 16) + 1
    return Workload("qwen3-32b-stack", seed, shape, reqs, n_resident=n_requests, initial_pages=0,
                    max_pages_per_req=cap, n_pages=n_pages)


def prefix_stress(seed: int = 4, n_groups: int = 16, group_size: int = 16, prompt_len: int = 2048,
                  n_steps: int = 8192, initial_pages: int = 8, extra_pages: int = 8) -> Workload:
    """Config 5: groups of requests sharing a refcounted prompt; copy-on-write at first compaction."""
    shape = Shape(1, 32, 8, 128)
    reqs = []
    for gidx in range(n_groups):
        for j in range(group_size):
            reqs.append(RequestSpec(gidx * group_size + j, prompt_len, n_steps, 0.05, share_group=gidx))
    p0 = max(initial_pages, prompt_len // 16 + 1)
    n_req = n_groups * group_size
    cap = p0 + _pages(n_steps, 16)
    n_pages = n_groups * _pages(prompt_len, 16) + n_req * (p0 + extra_pages)
    return Workload("prefix-stress", seed, shape, reqs, n_resident=n_req, initial_pages=initial_pages,
                    max_pages_per_req=cap, n_pages=n_pages)


def parity_instance(config: int) -> Workload:
    """Reduced instances of configs 2-5 that the float64 CPU checker finishes in seconds to minutes."""
    if config == 1:
        return tiny()
    if config == 2:
        return layer8b(n_requests=8, n_steps=320, prompt_range=(128, 512))
    if config == 3:
        # 12 layers, 8 residents of 14 requests, outputs up to 320 tokens; same pressure as the full config: the
        # pool holds far less than the residents ask for, so grants are refused, requests stall and are replaced
        wl = stack8b(n_layers=12, n_resident=8, n_total=14, out_range=(64, 320), prompt_range=(64, 256))
        wl.n_pages = 8 * 14
        return wl
    if config == 4:
        # 4 layers of the 64-query-head shape, 6 requests that run hundreds of steps past their direction shift
        wl = stack32b(n_layers=4, n_requests=6, out_range=(256, 640), prompt_range=(64, 192))
        wl.n_pages = 6 * 56
        return wl
    if config == 5:
        # 4 groups of 4 on a shared 256-token prompt, 512 steps
        return prefix_stress(n_groups=4, group_size=4, prompt_len=256, n_steps=512, initial_pages=8,
                             extra_pages=2)
    raise ValueError(config)


def batch_step_inputs(streams: List[RequestStream], step_of: List[int]) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Gather one decode step for a batch: q uint16 [L][B][H_q][d], k, v uint16 [L][B][H_kv][d].
    ``step_of[i]`` is the decode-step index of ``streams[i]``."""
    qs, ks, vs = [], [], []
    for st, t in zip(streams, step_of):
        q, k, v = st.steps(t, t + 1)
        qs.append(q[0]); ks.append(k[0]); vs.append(v[0])
    return (np.ascontiguousarray(np.stack(qs, axis=1)),
            np.ascontiguousarray(np.stack(ks, axis=1)),
            np.ascontiguousarray(np.stack(vs, axis=1)))
