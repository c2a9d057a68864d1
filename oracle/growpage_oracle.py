"""Float64 CPU oracle for the GrowPage paged-decode path.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
path computes, written from the paper, and is the yardstick the CUDA library is
compared against.  Nothing in the product may import it: only the tests, the
smoke check and the benchmark's CPU-baseline legs do.  It shares no code with
the CUDA path; it consumes the same seeded bf16 inputs as plain data.

The method is a heuristic iteration, not a shortcut to a closed form, so the
oracle follows the paper's steps in the paper's order and notation:

  Sec. 3.1  Eq. 2 (p-coverage demand), Eq. 3 (subset-renormalised output),
            Eq. 5 / Theorem 1 (worst-case error and capacity)
  Sec. 3.2  Eq. 6 (dual EMA query summaries), Eq. 7 (working-set size and ratio),
            Eq. 8 (mean aggregation, Delta_t), decision rule Delta_t > tau
  Sec. 3.3  Eq. 9 (token score), Eq. 10 (block-local + global selection),
            compaction inside the existing allocation, Grow by one page
  Sec. 4    page pool, block tables, fallback to compression
  App. D.1  slot-wise summary storage, first-step initialisation, Eq. 12 (RMS
            calibration), RoPE at the current position, candidate set
  App. D.2  refcounted prefix blocks, copy-on-write targets, release after compaction

Only the attention output has a plain definition (dense softmax attention over
the retained tokens); it is written out as that definition.

Readings the paper leaves open are fixed here and listed in the repository's
design notes; the ones with no independent check are marked "parity unpinned":
  * trailing boundary check (the step that fills the last slot runs the boundary)
  * initial capacity max(initial_pages, floor(n_prompt / b) + 1)
  * all layers and KV heads take part in Eq. 8
  * simultaneous boundaries: grants, then copy-on-write targets, each in ascending
    request id; references to replaced pages are dropped after all compactions
  * every shared page below the last one is replaced at a compression
  * asynchronous decoding and compression (App. "Asynchronous Decoding and Compression"): the appendix lets
    requests that compress leave the batch while the others decode, and rejoin a later batch; requests that grow
    resume once the page is installed.  Reading taken when `async_boundary` is set: the whole boundary chain of a
    request (demand estimate, decision, grant or compaction) runs beside the pool's next decode step, so every
    request that reaches its boundary at step t, whatever the decision turns out to be, sits step t + 1 out
    (ACT_HELD) and decodes again from step t + 2; the step reports ACT_PENDING for it and the decision is read
    afterwards.  Each token meets exactly the state it meets in the synchronous order
  * Shrink (Eq. 13, App. "capacity-control policies"): evicts 2b tokens of C by the same Eq. 10 rule with the
    target |C| - 2b, hands the request's last page back once compaction is over, and is replaced by
    Compress & Hold when the capacity left, (P - 1) b tokens, would be under the minimum capacity
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Tuple

import numpy as np

# status / action codes of the oracle's own interface
OK = 0
ERR_INVALID = -1
ERR_NO_SLOT = -2
ERR_NO_PAGES = -3
ERR_STATE = -5

ACT_NONE = 0
ACT_GROW = 1
ACT_COMPRESS = 2
ACT_COMPRESS_FALLBACK = 3
ACT_SHRINK = 4
ACT_PENDING = 5        # asynchronous boundary work: boundary reached, decision under way
ACT_HELD = 6           # asynchronous boundary work: sitting out the step after its boundary
ACT_STALLED = -1
ACT_INVALID = -3


# =============================================================================
# Sec. 3.1: attention demand and subset approximation
# =============================================================================
def p_coverage_demand(a: np.ndarray, p: float) -> int:
    """Eq. 2 / Eq. 7: the smallest k whose k largest weights sum to at least p.

    Weights are sorted in descending order and accumulated one by one in float64.
    If rounding keeps the running sum below p to the end, k = len(a)."""
    k, _ = p_coverage_demand_with_margin(a, p)
    return k


def p_coverage_demand_with_margin(a: np.ndarray, p: float) -> Tuple[int, float]:
    """As p_coverage_demand; also returns how close the running sum came to p at the
    crossing, relative to p: min(|c_K - p|, |c_{K-1} - p|) / p."""
    a = np.asarray(a, dtype=np.float64)
    n = a.shape[0]
    if n == 0:
        return 0, math.inf
    srt = -np.sort(-a)
    c = np.cumsum(srt)                      # sequential accumulation
    hit = np.nonzero(c >= p)[0]
    k = int(hit[0]) + 1 if hit.size else n
    below = c[k - 2] if k >= 2 else 0.0
    margin = min(abs(c[k - 1] - p), abs(below - p)) / p
    return k, float(margin)


def entropy_ratio(a: np.ndarray) -> Tuple[float, float]:
    """The ablation's other working-set metric ("Dual-Timescale Signal Ablation"): Shannon entropy of the view's
    attention distribution, H = -sum a_i ln a_i (terms with a_i = 0 contribute nothing), and its ratio to the
    entropy ln |C| of the uniform distribution, which plays the part of r^x of Eq. 7.  The paper names the metric
    without a formula; the normalisation by ln |C| is this build's reading (it makes the ratio 1 for a flat view
    and 0 for a one-hot one, like K/|C|).  Returns (H, ratio)."""
    a = np.asarray(a, dtype=np.float64)
    nz = a[a > 0.0]
    H = float(-(nz * np.log(nz)).sum())
    return H, (H / math.log(a.shape[0]) if a.shape[0] > 1 else 0.0)


def subset_output(a: np.ndarray, v: np.ndarray, S) -> Tuple[np.ndarray, float]:
    """Eq. 3: output over the retained subset S with renormalised weights, and m(S)."""
    a = np.asarray(a, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    S = np.asarray(sorted(S), dtype=np.int64)
    m = float(a[S].sum())
    return (a[S] / m) @ v[S], m


def worst_case_error(a: np.ndarray, S, v_max: float) -> float:
    """Eq. 5: sup over ||v_i|| <= Vmax of ||o - o_hat(S)|| = 2 Vmax (1 - m(S))."""
    a = np.asarray(a, dtype=np.float64)
    S = np.asarray(sorted(S), dtype=np.int64)
    return 2.0 * v_max * (1.0 - float(a[S].sum()))


# =============================================================================
# Sec. 3.2 / App. D.1: summaries, calibration, RoPE
# =============================================================================
def ema_update(s_bar: np.ndarray, l_bar: np.ndarray, q: np.ndarray, started: bool,
               beta_s: float, beta_l: float) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 6 on the pre-RoPE query.  On the first decode step of a slot both states are
    set to the query itself, overwriting whatever the slot held (App. D.1)."""
    if not started:
        return q.copy(), q.copy()
    return beta_s * s_bar + (1.0 - beta_s) * q, beta_l * l_bar + (1.0 - beta_l) * q


def rms(z: np.ndarray) -> np.ndarray:
    """Root mean square over the head dimension, no epsilon."""
    return np.sqrt(np.mean(z * z, axis=-1))


def rms_calibrate(q_bar: np.ndarray, q: np.ndarray) -> np.ndarray:
    """Eq. 12: gamma = RMS(q_t) / RMS(q_bar); returns gamma * q_bar, per head.
    A summary of zero RMS is left as it is (gamma = 1)."""
    den = rms(q_bar)
    gamma = np.where(den > 0.0, rms(q) / np.where(den > 0.0, den, 1.0), 1.0)
    return gamma[..., None] * q_bar


def rope(x: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing (i, i + d/2), angle pos * theta^(-2i/d).
    theta == 0 switches the rotation off."""
    if theta == 0.0:
        return x
    d = x.shape[-1]
    half = d // 2
    inv = theta ** (-2.0 * np.arange(half, dtype=np.float64) / d)
    ang = float(pos) * inv
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


# =============================================================================
# dense attention (the one step with a plain definition)
# =============================================================================
def attention_decode(q_hat: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """softmax_i(q.K_i / sqrt(d)) . V over the n retained tokens, native GQA mapping
    (query head g reads KV head g // G).  q_hat [H_q][d], K, V [H_kv][n][d]."""
    h_q, d = q_hat.shape
    h_kv = K.shape[0]
    G = h_q // h_kv
    out = np.empty((h_q, d), dtype=np.float64)
    for g in range(h_q):
        h = g // G
        z = K[h] @ q_hat[g] / math.sqrt(d)
        w = np.exp(z - z.max())
        out[g] = (w @ V[h]) / w.sum()
    return out


def summary_attention(q_tilde: np.ndarray, Kc: np.ndarray) -> np.ndarray:
    """Attention of one temporal view over the candidate set of one KV head: each of the
    G query heads of the group takes its own softmax over C, the group mean is the head's
    distribution (Sec. 3.2; query heads keep their own KV head, App. D.1).  q_tilde [G][d], Kc [|C|][d]."""
    d = q_tilde.shape[-1]
    z = q_tilde @ Kc.T / math.sqrt(d)                    # [G][|C|]
    w = np.exp(z - z.max(axis=1, keepdims=True))
    A = w / w.sum(axis=1, keepdims=True)
    return A.mean(axis=0)


# =============================================================================
# Sec. 3.3: scores and selection
# =============================================================================
def token_scores(a_s: np.ndarray, a_l: np.ndarray) -> np.ndarray:
    """Eq. 9."""
    return np.maximum(a_s, a_l)


def _top(cands: np.ndarray, s: np.ndarray, k: int) -> Tuple[np.ndarray, float]:
    """The k best of `cands` ordered by (score descending, slot ascending), and the relative
    gap between the last one kept and the first one dropped."""
    if k <= 0 or cands.size == 0:
        return cands[:0], math.inf
    order = cands[np.lexsort((cands, -s[cands]))]
    keep = order[:k]
    if k >= order.size:
        return keep, math.inf
    last, nxt = s[order[k - 1]], s[order[k]]
    gap = (last - nxt) / last if last > 0.0 else 0.0
    return keep, float(gap)


def select_retained(s: np.ndarray, n_blocks: int, b: int, K_t: int, k_loc: int) -> Tuple[np.ndarray, float]:
    """Eq. 10 for one (layer, KV head).  Candidates are slots 0 .. len(s) - 1, block j is the
    candidates among slots [j*b, (j+1)*b): n_blocks blocks, the last of which is short when the
    protected window is smaller than a block.  Every block keeps its k' = min(k_loc, floor(K_t /
    n_blocks)) best slots; the global best of the remaining candidates fill up to K_t.  Returns the
    retained slots in ascending order and the smallest relative score gap met at any cut."""
    n_c = s.shape[0]
    assert (n_blocks - 1) * b < n_c <= n_blocks * b
    if K_t <= 0:
        return np.zeros(0, dtype=np.int64), math.inf
    k_prime = min(k_loc, K_t // n_blocks)
    margin = math.inf
    local = []
    for j in range(n_blocks):
        blk = np.arange(j * b, min((j + 1) * b, n_c), dtype=np.int64)
        keep, gap = _top(blk, s, k_prime)
        local.append(keep)
        margin = min(margin, gap)
    s_loc = np.concatenate(local) if local else np.zeros(0, dtype=np.int64)
    is_loc = np.zeros(n_c, dtype=bool)
    is_loc[s_loc] = True
    rest = np.nonzero(~is_loc)[0].astype(np.int64)
    glob, gap = _top(rest, s, K_t - s_loc.size)
    margin = min(margin, gap)
    return np.sort(np.concatenate([s_loc, glob])), margin


# =============================================================================
# the pool and the per-step state machine
# =============================================================================
def shrink_policy(delta: float, tau: float = 0.0, shrink_below: float = -0.005) -> int:
    """Eq. 13: Shrink when Delta_t < -0.005, Compress & Hold when -0.005 <= Delta_t <= 0, Grow by One Page when
    Delta_t > 0 (`tau` and `shrink_below` carry the two thresholds; growing wins if they are set to overlap)."""
    if delta > tau:
        return ACT_GROW
    if delta < shrink_below:
        return ACT_SHRINK
    return ACT_COMPRESS


def random_draw(seed: int, req: int, pos: int) -> float:
    """Uniform draw in [0, 1) of the random capacity-control policy for request `req` at absolute position
    `pos`: the SplitMix64 finaliser of seed + 0x9E3779B97F4A7C15 (req + 1) + 0xBF58476D1CE4E5B9 pos (mod 2^64),
    top 53 bits.  The paper only fixes the probability (0.7); the generator is this build's, stated in the
    C header so that both sides draw the same numbers."""
    m = (1 << 64) - 1
    z = (seed + 0x9E3779B97F4A7C15 * (req + 1) + 0xBF58476D1CE4E5B9 * pos) & m
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & m
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & m
    z ^= z >> 31
    return (z >> 11) / 9007199254740992.0


@dataclasses.dataclass
class OracleConfig:
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_pages: int
    max_pages_per_req: int
    page_size: int = 16
    max_requests: int = 512          # M (App. D.1)
    beta_s: float = 0.9              # Sec. 3.2
    beta_l: float = 0.999
    top_p: float = 0.99
    tau: float = 0.0
    recent_window: int = 16          # |R_t|: protected newest tokens; at most the page size and a divisor of it
    k_loc: int = 4                   # a quarter of a page, the paper's 64 of 256
    rope_theta: float = 0.0
    policy: int = 0                  # 0 demand (Eq. 8), 1 inverse, 2 random, 3 shrink (Eq. 13): the ablation's controls
    policy_seed: int = 0
    p_compress: float = 0.7
    shrink_below: float = -0.005     # Eq. 13: Shrink when Delta_t is under this
    min_capacity: int = 1024         # tokens; a Shrink that would leave less is a Compress & Hold
    async_boundary: bool = False     # boundary work of step t beside step t + 1; the request sits that step out
    demand_metric: int = 0           # 0: Top-p working set (Eq. 7); 1: attention entropy (the ablation's other metric)


class _Request:
    __slots__ = ("P", "n", "pos", "started", "n_pristine", "table", "K", "V", "tok", "S", "Lg", "bstep", "last_act")


@dataclasses.dataclass
class BoundaryInfo:
    req: int
    P: int
    n_c: int
    n_e: int = 0                            # candidates of Eq. 10: history minus the protected window (= n_c when R = b)
    a_s: Optional[np.ndarray] = None       # [L][H_kv][|C|]: the views over the demand support (Eq. 7)
    a_l: Optional[np.ndarray] = None
    e_s: Optional[np.ndarray] = None       # [L][H_kv][n_e]: the views over the eviction support (Eq. 9, Eq. 10)
    e_l: Optional[np.ndarray] = None
    K_s: Optional[np.ndarray] = None       # [L][H_kv] int
    K_l: Optional[np.ndarray] = None
    ws_margin: Optional[np.ndarray] = None  # [L][H_kv][2]
    H_s: Optional[np.ndarray] = None       # [L][H_kv] entropies of the two views (entropy metric only)
    H_l: Optional[np.ndarray] = None
    delta: float = 0.0
    want_grow: bool = False
    want_shrink: bool = False               # policy 3 only, and only where a Shrink is admissible
    action_near_tie: bool = False
    action: int = ACT_NONE
    keep: Dict[Tuple[int, int], np.ndarray] = dataclasses.field(default_factory=dict)      # slots kept
    keep_tok: Dict[Tuple[int, int], np.ndarray] = dataclasses.field(default_factory=dict)  # their token ids
    sel_margin: Dict[Tuple[int, int], float] = dataclasses.field(default_factory=dict)
    cow_pages: int = 0
    moved_tokens: int = 0                   # per request: sum over (l,h) of slots whose position changed


@dataclasses.dataclass
class StepRecord:
    req_ids: List[int]
    out: np.ndarray                         # [L][B][H_q][d]
    actions: np.ndarray                     # [B]
    boundary: Dict[int, BoundaryInfo]


class OraclePool:
    def __init__(self, cfg: OracleConfig):
        assert cfg.n_q_heads % cfg.n_kv_heads == 0
        assert 0 < cfg.recent_window <= cfg.page_size and cfg.page_size % cfg.recent_window == 0
        self.cfg = cfg
        self.G = cfg.n_q_heads // cfg.n_kv_heads
        self.refcount = np.zeros(cfg.n_pages, dtype=np.int64)
        self.free: List[int] = list(range(cfg.n_pages - 1, -1, -1))   # pop() hands out page 0 first
        self.requests: Dict[int, _Request] = {}
        self.serial = 0                                   # decode steps so far
        self.counters = {"grow": 0, "compress": 0, "fallback": 0, "shrink": 0, "stalled": 0, "cow_pages": 0,
                         "moved_rows": 0, "scored_tokens": 0}

    # ---- pool primitives ------------------------------------------------------
    def _take_page(self) -> int:
        page = self.free.pop()
        assert self.refcount[page] == 0
        self.refcount[page] = 1
        return page

    def _drop_ref(self, page: int) -> None:
        self.refcount[page] -= 1
        assert self.refcount[page] >= 0
        if self.refcount[page] == 0:
            self.free.append(page)

    # ---- admission / release (Sec. 4.1, App. D.1, App. D.2) ---------------------
    def request_add(self, share_from: int, n_shared_pages: int, k_tail: Optional[np.ndarray],
                    v_tail: Optional[np.ndarray], n_tail: int, initial_pages: int) -> Tuple[int, int]:
        """k_tail, v_tail float64 [L][n_tail][H_kv][d] in cache form.  Returns (status, request id)."""
        c = self.cfg
        b = c.page_size
        if n_tail < 0 or n_shared_pages < 0:
            return ERR_INVALID, -1
        donor = None
        if n_shared_pages > 0:
            donor = self.requests.get(share_from)
            if donor is None or n_shared_pages > donor.n_pristine:
                return ERR_INVALID, -1
        free_ids = [i for i in range(c.max_requests) if i not in self.requests]
        if not free_ids:
            return ERR_NO_SLOT, -1
        n_prompt = n_shared_pages * b + n_tail
        P = max(initial_pages, n_prompt // b + 1)
        if P > c.max_pages_per_req or P - n_shared_pages > len(self.free):
            return ERR_NO_PAGES, -1
        r = _Request()
        rid = free_ids[0]
        cap = c.max_pages_per_req * b
        r.K = np.zeros((c.n_layers, c.n_kv_heads, cap, c.head_dim))
        r.V = np.zeros((c.n_layers, c.n_kv_heads, cap, c.head_dim))
        r.tok = np.full((c.n_layers, c.n_kv_heads, cap), -1, dtype=np.int64)
        ns = n_shared_pages * b
        r.table = []
        if donor is not None:
            r.K[:, :, :ns] = donor.K[:, :, :ns]
            r.V[:, :, :ns] = donor.V[:, :, :ns]
            r.tok[:, :, :ns] = donor.tok[:, :, :ns]
            for j in range(n_shared_pages):
                page = donor.table[j]
                self.refcount[page] += 1
                r.table.append(page)
        if n_tail:
            r.K[:, :, ns:n_prompt] = np.transpose(k_tail, (0, 2, 1, 3))
            r.V[:, :, ns:n_prompt] = np.transpose(v_tail, (0, 2, 1, 3))
            r.tok[:, :, ns:n_prompt] = np.arange(ns, n_prompt)
        while len(r.table) < P:
            r.table.append(self._take_page())
        r.P, r.n, r.pos, r.started = P, n_prompt, n_prompt, False
        r.bstep, r.last_act = None, ACT_NONE
        r.n_pristine = n_prompt // b                     # only full prompt pages can be shared
        r.S = np.zeros((c.n_layers, c.n_q_heads, c.head_dim))
        r.Lg = np.zeros((c.n_layers, c.n_q_heads, c.head_dim))
        self.requests[rid] = r
        return OK, rid

    def release(self, rid: int) -> int:
        r = self.requests.pop(rid, None)
        if r is None:
            return ERR_INVALID
        for page in r.table:
            self._drop_ref(page)
        return OK

    # ---- one decode step --------------------------------------------------------
    def decode_step(self, req_ids, q, k, v, overrides=None) -> StepRecord:
        rec = self.step_compute(req_ids, q, k, v)
        self.step_apply(rec, overrides)
        return rec

    def step_compute(self, req_ids, q: np.ndarray, k: np.ndarray, v: np.ndarray) -> StepRecord:
        """q float64 [L][B][H_q][d], k, v float64 [L][B][H_kv][d].  Runs append, attention and
        the summary update of every request, and at capacity boundaries the demand estimate.
        Page-level actions are taken by step_apply."""
        c = self.cfg
        b = c.page_size
        B = len(req_ids)
        out = np.zeros((c.n_layers, B, c.n_q_heads, c.head_dim))
        actions = np.zeros(B, dtype=np.int64)
        boundary: Dict[int, BoundaryInfo] = {}
        seen = set()
        for i, rid in enumerate(req_ids):
            r = self.requests.get(int(rid))
            if r is None or rid in seen:
                actions[i] = ACT_INVALID
                continue
            seen.add(rid)
            if c.async_boundary and r.bstep == self.serial - 1:
                actions[i] = ACT_HELD                # its boundary work runs beside this step: not stepped
                continue
            if r.n >= r.P * b:                       # stalled earlier and never resolved
                actions[i] = ACT_STALLED
                continue
            t = r.pos
            # 1. append (Sec. 3.3 "Grow by One Page": decoding continues into the free slots)
            r.K[:, :, r.n] = k[:, i]
            r.V[:, :, r.n] = v[:, i]
            r.tok[:, :, r.n] = t
            r.n += 1
            r.pos += 1
            # 2. attention over every retained token, the new one included
            for l in range(c.n_layers):
                q_hat = rope(q[l, i], t, c.rope_theta)
                out[l, i] = attention_decode(q_hat, r.K[l, :, :r.n], r.V[l, :, :r.n])
            # 3. Eq. 6 on the un-rotated query
            r.S, r.Lg = ema_update(r.S, r.Lg, q[:, i], r.started, c.beta_s, c.beta_l)
            r.started = True
            # 4. capacity boundary: the allocation is exhausted (Sec. 3.3)
            if r.n == r.P * b:
                boundary[int(rid)] = self._demand(int(rid), r, q[:, i], t)
                r.bstep = self.serial
                if c.async_boundary:
                    actions[i] = ACT_PENDING
        self.serial += 1
        return StepRecord([int(x) for x in req_ids], out, actions, boundary)

    def _demand(self, rid: int, r: _Request, q: np.ndarray, t: int) -> BoundaryInfo:
        """App. D.1 "Demand estimation at capacity boundaries" and Eq. 7, Eq. 8."""
        c = self.cfg
        b = c.page_size
        G = self.G
        n_c = (r.P - 1) * b                          # Eq. 7's support: history minus the most recent block
        n_e = r.P * b - c.recent_window              # Eq. 10's candidates: history minus the protected window
        info = BoundaryInfo(req=rid, P=r.P, n_c=n_c, n_e=n_e)
        if n_c == 0:
            info.want_grow = True
            return info
        L, H = c.n_layers, c.n_kv_heads
        info.a_s = np.empty((L, H, n_c))
        info.a_l = np.empty((L, H, n_c))
        info.K_s = np.empty((L, H), dtype=np.int64)
        info.K_l = np.empty((L, H), dtype=np.int64)
        info.ws_margin = np.empty((L, H, 2))
        use_entropy = c.demand_metric == 1
        if use_entropy:
            info.H_s, info.H_l = np.empty((L, H)), np.empty((L, H))
        two = n_e != n_c                             # R < b: the two supports differ, each has its own softmax
        info.e_s = np.empty((L, H, n_e)) if two else info.a_s
        info.e_l = np.empty((L, H, n_e)) if two else info.a_l
        for l in range(L):
            qs = rope(rms_calibrate(r.S[l], q[l]), t, c.rope_theta)       # Eq. 12, then RoPE at
            ql = rope(rms_calibrate(r.Lg[l], q[l]), t, c.rope_theta)      # the current position
            for h in range(H):
                Kc = r.K[l, h, :n_c]
                info.a_s[l, h] = summary_attention(qs[h * G:(h + 1) * G], Kc)
                info.a_l[l, h] = summary_attention(ql[h * G:(h + 1) * G], Kc)
                if two:
                    info.e_s[l, h] = summary_attention(qs[h * G:(h + 1) * G], r.K[l, h, :n_e])
                    info.e_l[l, h] = summary_attention(ql[h * G:(h + 1) * G], r.K[l, h, :n_e])
                if use_entropy:
                    info.H_s[l, h], info.H_l[l, h] = entropy_ratio(info.a_s[l, h])[0], entropy_ratio(info.a_l[l, h])[0]
                    info.K_s[l, h] = info.K_l[l, h] = 0
                    info.ws_margin[l, h] = math.inf
                    continue
                info.K_s[l, h], info.ws_margin[l, h, 0] = p_coverage_demand_with_margin(info.a_s[l, h], c.top_p)
                info.K_l[l, h], info.ws_margin[l, h, 1] = p_coverage_demand_with_margin(info.a_l[l, h], c.top_p)
        # Eq. 8 with a candidate set common to all heads: the mean of K/|C| is sum(K)/(N |C|),
        # so Delta is one division of exact integers and its sign is exact.
        num = int(info.K_s.sum()) - int(info.K_l.sum())
        info.delta = num / float(L * H * n_c)
        if use_entropy:
            # the same mean aggregation with H / ln |C| in the place of K / |C|; the differences are summed unit by
            # unit in (layer, head) order
            acc = 0.0
            for l in range(L):
                for h in range(H):
                    acc += info.H_s[l, h] - info.H_l[l, h]
            info.delta = acc / (float(L * H) * math.log(n_c)) if n_c > 1 else 0.0
            info.action_near_tie = abs(info.delta - c.tau) < 1e-12
        info.want_grow = info.delta > c.tau
        if c.policy == 1:            # inverse: grows when Delta <= tau, compresses when Delta > tau
            info.want_grow = not info.want_grow
        elif c.policy == 2:          # random: Compress & Hold with probability p_compress, whatever Delta says
            info.want_grow = not (random_draw(c.policy_seed, rid, r.pos - 1) < c.p_compress)
            return info              # no working-set near-tie can change a coin
        # Eq. 13: a Shrink needs two blocks of candidates and must leave the minimum capacity
        can_shrink = c.policy == 3 and r.P >= 3 and (r.P - 1) * b >= c.min_capacity and n_e > 2 * b
        if c.policy == 3:
            info.want_shrink = can_shrink and shrink_policy(info.delta, c.tau, c.shrink_below) == ACT_SHRINK
        # could a +-1 change of near-tied working-set sizes change the decision?
        near = int((info.ws_margin < 1e-6).sum())
        if near:
            d_lo, d_hi = (num - near) / float(L * H * n_c), (num + near) / float(L * H * n_c)
            info.action_near_tie = (d_lo > c.tau) != (d_hi > c.tau)
            if can_shrink:
                info.action_near_tie |= (d_lo < c.shrink_below) != (d_hi < c.shrink_below)
        return info

    def step_apply(self, rec: StepRecord, overrides: Optional[dict] = None) -> None:
        """Page-level actions for the requests at a boundary (Sec. 3.3, Sec. 4.2, App. D.2).
        `overrides[rid]` may carry 'want_grow' (bool) and 'keep' {(l,h): slots} to adopt a
        choice inside a certified near-tie."""
        c = self.cfg
        b = c.page_size
        overrides = overrides or {}
        order = sorted(rec.boundary)
        index_of: Dict[int, int] = {}
        for i, rid in enumerate(rec.req_ids):           # a repeated id is stepped at its first batch slot only
            index_of.setdefault(rid, i)
        # pass 1: grants, ascending request id
        compress: List[int] = []
        for rid in order:
            info = rec.boundary[rid]
            r = self.requests[rid]
            want = overrides.get(rid, {}).get("want_grow", info.want_grow)
            info.want_grow = bool(want)
            info.want_shrink = bool(overrides.get(rid, {}).get("want_shrink", info.want_shrink)) and not want
            self.counters["scored_tokens"] += info.n_c
            if want and r.P < c.max_pages_per_req and self.free:
                r.table.append(self._take_page())
                r.P += 1
                info.action = ACT_GROW
                self.counters["grow"] += 1
            elif info.n_c == 0:
                info.action = ACT_STALLED        # one page, nothing to evict, no page to be had
                self.counters["stalled"] += 1
            else:
                info.action = ACT_COMPRESS_FALLBACK if want else (ACT_SHRINK if info.want_shrink else ACT_COMPRESS)
                compress.append(rid)
        # pass 2: copy-on-write targets, ascending request id, then selection and compaction
        released: List[int] = []
        for rid in compress:
            info = rec.boundary[rid]
            r = self.requests[rid]
            shared = [j for j in range(r.P - 1) if self.refcount[r.table[j]] > 1]
            if len(shared) > len(self.free):
                info.action = ACT_STALLED        # the scheduler's preemption case (App. D.2)
                self.counters["stalled"] += 1
                continue
            for j in shared:
                released.append(r.table[j])
                r.table[j] = self._take_page()
            info.cow_pages = len(shared)
            self.counters["cow_pages"] += len(shared)
            kind = {ACT_COMPRESS_FALLBACK: "fallback", ACT_SHRINK: "shrink"}.get(info.action, "compress")
            self.counters[kind] += 1
            n_evict = 2 * b if info.action == ACT_SHRINK else b
            self._compress(r, info, overrides.get(rid, {}).get("keep", {}), set(shared), n_evict)
            r.n_pristine = 0
            if info.action == ACT_SHRINK:        # Eq. 13: one physical page goes back to the pool
                released.append(r.table.pop())
                r.P -= 1
        # pass 3: the replaced pages lose this request's reference once compaction is over
        for page in released:
            self._drop_ref(page)
        for rid in order:
            self.requests[rid].last_act = rec.boundary[rid].action
            if not c.async_boundary:                    # the asynchronous step has reported ACT_PENDING already
                rec.actions[index_of[rid]] = rec.boundary[rid].action

    def _compress(self, r: _Request, info: BoundaryInfo, keep_override: dict, cow: set, n_evict: int) -> None:
        """Eq. 9, Eq. 10 and the compaction, independently for every (layer, KV head).  `n_evict` tokens of C
        go: one page worth at a compression (the target is (P-1) b tokens, the protected page included), two
        at a Shrink."""
        c = self.cfg
        b = c.page_size
        R = c.recent_window
        n_c = info.n_e                       # the candidates: everything but the protected window
        K_t = n_c - n_evict                  # (P - 1) b - |R| at a compression: one block of slots is freed
        n_blocks = -(-n_c // b)
        moved = 0
        for l in range(c.n_layers):
            for h in range(c.n_kv_heads):
                if (l, h) in keep_override:
                    keep = np.sort(np.asarray(keep_override[(l, h)], dtype=np.int64))
                    margin = 0.0
                else:
                    s = token_scores(info.e_s[l, h], info.e_l[l, h])
                    keep, margin = select_retained(s, n_blocks, b, K_t, c.k_loc)
                assert keep.size == K_t
                info.keep[(l, h)] = keep
                info.keep_tok[(l, h)] = r.tok[l, h, keep].copy()
                info.sel_margin[(l, h)] = margin
                # retained history in slot order, then the protected page
                src = np.concatenate([keep, np.arange(n_c, n_c + R, dtype=np.int64)])
                dst = np.arange(src.size)
                moved += int(((src != dst) | np.isin(src // b, list(cow))).sum())
                r.K[l, h, :src.size] = r.K[l, h, src]
                r.V[l, h, :src.size] = r.V[l, h, src]
                r.tok[l, h, :src.size] = r.tok[l, h, src]
                r.tok[l, h, src.size:r.P * b] = -1
        r.n = K_t + R
        info.moved_tokens = moved
        self.counters["moved_rows"] += moved

    # ---- introspection -----------------------------------------------------------
    def retained(self, rid: int, l: int, h: int) -> np.ndarray:
        r = self.requests[rid]
        return r.tok[l, h, :r.n].copy()

    def summaries(self, rid: int) -> np.ndarray:
        """[L][2][H_q][d]: short then long."""
        r = self.requests[rid]
        return np.stack([r.S, r.Lg], axis=1)

    def request_state(self, rid: int) -> Tuple[int, int, int, List[int]]:
        r = self.requests[rid]
        return r.P, r.n, r.pos, list(r.table)

    def n_free(self) -> int:
        return len(self.free)

    def boundary_outcome(self, rid: int) -> Tuple[int, int]:
        """(decision, step number) of the request's most recent boundary; (ACT_NONE, -1) before the first."""
        r = self.requests[rid]
        return (ACT_NONE, -1) if r.bstep is None else (r.last_act, r.bstep)
