"""Plays the serving scheduler above the pool: admits requests of a synthetic workload, builds
each decode step's batch, and releases requests that finish or stall (continuous batching).

It drives anything with the pool interface (`request_add`, `decode_step`-style stepping,
`release`) and holds none of the method's arithmetic; the tests drive the CUDA pool and the CPU
checker with the same sequence of operations.
"""
from __future__ import annotations

import collections
import dataclasses
from typing import Dict, List, Optional, Tuple

import numpy as np

from . import workload as W


@dataclasses.dataclass
class AddOp:
    spec: W.RequestSpec
    share_from_spec: int          # index of the donor request in the workload, -1 for none
    n_shared_pages: int
    k_tail: Optional[np.ndarray]  # uint16 [L][n_tail][H_kv][d]
    v_tail: Optional[np.ndarray]
    n_tail: int
    initial_pages: int


@dataclasses.dataclass
class _Resident:
    spec: W.RequestSpec
    rid: int
    stream: W.RequestStream
    step: int = 0
    cache_blk: int = -1
    cache: Optional[Tuple[np.ndarray, np.ndarray, np.ndarray]] = None


HELD = 6                 # action code of a request that sat a step out (asynchronous boundary work)


class Scheduler:
    def __init__(self, wl: W.Workload, only=None):
        """`only`: indices of the workload's requests to run (default: all of them)."""
        self.wl = wl
        self.pending = collections.deque(wl.requests if only is None else [wl.requests[i] for i in only])
        self.resident: Dict[int, _Resident] = {}        # spec index -> state
        self.finished: List[int] = []
        self.stalled: List[int] = []
        self.tokens = 0

    # ---- admission ------------------------------------------------------------
    def next_admission(self) -> Optional[AddOp]:
        """The next pending request if a resident slot is open, else None."""
        if not self.pending or len(self.resident) >= self.wl.n_resident:
            return None
        spec = self.pending[0]
        b = self.wl.shape.page_size
        st = self.wl.stream(spec)
        k, v = st.prompt_kv()
        donor = -1
        n_shared = 0
        if spec.share_group >= 0:
            for idx, res in self.resident.items():
                if res.spec.share_group == spec.share_group and res.step == 0:
                    donor, n_shared = idx, spec.prompt_len // b
                    break
        ns = n_shared * b
        n_tail = spec.prompt_len - ns
        kt = np.ascontiguousarray(k[:, ns:]) if n_tail else None
        vt = np.ascontiguousarray(v[:, ns:]) if n_tail else None
        return AddOp(spec, donor, n_shared, kt, vt, n_tail, self.wl.initial_pages)

    def admitted(self, op: AddOp, rid: int) -> None:
        assert self.pending[0] is op.spec
        self.pending.popleft()
        self.resident[op.spec.index] = _Resident(op.spec, rid, self.wl.stream(op.spec))

    def rid_of(self, spec_index: int) -> int:
        return self.resident[spec_index].rid

    # ---- stepping -----------------------------------------------------------------
    def batch(self) -> Tuple[List[int], List[int], np.ndarray, np.ndarray, np.ndarray]:
        """(spec indices, request ids, q, k, v) of the next decode step; arrays are uint16 bf16
        bits, q [L][B][H_q][d], k and v [L][B][H_kv][d]."""
        specs = sorted(self.resident)
        rids, qs, ks, vs = [], [], [], []
        for idx in specs:
            res = self.resident[idx]
            blk = res.step // W.STEP_BLOCK
            if res.cache_blk != blk:
                res.cache = res.stream.steps(blk * W.STEP_BLOCK, (blk + 1) * W.STEP_BLOCK)
                res.cache_blk = blk
            o = res.step - blk * W.STEP_BLOCK
            rids.append(res.rid)
            qs.append(res.cache[0][o]); ks.append(res.cache[1][o]); vs.append(res.cache[2][o])
        q = np.ascontiguousarray(np.stack(qs, axis=1))
        k = np.ascontiguousarray(np.stack(ks, axis=1))
        v = np.ascontiguousarray(np.stack(vs, axis=1))
        return specs, rids, q, k, v

    def after_step(self, specs: List[int], actions) -> List[Tuple[int, int]]:
        """Advance the residents; returns (spec index, request id) of those to release now:
        finished ones, and stalled ones (the scheduler's preemption; they are not re-queued)."""
        out = []
        for idx, act in zip(specs, actions):
            res = self.resident[idx]
            if int(act) == HELD:             # asynchronous boundary work: sat the step out, its token comes next step
                continue
            res.step += 1
            self.tokens += 1
            if int(act) < 0:
                self.stalled.append(idx)
                out.append((idx, res.rid))
            elif res.step >= res.spec.n_steps:
                self.finished.append(idx)
                out.append((idx, res.rid))
        for idx, _ in out:
            del self.resident[idx]
        return out

    def done(self) -> bool:
        return not self.pending and not self.resident


def decode_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64 (exact)."""
    return W.bf16_bits_to_f64(x)
