#!/usr/bin/env python
"""Benchmark of the GrowPage decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--boundary async|sync]
                    [--workload layer|stack] [--policy P] [--entry step|layers]

Workload: the one-layer Qwen3-8B-shaped configuration (32 query / 8 KV heads, head_dim 128, bf16,
page 16; 64 concurrent requests, prompts uniform in [128, 1024], 4096 decode steps each, per-request
heavy-hitter fraction log-uniform in [0.5 %, 20 %], seed 1), synthetic inputs.  One "step" is one
`gp_decode_step` over all 64 requests: plan + summary update, fused append + paged GQA attention +
boundary logits, working sets + selection + decision + allocator, compaction.

The K timed steps are steps [S0, S0 + K) of the 4096-step job with S0 = (4096 - K) // 2, reached by
running the S0 preceding steps untimed; K = 4096 (the default) times the whole job.  Warm-up steps
run on the same pool, which is then re-initialised.  The headline is the asynchronous boundary mode
(the boundary chain of a step runs beside the next step and the requests it concerns sit that step
out; tokens are counted, not request-steps); the synchronous mode is timed in the same run, with
and without early planning, and reported beside it.  Prints ONE JSON line (rank 0).

`--gpus N` with N > 1 starts N ranks itself (one per GPU, torch.distributed.run on 127.0.0.1) unless
it already runs inside such a launch; every rank owns a pool and its own requests, nothing is
exchanged on the data path (weak scaling).
"""
from __future__ import annotations

import argparse
import concurrent.futures as cf
import json
import os
import socket
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_03494_b200 import shard  # noqa: E402
from paper_2609_03494_b200 import workload as W  # noqa: E402

METRIC = "decode tokens/s (attn+KV budgeting) @Qwen3-8B shape; % of HBM roofline"
JOB_STEPS = 4096
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per algorithmic byte of the attention kernel, from one ncu capture of a launch of this workload
# (dram__bytes_read.sum + dram__bytes_write.sum over the launch's algorithmic bytes); not measured by this run
TRAFFIC_RATIO = 1.02
TRAFFIC_SOURCE = "profiles/attention_qwen3_8b_layer.md (ncu capture of one launch), scaled by this run's algorithmic bytes"


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------------------------------
# inputs
# --------------------------------------------------------------------------------------------------
def generate_inputs(wl: W.Workload, t_end: int, torch, pin: bool):
    """All decode-step inputs of steps [0, t_end) as host int16 tensors (bf16 bits):
    q [T][L][B][H_q][d], k, v [T][L][B][H_kv][d]; and the prompts."""
    s = wl.shape
    B = len(wl.requests)
    mk = lambda h: torch.empty((t_end, s.n_layers, B, h, s.head_dim), dtype=torch.int16, pin_memory=pin)
    q_all, k_all, v_all = mk(s.n_q_heads), mk(s.n_kv_heads), mk(s.n_kv_heads)
    qn, kn, vn = (x.numpy().view(np.uint16) for x in (q_all, k_all, v_all))
    prompts = [None] * B

    def one(i):
        st = wl.stream(wl.requests[i])
        prompts[i] = st.prompt_kv()
        q, k, v = st.steps(0, t_end)
        qn[:, :, i] = q
        kn[:, :, i] = k
        vn[:, :, i] = v

    with cf.ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 4)) as ex:
        list(ex.map(one, range(B)))
    return q_all, k_all, v_all, prompts


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device: int):
        self.path = tempfile.mktemp(suffix=".csv")
        self.device = device
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.device)],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# --------------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------------
class Inputs:
    """The job's inputs, once on the host (pinned) and once on the device; shared by the pools of a run."""

    def __init__(self, wl, torch, device, t_end):
        self.q_host, self.k_host, self.v_host, prompts = generate_inputs(wl, t_end, torch, pin=True)
        dev = f"cuda:{device}"
        self.q_dev, self.k_dev, self.v_dev = self.q_host.to(dev), self.k_host.to(dev), self.v_host.to(dev)
        self.prompts_dev = [(torch.from_numpy(k.view(np.int16)).to(dev), torch.from_numpy(v.view(np.int16)).to(dev))
                            for k, v in prompts]


class Job:
    """One pool and the requests of the workload in it.  Step t of the job feeds every request the synthetic
    inputs of step t; a request that sits a step out (asynchronous boundary mode) skips that step's inputs,
    which are independent draws per step."""

    def __init__(self, wl, torch, device, inp: Inputs, host_staging=True, policy=0, async_boundary=False, async_slots=0,
                 overlap_slots=0):
        from paper_2609_03494_b200 import binding as B
        self.B, self.torch, self.wl, self.device, self.inp = B, torch, wl, device, inp
        s = wl.shape
        self.nreq = len(wl.requests)
        self.M = max(4, self.nreq)
        cfg = B.make_config(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, n_pages=wl.n_pages,
                            max_pages_per_req=wl.max_pages_per_req, max_requests=self.M, k_loc=wl.k_loc,
                            host_staging=host_staging, policy=policy, async_boundary=async_boundary, async_slots=async_slots,
                            overlap_slots=overlap_slots)
        self.pool = B.Pool(cfg, device)
        self.is_async = async_boundary
        dev = f"cuda:{device}"
        self.ids_dev = torch.arange(self.nreq, dtype=torch.int32, device=dev)
        self.ids_host = torch.arange(self.nreq, dtype=torch.int32).pin_memory()
        self.out_dev = torch.zeros((s.n_layers, self.nreq, s.n_q_heads, s.head_dim), dtype=torch.float32, device=dev)
        self.act_dev = torch.zeros(self.nreq, dtype=torch.int32, device=dev)
        self.out_host = torch.zeros((s.n_layers, self.nreq, s.n_q_heads, s.head_dim), dtype=torch.float32).pin_memory()
        self.act_host = torch.zeros(self.nreq, dtype=torch.int32).pin_memory()
        # a second pair of result buffers for the pipelined host loop (step t + 1 is issued while t's results are read)
        self.out_host2 = torch.zeros_like(self.out_host).pin_memory()
        self.act_host2 = torch.zeros_like(self.act_host).pin_memory()
        self._host_ptrs = None
        self.live = False
        self.by_layer = False           # True: steps go through gp_step_begin / gp_attn_layer / gp_step_end
        self.reset()

    def reset(self):
        B = self.B
        if self.live:
            for r in range(self.nreq):
                self.pool.release(r)
        for i, spec in enumerate(self.wl.requests):
            kd, vd = self.inp.prompts_dev[i]
            st, rid = self.pool.request_add(-1, 0, kd, vd, spec.prompt_len, self.wl.initial_pages)
            assert st == B.GP_OK and rid == i, (st, rid)
        self.live = True
        self.t = 0

    def step(self):
        f = self.pool.decode_step_layers if self.by_layer else self.pool.decode_step
        i = self.inp
        f(self.ids_dev, i.q_dev[self.t], i.k_dev[self.t], i.v_dev[self.t], self.out_dev, self.act_dev)
        self.t += 1

    def step_host(self):
        # gp_decode_step_host through the binding, with the host addresses of this step's inputs worked out here
        # (the tensors are contiguous [T][...]): the call a C caller makes, without a tensor view per argument
        i = self.inp
        if self._host_ptrs is None:
            self._host_ptrs = (self.pool.handle, self.ids_host.data_ptr(), i.q_host.data_ptr(), i.k_host.data_ptr(),
                               i.v_host.data_ptr(), self.out_host.data_ptr(), self.act_host.data_ptr(),
                               i.q_host[0].numel() * 2, i.k_host[0].numel() * 2, self.pool.stream())
        h, ids, qp, kp, vp, op, ap, qs, ks, strm = self._host_ptrs
        t = self.t
        self.B.gp_decode_step_host(h, ids, self.nreq, qp + t * qs, kp + t * ks, vp + t * ks, op, ap, strm)
        self.t += 1

    def step_host_async(self, which):
        # the same through gp_decode_step_host_async, results into buffer pair `which`
        assert self._host_ptrs is not None          # worked out by step_host's first call
        h, ids, qp, kp, vp, op, ap, qs, ks, strm = self._host_ptrs
        if which:
            op, ap = self.out_host2.data_ptr(), self.act_host2.data_ptr()
        t = self.t
        self.B.gp_decode_step_host_async(h, ids, self.nreq, qp + t * qs, kp + t * ks, vp + t * ks, op, ap, strm)
        self.t += 1

    def roll(self, t_to):
        while self.t < t_to:
            self.step()

    def state(self):
        P, n = self.B.gp_debug_state(self.pool.handle, self.M)
        return P[:self.nreq].astype(np.int64), n[:self.nreq].astype(np.int64)

    def counters(self):
        c = self.B.gp_debug_pool(self.pool.handle)[2]
        assert c[7] == 0, f"kernel error bits {c[7]}"
        return c

    def step_bytes(self, P, n_old, actions):
        """Algorithmic bytes of the step just run, from the requests' pages and tokens before it and its actions:
        attention (keys and values of every retained token, the appended row, query in, output out, page ids) and
        boundary scoring (the keys of the candidate set)."""
        B = self.B
        s = self.wl.shape
        Wb = s.token_bytes
        fixed = 2 * s.n_q_heads * s.head_dim + 4 * s.n_q_heads * s.head_dim
        stepped = np.isin(actions, (B.GP_ACT_NONE, B.GP_ACT_PENDING, B.GP_ACT_GROW, B.GP_ACT_COMPRESS,
                                    B.GP_ACT_COMPRESS_FALLBACK, B.GP_ACT_SHRINK)) | ((actions == B.GP_ACT_STALLED) & (n_old < P * 16))
        n_new = n_old + 1
        attn = float(s.n_layers * ((n_new[stepped] * Wb).sum() + stepped.sum() * (Wb + fixed)) + 4 * P[stepped].sum())
        at_b = stepped & (n_new == P * 16)
        score = float(s.n_layers * ((P[at_b] - 1) * 16).sum() * (Wb // 2))
        return attn, score, int(stepped.sum()), int(n_new[stepped].sum())


def timed_window(job, torch, device, S0, K, rank, sample_clocks=False):
    """K steps from step S0 on, device time by CUDA events on the launching stream; returns (ms on this rank,
    tokens decoded on this rank, kernels launched, clock record or None)."""
    B = job.B
    stream = torch.cuda.current_stream(device)
    # the clock sampler starts before the untimed roll to the window, so that the GPU is under load, not waking up
    # from an idle pause, when the timed steps begin
    sampler = ClockSampler(device) if (sample_clocks and rank == 0) else None
    if sampler:
        sampler.start()
        time.sleep(0.3)
    job.reset()
    job.roll(S0)
    torch.cuda.synchronize(device)
    tok0 = int(job.counters()[6])
    launches0 = B.gp_launch_count(job.pool.handle)
    shard.barrier(device)
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(K):
        job.step()
    B.gp_async_join(job.pool.handle, job.pool.stream())      # the last step's boundary work belongs to the timed region
    e1.record(stream)
    torch.cuda.synchronize(device)
    shard.barrier(device)
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if sampler else None
    launches = B.gp_launch_count(job.pool.handle) - launches0
    tokens = int(job.counters()[6]) - tok0
    return ms, tokens, launches, clocks


def run_ours(args):
    import torch
    rank, local_rank, world = shard.init("nccl")
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    device = local_rank
    torch.cuda.set_device(device)
    K, Wm = args.steps, max(args.warmup, 3)
    stack = args.workload == "stack"
    job_steps = 96 if stack else JOB_STEPS
    K = max(1, min(K, job_steps))
    S0 = (job_steps - K) // 2
    wl = W.stack8b_resident(seed=shard.shard_seed(2, rank)) if stack else W.layer8b(seed=shard.shard_seed(1, rank))
    s = wl.shape
    t_gen = time.time()
    inp = Inputs(wl, torch, device, S0 + K)
    t_gen = time.time() - t_gen
    policy = {"demand": 0, "inverse": 1, "random": 2, "shrink": 3}[args.policy]
    by_layer = args.entry == "layers"
    head_async = args.boundary == "async" and not by_layer      # the layer-by-layer calls exist in the synchronous mode only
    jobs = {"sync": Job(wl, torch, device, inp, policy=policy)}
    if head_async or args.boundary == "both":
        jobs["async"] = Job(wl, torch, device, inp, policy=policy, async_boundary=True, async_slots=args.async_slots)
    head = jobs["async"] if head_async else jobs["sync"]
    head.by_layer = by_layer
    B = head.B
    # ---- warm-up ------------------------------------------------------------------------------------
    for job in jobs.values():
        for _ in range(Wm):
            job.step()
    torch.cuda.synchronize(device)

    # ---- timed, inputs resident in HBM: the headline mode, then the others for comparison ----------------------
    ms_local, tokens_local, gpu_launches, clocks = timed_window(head, torch, device, S0, K, rank, sample_clocks=True)
    value, ms = shard.job_throughput(tokens_local, ms_local, device)
    modes = {}
    if not by_layer:
        sj = jobs["sync"]
        for name, early in (("sync", False), ("sync_early_plan", True)):
            B.gp_set_early_plan(sj.pool.handle, early)
            m, tk, _, _ = timed_window(sj, torch, device, S0, K, rank)
            v, m = shard.job_throughput(tk, m, device)
            modes[name] = {"ms_per_step": round(m / K, 5), "tokens_per_s": round(v, 1)}
        B.gp_set_early_plan(sj.pool.handle, False)
        for ov in [-1] + [int(x) for x in args.overlap_slots.split(",") if x]:
            oj = Job(wl, torch, device, inp, policy=policy, overlap_slots=ov)
            for _ in range(Wm):
                oj.step()
            for name, early in (("sync_four_kernels", False),) if ov == -1 else ((f"overlap{ov}", False), (f"overlap{ov}_early_plan", True)):
                B.gp_set_early_plan(oj.pool.handle, early)
                m, tk, _, _ = timed_window(oj, torch, device, S0, K, rank)
                v, m = shard.job_throughput(tk, m, device)
                modes[name] = {"ms_per_step": round(m / K, 5), "tokens_per_s": round(v, 1)}
            oj.pool.close()
        if "async" in jobs:
            if head_async:
                modes["async"] = {"ms_per_step": round(ms / K, 5), "tokens_per_s": round(value, 1)}
            else:
                m, tk, _, _ = timed_window(jobs["async"], torch, device, S0, K, rank)
                v, m = shard.job_throughput(tk, m, device)
                modes["async"] = {"ms_per_step": round(m / K, 5), "tokens_per_s": round(v, 1)}

    # ---- per-kernel timing pass (CUDA events around every kernel, on the launching streams) and the byte count -------
    head.by_layer = False               # per-kernel times come from the whole-step entry (same kernels)
    head.reset()
    head.roll(S0)
    torch.cuda.synchronize(device)
    moved0 = int(head.counters()[8])
    B.gp_set_profiling(head.pool.handle, True)
    attn_bytes = score_bytes = 0.0
    n_tok = n_kv = 0
    for _ in range(K):
        P, n_old = head.state()
        head.step()
        acts = head.act_dev.cpu().numpy()
        a, sc, st_n, kv_n = head.step_bytes(P, n_old, acts)
        attn_bytes += a
        score_bytes += sc
        n_tok += st_n
        n_kv += kv_n
    kms, kn = B.gp_get_kernel_times(head.pool.handle)
    B.gp_set_profiling(head.pool.handle, False)
    head.by_layer = by_layer
    moved = int(head.counters()[8]) - moved0
    compact_bytes = 2.0 * moved * (2 * s.head_dim * 2 + 4)
    summ_bytes = float(n_tok) * s.n_layers * 2 * s.n_q_heads * s.head_dim * 8 * 2      # both views, read + write, fp64
    step_bytes = attn_bytes + score_bytes + compact_bytes + summ_bytes
    peak, peak_kind = measured_peak()
    attn_ms = float(kms[1])
    achieved = attn_bytes / (attn_ms * 1e-3) / 1e9
    step_gbs = step_bytes / (ms_local * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": "gp_attn_kernel<128> (append + paged GQA attention + boundary logits)",
        "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s", "frac": round(achieved / peak, 4),
        "peak_kind": f"of {peak_kind}", "frac_of_nominal_8tbs": round(achieved / NOMINAL_HBM_GBS, 4),
        "traffic": round(TRAFFIC_RATIO * attn_bytes / K), "traffic_source": TRAFFIC_SOURCE,
        "algorithmic_bytes_per_launch": round(attn_bytes / K),
        "launch_us": round(attn_ms * 1e3 / K, 2),
        "whole_step_frac_of_nominal_8tbs": round(step_gbs / NOMINAL_HBM_GBS, 4),
        "kernel_share_of_step": {name: round(float(kms[i]) / float(kms.sum()), 4) for i, name in enumerate(B.KERNEL_NAMES)},
        "kernel_us_per_step": {name: round(float(kms[i]) * 1e3 / K, 2) for i, name in enumerate(B.KERNEL_NAMES)},
    }
    step_roofline = {
        "what": "bytes of K/V, page ids, queries, outputs, summaries, scored keys and moved rows of the timed steps over the "
                "timed window's device time; the north star's figure (target 0.70 of 8 TB/s)",
        "algorithmic_bytes_per_step": round(step_bytes / K),
        "attention": round(attn_bytes / K), "scoring": round(score_bytes / K), "compaction": round(compact_bytes / K),
        "summaries": round(summ_bytes / K),
        "achieved_gbs": round(step_gbs, 1), "frac_of_8tbs": round(step_gbs / NOMINAL_HBM_GBS, 4),
        "frac_of_measured": round(step_gbs / peak, 4), "mean_tokens_per_request": round(n_kv / max(n_tok, 1), 1),
        "tokens_per_step": round(n_tok / K, 2),
    }

    # ---- end to end: host buffers, copies inside the timed region -----------------------------------------------
    head.reset()
    head.roll(S0)
    torch.cuda.synchronize(device)
    tok0 = int(head.counters()[6])
    shard.barrier(device)
    t0 = time.perf_counter()
    for _ in range(K):
        head.step_host()
    B.gp_async_join(head.pool.handle, head.pool.stream())
    torch.cuda.synchronize(device)
    e2e_block_ms = (time.perf_counter() - t0) * 1e3
    shard.barrier(device)
    e2e_block_tokens = int(head.counters()[6]) - tok0
    e2e_block_value, _ = shard.job_throughput(e2e_block_tokens, e2e_block_ms, device)
    # The same with the host one step behind the GPU, as a serving loop with asynchronous scheduling runs it: step t
    # is issued (gp_decode_step_host_async: inputs fetched from pinned host memory, results written to pinned host
    # memory by the kernels), then the host waits for step t - 1 and reads its actions.  Every step's inputs cross
    # the bus inside the timed region, every step's results are read by the host inside it.
    head.reset()
    head.roll(max(S0 - 2, 0))
    while head.t < S0:                      # untimed: the path's own first calls (its streams and events are made then)
        head.step_host_async(head.t & 1)
        head.pool.host_wait()
    torch.cuda.synchronize(device)
    tok0 = int(head.counters()[6])
    act_np = [head.act_host.numpy(), head.act_host2.numpy()]      # views of the pinned result buffers
    acts_seen = 0
    shard.barrier(device)
    t0 = time.perf_counter()
    for j in range(K):
        head.step_host_async(j & 1)
        if j > 0:
            head.pool.host_wait()                                   # step j - 1: its results are in the host buffers
            acts_seen += int(np.count_nonzero(act_np[(j - 1) & 1]))
    head.pool.host_wait()
    acts_seen += int(np.count_nonzero(act_np[(K - 1) & 1]))
    B.gp_async_join(head.pool.handle, head.pool.stream())
    torch.cuda.synchronize(device)
    e2e_ms_local = (time.perf_counter() - t0) * 1e3
    shard.barrier(device)
    assert B.gp_pool_status(head.pool.handle)[0] == B.GP_OK
    e2e_tokens = int(head.counters()[6]) - tok0
    e2e_value, _ = shard.job_throughput(e2e_tokens, e2e_ms_local, device)
    h2d = int(s.n_layers * head.nreq * (s.n_q_heads + 2 * s.n_kv_heads) * s.head_dim * 2 + 4 * head.nreq)
    d2h = int(s.n_layers * head.nreq * s.n_q_heads * s.head_dim * 4 + 4 * head.nreq)
    counters = head.counters()

    # ---- CPU baseline: the oracle as it stands, on a bounded sample, one process per host core ---------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = time_oracle_all_cores(wl, n_steps=2048 if not stack else 32, stack=stack)

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": round(ms / K, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": ("qwen3-8b-stack-resident: L=36, 32q/8kv heads, d=128, page 16, 16 requests x 96 decode "
                                    "steps, prompts U[400,1000], heavy-hitter fraction logU[0.5%,20%], seed 2 (not the headline "
                                    "workload)") if stack else
                                   ("qwen3-8b-layer: L=1, 32q/8kv heads, d=128, page 16, 64 requests x 4096 decode steps, "
                                    "prompts U[128,1024], heavy-hitter fraction logU[0.5%,20%], seed 1"),
                       "entry": "gp_decode_step" if not by_layer else "gp_step_begin + gp_attn_layer per layer + gp_step_end",
                       "boundary": ("async: the boundary chain of a step runs beside the next step, the requests it concerns sit "
                                    "that step out; value counts decoded tokens") if head_async else "sync",
                       "early_plan": False, "policy": args.policy, "requests_per_gpu": head.nreq,
                       "timed_steps": [S0, S0 + K], "job_steps": job_steps,
                       "l2": "per-step working set (all resident K/V) is larger than L2; no flush needed",
                       "input_generation_s": round(t_gen, 1)},
            "modes": modes,
            "north_star": {"whole_step_frac_of_8tbs": step_roofline["frac_of_8tbs"], "target": 0.70,
                           "met": bool(step_roofline["frac_of_8tbs"] >= 0.70)},
            "roofline": roofline, "step_roofline": step_roofline,
            "cpu_baseline": cpu,
            "e2e": {"value": round(e2e_value, 1), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms_local / K, 5),
                    "how": "gp_decode_step_host_async + gp_decode_step_host_wait, the host reads step t - 1's results while step t runs",
                    "blocking": {"value": round(e2e_block_value, 1), "ms_per_step": round(e2e_block_ms / K, 5),
                                 "how": "gp_decode_step_host, one synchronisation per step"},
                    "boundary_actions_read": acts_seen},
            "gpu_launches": int(gpu_launches),
            "clocks": clocks,
            "events": {"grow": int(counters[0]), "compress": int(counters[1]), "fallback": int(counters[2]),
                       "stalled": int(counters[3]), "shrink": int(counters[10])},
        }
        print(json.dumps(line))
    for job in jobs.values():
        job.pool.close()
    shard.finish()


# --------------------------------------------------------------------------------------------------
# the oracle as CPU baseline / reference arm
# --------------------------------------------------------------------------------------------------
def _oracle_run(wl_args, req_lo, req_hi, n_steps, warmup, budget_s):
    """Runs requests [req_lo, req_hi) of the workload through a pool of the oracle for `n_steps` decode steps;
    returns (wall seconds of the decode steps, request-steps done, steps done)."""
    from oracle import growpage_oracle as O
    from paper_2609_03494_b200 import harness as H
    stack, seed = wl_args
    wl = W.stack8b_resident(seed=seed) if stack else W.layer8b(seed=seed)
    s = wl.shape
    n_requests = req_hi - req_lo
    sub = W.Workload(wl.name, wl.seed, s, wl.requests, n_resident=n_requests,
                     initial_pages=wl.initial_pages, max_pages_per_req=wl.max_pages_per_req,
                     n_pages=n_requests * wl.max_pages_per_req, k_loc=wl.k_loc)
    cfg = O.OracleConfig(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, n_pages=sub.n_pages,
                         max_pages_per_req=sub.max_pages_per_req, k_loc=sub.k_loc, max_requests=max(4, n_requests))
    pool = O.OraclePool(cfg)
    sch = H.Scheduler(sub, only=range(req_lo, req_hi))
    while True:
        op = sch.next_admission()
        if op is None:
            break
        st, rid = pool.request_add(-1, 0, H.decode_bits(op.k_tail), H.decode_bits(op.v_tail), op.n_tail, op.initial_pages)
        assert st == O.OK
        sch.admitted(op, rid)

    def one():
        specs, rids, q, k, v = sch.batch()
        q, k, v = H.decode_bits(q), H.decode_bits(k), H.decode_bits(v)
        t0 = time.perf_counter()
        rec = pool.decode_step(rids, q, k, v)
        dt = time.perf_counter() - t0
        sch.after_step(specs, rec.actions)
        return dt

    for _ in range(warmup):
        one()
    wall, done = 0.0, 0
    for _ in range(n_steps):
        wall += one()
        done += 1
        if wall > budget_s:
            break
    return wall, done * n_requests, done


def time_oracle(wl_args, n_requests: int, n_steps: int, warmup: int, budget_s: float = 25.0):
    """The oracle in this process (numpy; as many threads as its BLAS takes)."""
    cpu0 = time.process_time()
    wall, units, done = _oracle_run(wl_args, 0, n_requests, n_steps, warmup, budget_s)
    cpu_used = time.process_time() - cpu0
    cores = max(1, int(round(cpu_used / max(wall, 1e-9))))
    return {"value": round(units / wall, 2), "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": f"first {n_requests} requests of the workload, decode steps {warmup}..{warmup + done} of the job "
                      f"(float64 numpy, {os.cpu_count()} host cores present, timed region excludes input decoding)",
            "steps": done, "wall_s": round(wall, 4)}


def time_oracle_all_cores(wl, n_steps: int, stack: bool):
    """One process per host core, each with its own oracle pool and its share of the requests (requests are
    independent while neither the pool nor the cap binds, as here); throughput = all request-steps over the
    slowest process's decode time."""
    n_proc = max(1, min(os.cpu_count() or 1, len(wl.requests)))
    per = len(wl.requests) // n_proc
    parts = [(i * per, (i + 1) * per) for i in range(n_proc)]
    os.environ.setdefault("OMP_NUM_THREADS", "1")
    t0 = time.perf_counter()
    with cf.ProcessPoolExecutor(max_workers=n_proc) as ex:
        futs = [ex.submit(_oracle_run, (stack, wl.seed), lo, hi, n_steps, 0, 20.0) for lo, hi in parts]
        res = [f.result() for f in futs]
    wall_all = time.perf_counter() - t0
    slowest = max(r[0] for r in res)
    units = sum(r[1] for r in res)
    steps = min(r[2] for r in res)
    return {"value": round(units / slowest, 2), "unit": "tokens/s", "cores": n_proc, "kind": "oracle",
            "sample": f"{n_proc} processes x {per} requests of the workload ({n_proc * per} of {len(wl.requests)}), decode steps "
                      f"0..{steps} of the job, not the timed window (float64 numpy, one thread per process; the figure "
                      f"divides by the slowest process's decode time; input decoding excluded)",
            "steps": steps, "wall_s": round(slowest, 4), "wall_with_setup_s": round(wall_all, 2)}


def run_reference(args):
    rank, _, world = shard.env_world()
    if rank != 0:
        return
    K, Wm = max(1, args.steps), max(0, args.warmup)
    n_req = 4
    res = time_oracle((False, 1), n_requests=n_req, n_steps=K, warmup=Wm, budget_s=150.0)
    line = {
        "impl": "reference", "metric": METRIC, "value": res["value"], "unit": "tokens/s",
        "n_gpus": world if world > 1 else max(1, args.gpus),
        "steps": res["steps"], "warmup": Wm, "ms_per_step": round(1e3 * res["wall_s"] / res["steps"], 4),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "qwen3-8b-layer (bounded sample: each step decodes the first 4 of the 64 requests once, "
                               "from the start of the job)"},
        "cpu_baseline": {"value": res["value"], "unit": "tokens/s", "cores": res["cores"], "kind": "oracle",
                         "sample": res["sample"]},
        "e2e": {"value": res["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_size(args):
    """The configurations whose full size only the GPU can hold (36 or 64 layers on a 120 GB pool; 256 requests on
    shared 2048-token prompts): `steps` decode steps with continuous batching on device-drawn inputs, device time
    by CUDA events around the decode steps, and the any-size invariants checked on the state read back."""
    import torch
    from paper_2609_03494_b200 import synth
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    sc = {"config3": synth.config3, "config4": synth.config4, "config5": synth.config5}[args.workload]()
    K = args.steps if args.steps != JOB_STEPS else (256 if args.workload != "config5" else 2048)
    res = synth.run_at_size(sc, n_steps=K, chunk=8, async_boundary=args.boundary == "async", check_every=8,
                            seed={"config3": 2, "config4": 3, "config5": 4}[args.workload])
    peak, peak_kind = measured_peak()
    line = {"metric": METRIC, "value": res["tokens_per_s"], "unit": "tokens/s", "n_gpus": 1, "steps": K, "warmup": 0,
            "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic (drawn on the device)",
            "config": {"workload": f"{res['config']} at its stated size (not the headline workload): {res['layers']} layers, "
                                   f"{sc.n_resident} residents, pool {res['pool_kv_gb']} GB of K/V in a blob of {res['blob_gb']} GB",
                       "boundary": "async" if res["async_boundary"] else "sync"},
            "step_roofline": {"what": "keys and values of the residents' retained tokens over the decode steps' device time (attention "
                                      "traffic only; boundary scoring and compaction not counted)",
                              "achieved_gbs": res["attention_bytes_over_step_time_gbs"],
                              "frac_of_8tbs": round(res["attention_bytes_over_step_time_gbs"] / NOMINAL_HBM_GBS, 4),
                              "frac_of_measured": round(res["attention_bytes_over_step_time_gbs"] / peak, 4), "peak_kind": peak_kind},
            "size_run": res}
    print(json.dumps(line))


def spawn_ranks(n: int) -> int:
    """`--gpus N` outside a torchrun launch: start N ranks of this command, one per GPU, on this node."""
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=JOB_STEPS)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--boundary", default="both", choices=["async", "sync", "both"],
                    help="both (default): headline synchronous, the asynchronous boundary mode timed beside it; sync: synchronous "
                         "only; async: headline asynchronous (boundary work beside the next step)")
    ap.add_argument("--async-slots", type=int, default=0, help="thread blocks the attention kernel leaves to the boundary kernels")
    ap.add_argument("--overlap-slots", default="", help="comma-separated overlap_slots values to time as extra modes (synchronous mode, boundary work beside the attention kernel)")
    ap.add_argument("--entry", default="step", choices=["step", "layers"],
                    help="step: gp_decode_step; layers: the same step through gp_step_begin / gp_attn_layer / gp_step_end")
    ap.add_argument("--workload", default="layer", choices=["layer", "stack", "config3", "config4", "config5"],
                    help="layer: the headline one-layer Qwen3-8B-shaped workload; stack: the 36-layer shape, 16 resident requests; "
                         "config3 / config4 / config5: the multi-layer and prefix-sharing configurations at their stated sizes, "
                         "inputs drawn on the device (throughput and invariants, no per-kernel pass)")
    ap.add_argument("--policy", default="demand", choices=["demand", "inverse", "random", "shrink"],
                    help="capacity-control policy (the paper's default, or one of its ablation's controls)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload.startswith("config"):
        run_size(args)
    elif args.gpus > 1 and "RANK" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
