#!/usr/bin/env python
"""Benchmark of the GrowPage decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload layer|stack]

Workload: the one-layer Qwen3-8B-shaped configuration (32 query / 8 KV heads, head_dim 128, bf16,
page 16; 64 concurrent requests, prompts uniform in [128, 1024], 4096 decode steps each, per-request
heavy-hitter fraction log-uniform in [0.5 %, 20 %], seed 1), synthetic inputs.  One "step" is one
`gp_decode_step` over all 64 requests: plan + summary update, fused append + paged GQA attention +
boundary logits, working sets + selection + decision + allocator, compaction.

The K timed steps are steps [S0, S0 + K) of the 4096-step job with S0 = (4096 - K) // 2, reached by
running the S0 preceding steps untimed; K = 4096 (the default) times the whole job.  Warm-up steps
run on the same pool, which is then re-initialised.  Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import concurrent.futures as cf
import json
import os
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


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def traffic_ratio():
    """DRAM bytes per algorithmic byte of the attention kernel, from the committed ncu summary."""
    path = os.path.join(ROOT, "profiles", "attention_qwen3_8b_layer.md")
    try:
        for line in open(path):
            if line.startswith("dram_bytes_per_algorithmic_byte"):
                return float(line.split("=")[1].split()[0])
    except Exception:
        pass
    return None


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
class Job:
    def __init__(self, wl, torch, device, q_all, k_all, v_all, prompts, host_staging=True, policy=0):
        from paper_2609_03494_b200 import binding as B
        self.B, self.torch, self.wl, self.device = B, torch, wl, device
        s = wl.shape
        self.nreq = len(wl.requests)
        cfg = B.make_config(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, n_pages=wl.n_pages,
                            max_pages_per_req=wl.max_pages_per_req, max_requests=max(4, self.nreq), k_loc=wl.k_loc,
                            host_staging=host_staging, policy=policy)
        self.pool = B.Pool(cfg, device)
        # every step's inputs are resident tensors written long before the step is enqueued, and nothing else is
        # enqueued between steps: the precondition of early planning holds
        B.gp_set_early_plan(self.pool.handle, True)
        dev = f"cuda:{device}"
        self.q_host, self.k_host, self.v_host = q_all, k_all, v_all
        self.q_dev, self.k_dev, self.v_dev = q_all.to(dev), k_all.to(dev), v_all.to(dev)
        self.prompts_dev = [(torch.from_numpy(k.view(np.int16)).to(dev), torch.from_numpy(v.view(np.int16)).to(dev))
                            for k, v in prompts]
        self.ids_dev = torch.arange(self.nreq, dtype=torch.int32, device=dev)
        self.ids_host = torch.arange(self.nreq, dtype=torch.int32).pin_memory()
        self.out_dev = torch.zeros((s.n_layers, self.nreq, s.n_q_heads, s.head_dim), dtype=torch.float32, device=dev)
        self.act_dev = torch.zeros(self.nreq, dtype=torch.int32, device=dev)
        self.out_host = torch.zeros((s.n_layers, self.nreq, s.n_q_heads, s.head_dim), dtype=torch.float32).pin_memory()
        self.act_host = torch.zeros(self.nreq, dtype=torch.int32).pin_memory()
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
            kd, vd = self.prompts_dev[i]
            st, rid = self.pool.request_add(-1, 0, kd, vd, spec.prompt_len, self.wl.initial_pages)
            assert st == B.GP_OK and rid == i, (st, rid)
        self.live = True
        self.P = np.array([max(self.wl.initial_pages, sp.prompt_len // 16 + 1) for sp in self.wl.requests])
        self.n = np.array([sp.prompt_len for sp in self.wl.requests])
        self.t = 0

    def step(self):
        f = self.pool.decode_step_layers if self.by_layer else self.pool.decode_step
        f(self.ids_dev, self.q_dev[self.t], self.k_dev[self.t], self.v_dev[self.t], self.out_dev, self.act_dev)
        self.t += 1

    def step_host(self):
        # gp_decode_step_host through the binding, with the host addresses of this step's inputs worked out here
        # (the tensors are contiguous [T][...]): the call a C caller makes, without a tensor view per argument
        if self._host_ptrs is None:
            self._host_ptrs = (self.pool.handle, self.ids_host.data_ptr(), self.q_host.data_ptr(), self.k_host.data_ptr(),
                               self.v_host.data_ptr(), self.out_host.data_ptr(), self.act_host.data_ptr(),
                               self.q_host[0].numel() * 2, self.k_host[0].numel() * 2, self.pool.stream())
        h, ids, qp, kp, vp, op, ap, qs, ks, strm = self._host_ptrs
        t = self.t
        self.B.gp_decode_step_host(h, ids, self.nreq, qp + t * qs, kp + t * ks, vp + t * ks, op, ap, strm)
        self.t += 1

    def roll(self, t_to):
        while self.t < t_to:
            self.step()

    # host mirror of (P, n) driven by the actions the step returned: algorithmic bytes come from here
    def mirror(self, actions):
        B = self.B
        s = self.wl.shape
        Wb = s.token_bytes
        fixed = 2 * s.n_q_heads * s.head_dim + 4 * s.n_q_heads * s.head_dim        # query rows in, output rows out
        n_new = self.n + 1
        attn = float(s.n_layers * (n_new.sum() * Wb + self.nreq * (Wb + fixed)) + 4 * self.P.sum())
        at_b = n_new == self.P * 16
        score = float(s.n_layers * ((self.P[at_b] - 1) * 16).sum() * (Wb // 2))
        self.n = n_new
        grow = actions == B.GP_ACT_GROW
        comp = (actions == B.GP_ACT_COMPRESS) | (actions == B.GP_ACT_COMPRESS_FALLBACK)
        shrink = actions == B.GP_ACT_SHRINK
        self.P = self.P + grow
        self.n = np.where(comp, (self.P - 1) * 16, self.n)
        self.n = np.where(shrink, (self.P - 2) * 16, self.n)
        self.P = self.P - shrink
        return attn, score

    def moved_rows(self):
        return int(self.B.gp_debug_pool(self.pool.handle)[2][8])

    def check_healthy(self):
        c = self.B.gp_debug_pool(self.pool.handle)[2]
        assert c[7] == 0, f"kernel error bits {c[7]}"
        return c


def run_ours(args):
    import torch
    rank, local_rank, world = shard.init("nccl")
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    device = local_rank
    torch.cuda.set_device(device)
    K, Wm = args.steps, args.warmup
    stack = args.workload == "stack"
    job_steps = 96 if stack else JOB_STEPS
    K = max(1, min(K, job_steps))
    S0 = (job_steps - K) // 2
    wl = W.stack8b_resident(seed=shard.shard_seed(2, rank)) if stack else W.layer8b(seed=shard.shard_seed(1, rank))
    s = wl.shape
    t_gen = time.time()
    q_all, k_all, v_all, prompts = generate_inputs(wl, S0 + K, torch, pin=True)
    t_gen = time.time() - t_gen
    policy = {"demand": 0, "inverse": 1, "random": 2, "shrink": 3}[args.policy]
    job = Job(wl, torch, device, q_all, k_all, v_all, prompts, policy=policy)
    job.by_layer = args.entry == "layers"
    B = job.B
    stream = torch.cuda.current_stream(device)

    # ---- warm-up ------------------------------------------------------------------------------------
    for _ in range(max(Wm, 3)):
        job.step()
    torch.cuda.synchronize(device)
    job.reset()

    # ---- timed, inputs resident in HBM -----------------------------------------------------------------
    job.roll(S0)
    launches0 = B.gp_launch_count(job.pool.handle)
    sampler = ClockSampler(device)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    shard.barrier(device)
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(K):
        job.step()
    e1.record(stream)
    torch.cuda.synchronize(device)
    shard.barrier(device)
    ms_local = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    gpu_launches = B.gp_launch_count(job.pool.handle) - launches0
    counters = job.check_healthy()
    tokens_local = K * job.nreq
    value, ms = shard.job_throughput(tokens_local, ms_local, device)

    # ---- per-kernel timing pass (CUDA events around every kernel, on the launching stream) -------------------
    job.reset()
    job.roll(S0)
    torch.cuda.synchronize(device)
    moved0 = job.moved_rows()
    by_layer, job.by_layer = job.by_layer, False        # per-kernel times come from the whole-step entry (same kernels)
    B.gp_set_profiling(job.pool.handle, True)
    attn_bytes = score_bytes = 0.0
    n_sum = 0
    for _ in range(K):
        job.step()
        acts = job.act_dev.cpu().numpy()
        a, sc = job.mirror(acts)
        attn_bytes += a
        score_bytes += sc
        n_sum += int(job.n.sum())
    kms, kn = B.gp_get_kernel_times(job.pool.handle)
    B.gp_set_profiling(job.pool.handle, False)
    job.by_layer = by_layer
    moved = job.moved_rows() - moved0
    compact_bytes = 2.0 * moved * (2 * s.head_dim * 2 + 4)
    summ_bytes = float(K) * job.nreq * s.n_layers * 2 * s.n_q_heads * s.head_dim * 8 * 2      # both views, read + write, fp64
    step_bytes = attn_bytes + score_bytes + compact_bytes + summ_bytes
    peak, peak_kind = measured_peak()
    attn_ms = float(kms[1])
    achieved = attn_bytes / (attn_ms * 1e-3) / 1e9
    ratio = traffic_ratio()
    roofline = {
        "bound": "hbm", "kernel": "gp_attn_kernel<128> (append + paged GQA attention + boundary logits)",
        "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s", "frac": round(achieved / peak, 4),
        "peak_kind": f"of {peak_kind}", "frac_of_nominal_8tbs": round(achieved / NOMINAL_HBM_GBS, 4),
        "traffic": None if ratio is None else round(ratio * attn_bytes / K),
        "algorithmic_bytes_per_launch": round(attn_bytes / K),
        "launch_us": round(attn_ms * 1e3 / K, 2),
        "kernel_share_of_step": {name: round(float(kms[i]) / float(kms.sum()), 4) for i, name in enumerate(B.KERNEL_NAMES)},
        "kernel_us_per_step": {name: round(float(kms[i]) * 1e3 / K, 2) for i, name in enumerate(B.KERNEL_NAMES)},
    }
    step_gbs = step_bytes / (ms_local * 1e-3) / 1e9
    step_roofline = {
        "algorithmic_bytes_per_step": round(step_bytes / K),
        "attention": round(attn_bytes / K), "scoring": round(score_bytes / K), "compaction": round(compact_bytes / K),
        "summaries": round(summ_bytes / K),
        "achieved_gbs": round(step_gbs, 1), "frac_of_8tbs": round(step_gbs / NOMINAL_HBM_GBS, 4),
        "frac_of_measured": round(step_gbs / peak, 4), "mean_tokens_per_request": round(n_sum / K / job.nreq, 1),
    }

    # ---- end to end: host buffers, copies inside the timed region -----------------------------------------------
    job.reset()
    job.roll(S0)
    torch.cuda.synchronize(device)
    shard.barrier(device)
    t0 = time.perf_counter()
    for _ in range(K):
        job.step_host()
    torch.cuda.synchronize(device)
    e2e_ms_local = (time.perf_counter() - t0) * 1e3
    shard.barrier(device)
    e2e_value, _ = shard.job_throughput(tokens_local, e2e_ms_local, device)
    h2d = int(s.n_layers * job.nreq * (s.n_q_heads + 2 * s.n_kv_heads) * s.head_dim * 2 + 4 * job.nreq)
    d2h = int(s.n_layers * job.nreq * s.n_q_heads * s.head_dim * 4 + 4 * job.nreq)
    job.check_healthy()

    # ---- CPU baseline: the oracle as it stands, on a bounded sample -------------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = time_oracle(wl, n_requests=8, n_steps=256, warmup=0) if not stack else time_oracle(wl, n_requests=2, n_steps=32, warmup=0)

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": max(Wm, 3),
            "ms_per_step": round(ms / K, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": ("qwen3-8b-stack-resident: L=36, 32q/8kv heads, d=128, page 16, 16 requests x 96 decode "
                                    "steps, prompts U[400,1000], heavy-hitter fraction logU[0.5%,20%], seed 2 (not the headline "
                                    "workload)") if stack else
                                   ("qwen3-8b-layer: L=1, 32q/8kv heads, d=128, page 16, 64 requests x 4096 decode steps, "
                                    "prompts U[128,1024], heavy-hitter fraction logU[0.5%,20%], seed 1"),
                       "entry": "gp_decode_step" if not job.by_layer else "gp_step_begin + gp_attn_layer per layer + gp_step_end",
                       "policy": args.policy, "early_plan": True, "requests_per_gpu": job.nreq, "timed_steps": [S0, S0 + K], "job_steps": job_steps,
                       "l2": "per-step working set (all resident K/V) is larger than L2; no flush needed",
                       "input_generation_s": round(t_gen, 1)},
            "roofline": roofline, "step_roofline": step_roofline,
            "cpu_baseline": cpu,
            "e2e": {"value": round(e2e_value, 1), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms_local / K, 5)},
            "gpu_launches": int(gpu_launches),
            "clocks": clocks,
            "events": {"grow": int(counters[0]), "compress": int(counters[1]), "fallback": int(counters[2]),
                       "stalled": int(counters[3]), "shrink": int(counters[10])},
        }
        print(json.dumps(line))
    job.pool.close()
    shard.finish()


# --------------------------------------------------------------------------------------------------
# the oracle as CPU baseline / reference arm
# --------------------------------------------------------------------------------------------------
def time_oracle(wl, n_requests: int, n_steps: int, warmup: int, budget_s: float = 25.0):
    from oracle import growpage_oracle as O
    from paper_2609_03494_b200 import harness as H
    s = wl.shape
    sub = W.Workload(wl.name, wl.seed, s, wl.requests[:n_requests], n_resident=n_requests,
                     initial_pages=wl.initial_pages, max_pages_per_req=wl.max_pages_per_req,
                     n_pages=n_requests * wl.max_pages_per_req, k_loc=wl.k_loc)
    cfg = O.OracleConfig(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, n_pages=sub.n_pages,
                         max_pages_per_req=sub.max_pages_per_req, k_loc=sub.k_loc, max_requests=max(4, n_requests))
    pool = O.OraclePool(cfg)
    sch = H.Scheduler(sub)
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
    cpu0, wall, done = time.process_time(), 0.0, 0
    for _ in range(n_steps):
        wall += one()
        done += 1
        if wall > budget_s:
            break
    cpu_used = time.process_time() - cpu0
    cores = max(1, int(round(cpu_used / max(wall, 1e-9))))
    return {"value": round(done * n_requests / wall, 2), "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": f"first {n_requests} requests of the workload, decode steps {warmup}..{warmup + done} of the job "
                      f"(float64 numpy, {os.cpu_count()} host cores present, timed region excludes input decoding)",
            "steps": done, "wall_s": round(wall, 4)}


def run_reference(args):
    rank, _, world = shard.env_world()
    if rank != 0:
        return
    wl = W.layer8b(seed=1)
    K, Wm = max(1, args.steps), max(0, args.warmup)
    n_req = 4
    res = time_oracle(wl, n_requests=n_req, n_steps=K, warmup=Wm, budget_s=150.0)
    line = {
        "impl": "reference", "metric": METRIC, "value": res["value"], "unit": "tokens/s", "n_gpus": world,
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=JOB_STEPS)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--entry", default="step", choices=["step", "layers"],
                    help="step: gp_decode_step; layers: the same step through gp_step_begin / gp_attn_layer / gp_step_end")
    ap.add_argument("--workload", default="layer", choices=["layer", "stack"],
                    help="layer: the headline one-layer Qwen3-8B-shaped workload; stack: the 36-layer shape, 16 resident requests")
    ap.add_argument("--policy", default="demand", choices=["demand", "inverse", "random", "shrink"],
                    help="capacity-control policy (the paper's default, or one of its ablation's controls)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
