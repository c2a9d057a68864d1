// Host side of the C ABI, the blob layout, and the small bookkeeping kernels:
// step plan, decision + device allocator, admission, prompt ingest, release, debug gathers.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "../../include/growpage.h"
#include "gp_dev.cuh"

#define GP_PLAN_THREADS 1024
#define GP_NEVER (-(1 << 30))      // bstep of a request that has not reached a boundary

struct gp_pool {
  gp_config cfg;
  int device;
  GpDev dev;
  // asynchronous boundary mode: steps alternate between two sets of the scratch that a step's boundary chain
  // still reads while the next step runs (dev, dev_alt); the chain of a step is launched behind the attention
  // kernel of the next step (or by whatever call needs the pool's pages settled first)
  GpDev dev_alt;
  int chain_pending;                                // the last step's boundary chain has not been launched yet
  int attn_grid_async, chain_grid;
  int attn_grid_ov, chain_grid_ov;                  // synchronous mode with the boundary work beside the attention kernel
  long long serial;                                 // decode steps issued so far
  void* blob;
  size_t bytes;
  std::vector<uint8_t> live;      // host mirror of the slot free list
  int num_sms, attn_grid, sel_grid, compact_grid;
  int step_open, step_n_req, step_layers_done;      // per-layer entry points: a step begun and not yet ended
  std::vector<uint8_t> step_layer_seen;             // layers gp_attn_layer has run in the open step
  // error bits set by the kernels (GP_E_*): one int of page-locked host memory that the device addresses directly,
  // so that the host reads it without a copy once the work that could set it has completed
  int* h_err;
  // staging for the host-pointer entry point (inside the blob)
  int* st_ids; void* st_q; void* st_k; void* st_v; float* st_out; int* st_act;
  // The host entry points fetch a step's inputs on a stream of their own into one of two staging sets, so that the
  // fetch of step t + 1 runs beside the kernels of step t when the caller issues steps ahead.
  int* st2_ids; void* st2_q; void* st2_k; void* st2_v;
  cudaStream_t fetch_stream;                        // inputs in, beside the steps on the caller's stream
  cudaEvent_t ev_fetch[2], ev_used[2], ev_out[2];   // set fetched; its step has run; its results are in the caller's buffers
  long long host_steps;                             // steps issued through the host entry points
  long long host_waited;                            // gp_decode_step_host_async calls whose results have been waited for
  long long host_async_issued;                      // ... and issued
  int host_async_set[2];                            // the staging sets of the (at most two) calls not yet waited for
  __nv_bfloat16* qn; __nv_bfloat16* kn;             // one layer's normalised queries and keys (gp_attn_layer_qknorm)
  // small device words
  int* d_status;
  uint8_t* dbg;                   // gather target of the debug getters
  // measurement
  int profiling;
  cudaStream_t last_stream;       // stream of the last decode step
  int early_plan;                 // gp_set_early_plan: the plan kernel reads the caller's inputs before its wait
  int first_plain;                // the step's first kernel follows a kernel of another kind: plain launch
  int32_t* actions_copy;          // host entry points: the caller's (mapped) array the boundary kernel copies the actions to
  cudaEvent_t ev[GP_N_KERNELS + 1];
  float ms[GP_N_KERNELS];
  int64_t launches[GP_N_KERNELS];
  int64_t launch_count;
};


namespace {

struct Layout {
  size_t kv, tok, refcount, free_stack, words, page_table, shadow, reqi, pos, summ, Kx, Hx, delta, rc,
      mc_list, bnd_info, bnd_acc, free_peek, cmp_info, zbuf, qtil, zstat, sum_par,
      unit_ready, shard_sums, bnd_info2, bnd_acc2, zbuf2, zstat2, rc2, mc_list2, qtil2, rope_cs2,
      evict, evict2, cflags, rope_cs, partials, scores, counters, dbg,
      st_ids, st_q, st_k, st_v, st_out, st_act, st2_ids, st2_q, st2_k, st2_v, qn, kn, total;
  int max_rc;
  long long max_batch_tokens, max_boundary_tokens;
};

inline size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

// Pages per attention work item: 64 (two page ids per producer lane), and half of that for requests at their
// capacity boundary, whose pages also pay for the fp64 logits.  When an attention launch has less than one such
// item of work per CTA (small batches, short sequences; a layer-by-layer launch, which covers one layer's heads
// only), smaller items (32 and 8 pages) keep more CTAs busy (measured: the 36-layer shape with 16 requests,
// layer by layer, takes 1030 us per step that way, 1252 with the large items).
constexpr int GP_CHUNK = 64, GP_BCHUNK = 32;
constexpr int GP_FINE_CHUNK = 32, GP_FINE_BCHUNK = 8;
int chunk_pages_setting() { return GP_CHUNK; }
int bchunk_pages_setting() { return GP_BCHUNK; }

bool valid_config(const gp_config* c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1) return false;
  if (c->n_q_heads % c->n_kv_heads) return false;
  const int G = c->n_q_heads / c->n_kv_heads;
  if (G > 8 || (G & (G - 1))) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  // page_size: 16, 32, ..., 256 tokens; the protected window is one 16-token tile (so it equals the page at 16)
  if (c->page_size < GP_PAGE || c->page_size > GP_MAX_BLK || (c->page_size & (c->page_size - 1))) return false;
  if (c->recent_window != GP_PAGE) return false;
  const long long sub = c->page_size / GP_PAGE;
  if (c->max_requests < 1 || c->max_requests > GP_MAX_REQ) return false;
  if (c->max_pages_per_req < 1 || c->max_pages_per_req * sub > (1 << 20)) return false;
  if (gp_bsel_smem_for_cap(c->max_pages_per_req * sub) > GP_MAX_DYN_SMEM) return false;   // about 61 000 tiles of 16 tokens
  if (c->n_pages < 1 || c->n_pages * sub > 0x7fffffffLL / GP_PAGE) return false;
  if (c->k_loc < 0 || c->k_loc > c->page_size) return false;
  if (c->max_batch_tokens < 0 || c->max_boundary_tokens < 0) return false;
  if (c->demand_metric < GP_METRIC_TOP_P || c->demand_metric > GP_METRIC_ENTROPY) return false;
  if (c->async_boundary < 0 || c->async_boundary > 1 || c->async_slots < 0 || c->async_slots > 4096) return false;
  if (c->overlap_slots < -2 || c->overlap_slots > 4096) return false;
  if (c->kv_shard_count < 1 || c->kv_shard_count > 64 || c->reserved != 0) return false;
  // spread over several pools, the mean of Eq. 8 is completed by adding up integers; the entropy variant sums doubles
  if (c->kv_shard_count > 1 && (c->demand_metric != GP_METRIC_TOP_P || c->async_boundary)) return false;
  if (!(c->beta_s >= 0.0 && c->beta_s < 1.0 && c->beta_l >= 0.0 && c->beta_l < 1.0)) return false;
  if (!(c->top_p > 0.0 && c->top_p < 1.0)) return false;
  if (!(c->rope_theta >= 0.0)) return false;
  if (c->policy < GP_POLICY_DEMAND || c->policy > GP_POLICY_SHRINK) return false;
  if (!(c->p_compress >= 0.0 && c->p_compress <= 1.0)) return false;
  if (c->min_capacity < 0 || !(c->shrink_below == c->shrink_below)) return false;
  return true;
}

Layout make_layout(const gp_config& c) {
  Layout L;
  // everything below is in physical (16-token) pages: a page of the method is `sub` of them
  const size_t sub = (size_t)c.page_size / GP_PAGE, blk = (size_t)c.page_size;
  const size_t M = c.max_requests, cap = (size_t)c.max_pages_per_req * sub, b = GP_PAGE, d = c.head_dim;
  const size_t LH = (size_t)c.n_layers * c.n_kv_heads, G = c.n_q_heads / c.n_kv_heads;
  const size_t np = (size_t)c.n_pages * sub;
  L.max_batch_tokens = c.max_batch_tokens > 0 ? c.max_batch_tokens : (long long)(np * b);
  // candidate tokens of one step's boundary requests: by default every request of a batch may be at its boundary
  // (equal prompts reach it together); a caller that knows better sizes the boundary scratch smaller
  L.max_boundary_tokens = c.max_boundary_tokens > 0 ? c.max_boundary_tokens : L.max_batch_tokens;
  if (L.max_boundary_tokens < (long long)(cap * b) && L.max_batch_tokens >= (long long)(cap * b)) L.max_boundary_tokens = (long long)(cap * b);
  const size_t Tb = (size_t)L.max_boundary_tokens;
  const int ch = chunk_pages_setting();
  int bch = bchunk_pages_setting() < ch ? bchunk_pages_setting() : ch;
  if (bch > GP_FINE_BCHUNK) bch = GP_FINE_BCHUNK;            // small launches cut finer
  L.max_rc = (int)((size_t)L.max_batch_tokens / (b * bch) + 2 * M + 1);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
  L.kv = take(LH * np * 2 * b * d * 2);
  L.tok = take(LH * np * b * 4);
  L.refcount = take(np * 4);
  L.free_stack = take(np * 4);
  L.words = take(256 * 4);                       // free_top, err, plan header, status
  L.page_table = take(M * cap * 4);
  L.shadow = take(M * cap * 4);
  L.reqi = take(8 * M * 4);                      // P, n, started, sum_par, live, n_pristine, bstep, last_act
  L.pos = take(M * 8);
  L.summ = take((size_t)c.n_layers * M * 2 * 2 * c.n_q_heads * d * 8);
  L.Kx = take(M * LH * 2 * 4);
  L.Hx = take(c.demand_metric == GP_METRIC_ENTROPY ? M * LH * 2 * 8 : 16);
  L.delta = take(M * 8);
  L.rc = take((size_t)L.max_rc * GP_DESC_INTS * 4);
  L.mc_list = take(M * 16);
  L.bnd_info = take(M * 32);
  L.bnd_acc = take(M * 16);
  L.unit_ready = take((size_t)M * LH * 4);
  L.shard_sums = take((size_t)M * 2 * 4);
  L.free_peek = take((M + 1) * 4);
  L.cmp_info = take((M + 1) * 16);
  L.zbuf = take(LH * (Tb + b) * 2 * G * 8);
  L.qtil = take(M * LH * 2 * (size_t)G * d * 8);
  L.zstat = take(LH * (Tb / b + 1) * 2 * G * 2 * 8);
  L.evict = take(M * LH * blk * 4);
  L.evict2 = take(c.policy == GP_POLICY_SHRINK ? M * LH * 2 * blk * 4 : 16);
  L.cflags = take(LH * ((Tb + M * b) / GP_MOVE_TOK + 2 * M + 1) * 4);
  L.rope_cs = take(M * (d / 2) * 2 * 8);
  L.partials = take((size_t)L.max_rc * LH * G * (d + 2) * 4);
  L.scores = take((c.policy == GP_POLICY_SHRINK ? 4 : 3) * LH * Tb * 8);
  if (c.async_boundary) {                        // the second set of what a boundary chain reads beside the next step
    L.bnd_info2 = take(M * 32);
    L.bnd_acc2 = take(M * 16);
    L.zbuf2 = take(LH * (Tb + b) * 2 * G * 8);
    L.zstat2 = take(LH * (Tb / b + 1) * 2 * G * 2 * 8);
    // and of what the plan of a step writes while the attention kernel of the step before may still read its own
    L.rc2 = take((size_t)L.max_rc * GP_DESC_INTS * 4);
    L.mc_list2 = take(M * 16);
    L.qtil2 = take(M * LH * 2 * (size_t)G * d * 8);
    L.rope_cs2 = take(M * (d / 2) * 2 * 8);
  } else {
    L.bnd_info2 = L.bnd_acc2 = L.zbuf2 = L.zstat2 = L.rc2 = L.mc_list2 = L.qtil2 = L.rope_cs2 = 0;
  }
  L.counters = take(16 * 8);
  L.dbg = take(cap * b * (4 + 2 * d * 2));
  if (c.host_staging) {
    L.st_ids = take(M * 4);
    L.st_q = take((size_t)c.n_layers * M * c.n_q_heads * d * 2);
    L.st_k = take((size_t)c.n_layers * M * c.n_kv_heads * d * 2);
    L.st_v = take((size_t)c.n_layers * M * c.n_kv_heads * d * 2);
    L.st2_ids = take(M * 4);
    L.st2_q = take((size_t)c.n_layers * M * c.n_q_heads * d * 2);
    L.st2_k = take((size_t)c.n_layers * M * c.n_kv_heads * d * 2);
    L.st2_v = take((size_t)c.n_layers * M * c.n_kv_heads * d * 2);
    L.st_out = take((size_t)c.n_layers * M * c.n_q_heads * d * 4);
    L.st_act = take(M * 4);
  } else {
    L.st_ids = L.st_q = L.st_k = L.st_v = L.st_out = L.st_act = L.st2_ids = L.st2_q = L.st2_k = L.st2_v = 0;
  }
  L.qn = take(M * c.n_q_heads * d * 2);              // one layer's normalised queries and keys (fused QK-norm)
  L.kn = take(M * c.n_kv_heads * d * 2);
  L.total = o;
  return L;
}

// ---------------------------------------------------------------------------------------------------
// kernels
// ---------------------------------------------------------------------------------------------------
__global__ void gp_init_kernel(GpDev p) {
  const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long stride = (long long)gridDim.x * blockDim.x;
  // page 0 is handed out first
  for (long long i = i0; i < p.n_pages; i += stride) p.free_stack[i] = (int)(p.n_pages - 1 - i);
  for (long long i = i0; i < (long long)p.M * p.cap; i += stride) p.shadow[i] = -1;
  for (long long i = i0; i < p.M; i += stride) p.bstep[i] = GP_NEVER;
  if (i0 == 0) *p.free_top = (int)p.n_pages;
}

// exclusive scan over the CTA (1024 threads) of an int and a long long; also returns the totals
__device__ __forceinline__ void plan_scan(int v, long long w, int& ev, long long& ew, int& tv, long long& tw,
                                          int* sv, long long* sw) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int iv = v; long long iw = w;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int a = __shfl_up_sync(0xffffffffu, iv, off);
    const long long b2 = __shfl_up_sync(0xffffffffu, iw, off);
    if (lane >= off) { iv += a; iw += b2; }
  }
  if (lane == 31) { sv[warp] = iv; sw[warp] = iw; }
  __syncthreads();
  if (warp == 0) {                       // scan of the 32 warp totals: exclusive prefix in [0..31], total in [32]
    int xv = sv[lane]; long long xw = sw[lane];
    const int ov = xv; const long long ow = xw;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, xv, off);
      const long long b2 = __shfl_up_sync(0xffffffffu, xw, off);
      if (lane >= off) { xv += a; xw += b2; }
    }
    sv[lane] = xv - ov; sw[lane] = xw - ow;
    if (lane == 31) { sv[32] = xv; sw[32] = xw; }
  }
  __syncthreads();
  ev = sv[warp] + iv - v;
  ew = sw[warp] + iw - w;
  tv = sv[32];
  tw = sw[32];
  __syncthreads();
}

// Fused QK-norm of the layer-by-layer entry (null weights: queries and keys arrive normalised).  Queries and keys
// of the call are raw; the summary CTAs, which read every query row anyway, normalise them per head (RMS over the
// head dimension, a learned weight per element), rotate the key to its cache form and leave both, rounded to
// bf16, where the attention kernel then finds them.
struct GpNorm {
  const float* wq; const float* wk;
  double eps;
  const __nv_bfloat16* k_raw;
  __nv_bfloat16* qn; __nv_bfloat16* kn;
};

// double -> float -> bf16, each round-to-nearest-even (the order a host library takes)
__device__ __forceinline__ __nv_bfloat16 to_bf16(double x) { return __float2bfloat16_rn((float)x); }

// Summary update of one (batch slot, layer, KV head) unit, run by the CTAs of the plan kernel other than the
// first, concurrently with the planning: Eq. 6 on the un-rotated query of every head of the group (read from
// one of the request's two buffers, written to the other; the decision step flips the buffers of the requests
// that were really stepped, so a unit that turns out not to step leaves no trace), and, for a request that
// reaches its capacity boundary, the calibrated (Eq. 12) and rotated summaries q~ in fp64 for the attention
// kernel's logits.  One warp per (view, head) row; a CTA takes as many units at a time as its warps cover.
template <int D>
__device__ void prepare_row(const GpDev& p, int n_req, const __nv_bfloat16* __restrict__ q, int bi, int lh, int row, int r,
                            int n_old, int Pr, int started, int par, long long pos, const GpNorm& nm) {
  constexpr int PER = D / 32;
  const int lane = threadIdx.x & 31;
  const int G = p.G;
  const int l = lh / p.Hkv, h = lh % p.Hkv;
  const int x = row / G, g = row % G;
  const int head = h * G + g;
  // one round trip: the query row and the old summary from the request's current buffer (the request's state
  // was staged in shared memory by the CTA)
  const __nv_bfloat16* qrow = q + (((size_t)l * n_req + bi) * p.Hq + head) * D;
  float qf[PER];
#pragma unroll
  for (int e = 0; e < PER; ++e) qf[e] = __bfloat162float(qrow[lane + 32 * e]);
  if (nm.wq) {
    // the raw query row becomes the normalised one (Sec. 3.2: the summaries follow the query after its
    // normalisation and before its rotation); the short view's warp leaves it for the attention kernel
    double ssq = 0.0;
#pragma unroll
    for (int e = 0; e < PER; ++e) ssq += (double)qf[e] * (double)qf[e];
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) ssq += __shfl_xor_sync(0xffffffffu, ssq, o2);
    const double scale = 1.0 / sqrt(ssq / (double)D + nm.eps);
    __nv_bfloat16* qout = nm.qn + (((size_t)l * n_req + bi) * p.Hq + head) * D;
#pragma unroll
    for (int e = 0; e < PER; ++e) {
      const __nv_bfloat16 v = to_bf16((double)qf[e] * scale * (double)nm.wq[lane + 32 * e]);
      qf[e] = __bfloat162float(v);
      if (x == 0) qout[lane + 32 * e] = v;
    }
    if (row == 0) {                        // the unit's key row: normalise, rotate to the token's position, leave
      const __nv_bfloat16* krow = nm.k_raw + (((size_t)l * n_req + bi) * p.Hkv + h) * D;
      double kv[PER];
      double ks = 0.0;
#pragma unroll
      for (int e = 0; e < PER; ++e) { kv[e] = (double)__bfloat162float(krow[lane + 32 * e]); ks += kv[e] * kv[e]; }
#pragma unroll
      for (int o2 = 16; o2 > 0; o2 >>= 1) ks += __shfl_xor_sync(0xffffffffu, ks, o2);
      const double kscale = 1.0 / sqrt(ks / (double)D + nm.eps);
#pragma unroll
      for (int e = 0; e < PER; ++e) kv[e] = kv[e] * kscale * (double)nm.wk[lane + 32 * e];
      __nv_bfloat16* kout = nm.kn + (((size_t)l * n_req + bi) * p.Hkv + h) * D;
      if (p.rope_theta != 0.0) {
#pragma unroll
        for (int e = 0; e < PER / 2; ++e) {
          const int j = lane + 32 * e;
          const double inv = pow(p.rope_theta, -2.0 * (double)j / (double)D);
          double si, co;
          sincos((double)pos * inv, &si, &co);
          kout[j] = to_bf16(kv[e] * co - kv[e + PER / 2] * si);
          kout[j + D / 2] = to_bf16(kv[e + PER / 2] * co + kv[e] * si);
        }
      } else {
#pragma unroll
        for (int e = 0; e < PER; ++e) kout[lane + 32 * e] = to_bf16(kv[e]);
      }
    }
  }
  double ovv[PER];
  {
    const double* o0 = p.summ + gp_summ_off(p, l, r, par, x, head);
#pragma unroll
    for (int e = 0; e < PER; ++e) ovv[e] = __ldcg(o0 + lane + 32 * e);
  }
  const bool need_qt = (n_old + 1 == Pr * GP_PAGE) && Pr > 1;
  {
    const double beta = x ? p.beta_l : p.beta_s;
    double* newp = p.summ + gp_summ_off(p, l, r, par ^ 1, x, head);
    double nv[PER];
    double sq = 0.0, ss = 0.0;
#pragma unroll
    for (int e = 0; e < PER; ++e) {
      const double qv = (double)qf[e];
      const double ov = ovv[e];
      sq += qv * qv;
      nv[e] = started ? beta * ov + (1.0 - beta) * qv : qv;              // Eq. 6
      newp[lane + 32 * e] = nv[e];
      ss += nv[e] * nv[e];
    }
    if (need_qt) {
#pragma unroll
      for (int o2 = 16; o2 > 0; o2 >>= 1) {
        sq += __shfl_xor_sync(0xffffffffu, sq, o2);
        ss += __shfl_xor_sync(0xffffffffu, ss, o2);
      }
      // Eq. 12
      const double gamma = ss > 0.0 ? sqrt(sq / (double)D) / sqrt(ss / (double)D) : 1.0;
      double* dst = p.qtil + (((size_t)bi * p.L * p.Hkv + lh) * 2 * G + row) * D;
      if (p.rope_theta != 0.0) {
#pragma unroll
        for (int e = 0; e < PER / 2; ++e) {
          const int j = lane + 32 * e;
          const double inv = pow(p.rope_theta, -2.0 * (double)j / (double)D);
          double si, co;
          sincos((double)pos * inv, &si, &co);
          const double x1 = gamma * nv[e], x2 = gamma * nv[e + PER / 2];
          dst[j] = x1 * co - x2 * si;
          dst[j + D / 2] = x2 * co + x1 * si;
        }
      } else {
#pragma unroll
        for (int e = 0; e < PER; ++e) dst[lane + 32 * e] = gamma * nv[e];
      }
    }
  }
}

// Step plan: validates the batch, cuts every stepped request into chunks and writes one work descriptor
// per chunk for the attention kernel, lists the requests that reach their capacity boundary with this
// step's append (trailing check: n + 1 == P b) and hands each a slice of the logit scratch.
__global__ void __launch_bounds__(GP_PLAN_THREADS)
gp_plan_kernel(const __grid_constant__ GpDev p, const int* __restrict__ req_ids, int n_req, int* __restrict__ actions,
               const __nv_bfloat16* __restrict__ q, int plan_on, int lh0, int lh_n, int cp_norm, int cp_bnd,
               int launch_units, int launch_grid, int serial, const GpNorm nm) {
  // serial: number of this decode step (asynchronous boundary mode: a request that reached its boundary at
  // step serial - 1 sits this step out; its counters and pages belong to that step's boundary chain, which may
  // still be running)
  // cp_norm, cp_bnd: pages per work item, for requests in general and for those at their capacity boundary, when
  // the attention launch has work for large items; launch_units: (layer, head) units per request in one
  // attention launch; launch_grid: its CTAs
  // plan_on: 0: no planning (the per-layer calls after the step's first); 1: CTA 0 plans; 2: CTA 0 plans and
  // the caller's inputs may be read before the wait for the preceding kernel (see below).  The summary CTAs
  // cover the (layer, KV head) units [lh0, lh0 + lh_n) (none when lh_n is 0: the query rows come layer by layer)
  __shared__ int sv[33];
  __shared__ long long sw[33];
  __shared__ __align__(16) int s_first[GP_MAX_REQ];      // lowest batch index naming a request
  __shared__ int s_chunks[GP_MAX_REQ], s_pos[GP_MAX_REQ];
  __shared__ int s_req[GP_MAX_REQ], s_state[GP_MAX_REQ];     // summary CTAs: request of a batch slot, flags
  __shared__ long long s_pos64[GP_MAX_REQ];
  __shared__ int s_bin[GP_COST_BINS], s_binbase[GP_COST_BINS], s_nmc;
  const int i = threadIdx.x;
  const bool in = i < n_req;
  // What runs before the wait for the kernel before this one.  In a whole-step launch that kernel is the
  // compaction of the step before (or something the caller put in between, which then has completed): this
  // grid became schedulable only after that step's decisions had completed, and compaction touches neither the
  // requests' counters, nor the summaries, nor anything the plan writes except the step stamp.  So the summary
  // CTAs do not wait at all, and CTA 0 plans the whole step first and waits only before it looks at the free
  // list (which compaction's last CTA may still change) and stamps the step.  CTA 0 does wait, so the grid as
  // a whole still ends after everything before it.  The layer-by-layer launches (plan_on == 0) have no CTA 0
  // work and keep the wait in every CTA, so that completion stays transitive.  The next kernel may be scheduled
  // as soon as every CTA of this grid has started; it waits for this grid's end at its own top.
  // All of this reads the caller's request ids and queries before the wait, which is only right if they were
  // complete before the preceding kernel could signal: the caller says so (plan_on == 2); otherwise every CTA
  // waits first (the later wait of CTA 0 is then a no-op).
  if (plan_on != 2) gp_pdl_wait();
  gp_pdl_launch_dependents();
  if (blockIdx.x > 0) {                       // summary CTAs: one warp per (unit, view, head)
    // The state of the batch's requests is staged once per CTA, from the L2 (these CTAs may run before the wait,
    // and an L1 line could date from the step before): request of a slot (-1: not stepped by these CTAs:
    // out of range, dead, or named by an earlier slot), tokens, pages, flags, position.
    if (i < GP_MAX_REQ) s_first[i] = 0x7fffffff;
    __syncthreads();
    int r = -1;
    if (in) {
      r = req_ids[i];
      if (r >= 0 && r < p.M) atomicMin(&s_first[r], i); else r = -1;
    }
    __syncthreads();
    if (in) {
      int ok = 0;
      if (r >= 0 && s_first[r] == i && __ldcg(p.live + r) && !(p.async && __ldcg(p.bstep + r) == serial - 1)) {
        ok = 1;
        s_chunks[i] = __ldcg(p.n + r);
        s_pos[i] = __ldcg(p.P + r);
        s_state[i] = (__ldcg(p.started + r) ? 1 : 0) | (__ldcg(p.sum_par + r) ? 2 : 0);
        s_pos64[i] = __ldcg(p.pos + r);
      }
      s_req[i] = ok ? r : -1;
    }
    __syncthreads();
    const int rows = 2 * p.G, upc = 32 / rows;             // units per CTA and pass
    const int warp = threadIdx.x >> 5;
    const long long units = (long long)n_req * lh_n;
    if (warp < upc * rows) {
      for (long long u = ((long long)blockIdx.x - 1) * upc + warp / rows; u < units; u += ((long long)gridDim.x - 1) * upc) {
        const int bi = (int)(u / lh_n), lh = lh0 + (int)(u % lh_n);
        const int rr = s_req[bi];
        if (rr < 0) continue;
        const int st = s_state[bi];
        if (p.d == 128) prepare_row<128>(p, n_req, q, bi, lh, warp % rows, rr, s_chunks[bi], s_pos[bi], st & 1, (st >> 1) & 1, s_pos64[bi], nm);
        else prepare_row<64>(p, n_req, q, bi, lh, warp % rows, rr, s_chunks[bi], s_pos[bi], st & 1, (st >> 1) & 1, s_pos64[bi], nm);
      }
    }
    return;
  }
  if (!plan_on) return;
  s_first[i] = 0x7fffffff;
  if (i < GP_COST_BINS) s_bin[i] = 0;
  if (i == 0) s_nmc = 0;
  // The number this step goes by: the host's count of decode steps in the asynchronous mode (the two scratch sets
  // count on their own); otherwise the pool's own counter on the device, so that a step replayed from a CUDA graph
  // still gets a number of its own.
  const int step_no = p.async ? serial : __ldcg(p.hdr + HDR_STEP);
  __syncthreads();
  int r = -1;
  if (in) {
    r = req_ids[i];
    if (r >= 0 && r < p.M) atomicMin(&s_first[r], i);
  }
  __syncthreads();
  int chunks = 0, pages = 0, n_old = 0, act = GP_ACT_NONE, Pr = 0, started = 0, par = 0;
  long long nc = 0, pos = 0;
  int isb = 0;
  int cp = cp_norm;                       // pages per work item of this request
  int live = 0, held = 0;
  if (in && r >= 0 && r < p.M) {          // independent loads, issued together (from the L2: before the wait)
    live = __ldcg(p.live + r); n_old = __ldcg(p.n + r); Pr = __ldcg(p.P + r); pos = __ldcg(p.pos + r);
    started = __ldcg(p.started + r); par = __ldcg(p.sum_par + r);
    if (p.async) held = __ldcg(p.bstep + r) == serial - 1;
  }
  if (in) {
    const bool inrange = r >= 0 && r < p.M;
    const bool valid = inrange && live && s_first[r] == i;
    if (!valid) {
      act = GP_ACT_INVALID;
    } else if (held) {
      act = GP_ACT_HELD;                  // its boundary chain may still be running: nothing of it is looked at
    } else if (n_old >= Pr * GP_PAGE) {
      act = GP_ACT_STALLED;
    } else {
      pages = n_old / GP_PAGE + 1;
      if (n_old + 1 == Pr * GP_PAGE) { isb = 1; nc = (long long)(Pr - 1) * GP_PAGE; }
    }
  }
  {
    // Large items when an attention launch has at least one of them per CTA (pages of the batch x units per
    // request / CTAs >= an item), fine ones otherwise: small batches, short sequences, layer-by-layer launches.
    // Measured on one layer of the 8B shape: 8 to 48 requests of 30 to 50 pages are 2 to 8 us per step faster
    // with fine items, 64 requests of 44 pages and more 3 us faster with large ones.
    int e0, tot_pages; long long d0, d1;
    plan_scan(pages, 0, e0, d0, tot_pages, d1, sv, sw);
    if ((long long)tot_pages * launch_units < (long long)cp_norm * launch_grid) { cp_norm = GP_FINE_CHUNK; cp_bnd = GP_FINE_BCHUNK; }
  }
  if (pages > 0) {
    // a page of a boundary request also pays for the fp64 summary logits: its items are half as large
    // (measured best: 16, 24, 40 and 48 pages against 64 for the others were all slower)
    cp = isb ? cp_bnd : cp_norm;
    chunks = (pages + cp - 1) / cp;
    cp = (pages + chunks - 1) / chunks;              // equal sizes: chunks of cp pages, the last one shorter
  }
  int rc_off, n_rc; long long tok_off, tok_tot;
  plan_scan(chunks, nc, rc_off, tok_off, n_rc, tok_tot, sv, sw);
  // A batch whose summed lengths exceed max_batch_tokens (the caller's bound; with shared prompt pages the sum
  // can exceed what the pool holds) does not fit the scratch: a request whose boundary logits or whose work
  // items do not fit is not stepped (its state stays as it is, it can be stepped again in a later batch).  The
  // offsets are then taken again over what is left, so that the item list has no holes.
  const bool dropped = chunks > 0 && ((isb && tok_off + nc > p.max_boundary_tokens) || rc_off + chunks > p.max_rc);
  if (dropped) { chunks = 0; isb = 0; nc = 0; act = GP_ACT_SCRATCH; }
  if (__syncthreads_or(dropped)) plan_scan(chunks, nc, rc_off, tok_off, n_rc, tok_tot, sv, sw);
  int bnd_idx, n_bnd, n_active; long long d0, d1;
  plan_scan(isb, chunks > 0, bnd_idx, d0, n_bnd, d1, sv, sw);
  n_active = (int)d1;
  // Work items are listed by descending cost (pages, times four for boundary requests, which also pay for the
  // fp64 logits): the attention kernel deals them out in that order, largest first.  Counting sort.
  const int key = chunks > 0 ? min(GP_COST_BINS - 1, cp * (isb ? 4 : 1)) : 0;
  // Items of equal cost keep the batch's order (a rank counted over the earlier batch slots, not the order in
  // which atomics land), so that the same batch is dealt to the thread blocks the same way every time and the
  // attention outputs repeat bit for bit.
  s_first[i] = chunks > 0 ? (key << 16) | chunks : 0;        // s_first has served its purpose: cost class and items
  if (chunks > 0) atomicAdd(&s_bin[key], chunks);
  __syncthreads();
  int within = 0;
  if (chunks > 0) {
    const int4* e4 = reinterpret_cast<const int4*>(s_first);
    int j = 0;
    for (; j + 4 <= i; j += 4) {
      const int4 e = e4[j >> 2];
      within += ((e.x >> 16) == key ? (e.x & 0xffff) : 0) + ((e.y >> 16) == key ? (e.y & 0xffff) : 0) +
                ((e.z >> 16) == key ? (e.z & 0xffff) : 0) + ((e.w >> 16) == key ? (e.w & 0xffff) : 0);
    }
    for (; j < i; ++j) { const int e = s_first[j]; within += (e >> 16) == key ? (e & 0xffff) : 0; }
  }
  __syncthreads();
  if (threadIdx.x < 32) {                             // descending exclusive scan over the cost bins
    int carry = 0;
    for (int b0 = GP_COST_BINS - 32; b0 >= 0; b0 -= 32) {
      const int b = b0 + 31 - (int)threadIdx.x;       // lane 0 takes the costliest bin of the block of 32
      const int v = s_bin[b];
      int inc = v;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, inc, off);
        if ((int)threadIdx.x >= off) inc += a;
      }
      s_binbase[b] = carry + inc - v;
      carry += __shfl_sync(0xffffffffu, inc, 31);
    }
  }
  __syncthreads();
  const int sorted0 = s_binbase[key] + within;
  s_chunks[i] = chunks; s_pos[i] = (int)pos;
  if (in) {
    if (isb) { p.bstep[r] = step_no; if (p.async) act = GP_ACT_PENDING; }
    actions[i] = act;
    if (isb) {
      p.bnd_info[2 * bnd_idx] = make_int4(i, r, Pr, (int)pos);     // pos: position of this step's token
      // .z: reports the attention kernel makes per (layer, head) unit of this request (one per consumer warp and item)
      p.bnd_info[2 * bnd_idx + 1] = make_int4((int)(unsigned)(tok_off & 0xffffffffLL), (int)(tok_off >> 32), GP_ATTN_CONSUMERS * chunks, 0);
      reinterpret_cast<int4*>(p.bnd_acc)[bnd_idx] = make_int4(0, 0, 0, 0);
    }
    // descriptors of this request's chunks: four 16-byte stores each
    const int flags = isb | (started ? 2 : 0);
    for (int c = 0; c < chunks; ++c) {
      const int pg0 = c * cp;
      int4* d = reinterpret_cast<int4*>(p.rcx + (size_t)(sorted0 + c) * GP_DESC_INTS);
      d[0] = make_int4(i, r, pg0, min(cp, pages - pg0));
      d[1] = make_int4(c, chunks, n_old, (int)pos);
      d[2] = make_int4(flags, Pr, (int)(unsigned)(tok_off & 0xffffffffLL), (int)(tok_off >> 32));
      d[3] = make_int4(par, rc_off + c, 0, isb ? bnd_idx : 0);
    }
    if (chunks > 1) p.mc_list[atomicAdd(&s_nmc, 1)] = make_int4(i, rc_off, chunks, 0);
  }
  __syncthreads();
  if (p.rope_theta != 0.0) {                                      // cos / sin of the step's position
    __syncthreads();
    const int half = p.d / 2;
    for (int idx = threadIdx.x; idx < n_req * half; idx += GP_PLAN_THREADS) {
      const int bi = idx / half, j = idx % half;
      if (s_chunks[bi] > 0) {
        const double inv = pow(p.rope_theta, -2.0 * (double)j / (double)p.d);
        const double ang = (double)s_pos[bi] * inv;
        double sn, cs;
        sincos(ang, &sn, &cs);
        p.rope_cs[(size_t)idx * 2] = cs;
        p.rope_cs[(size_t)idx * 2 + 1] = sn;
      }
    }
  }
  // the attention kernel counts, per unit of a boundary request, the work items its consumer warps have finished
  for (int idx = threadIdx.x; idx < n_bnd * p.L * p.Hkv; idx += GP_PLAN_THREADS) p.unit_ready[idx] = 0;
  __syncthreads();
  if (threadIdx.x == 0) {
    p.hdr[HDR_N_MC] = s_nmc;
    p.hdr[HDR_N_RC] = n_rc;
    p.hdr[HDR_N_BND] = n_bnd;
    p.hdr[HDR_N_ACTIVE] = n_active;
  }
  // ---- from here on the kernel before this one has completed --------------------------------------------
  gp_pdl_wait();
  if (!p.async) {
    // the top of the free list, one page per boundary request: what this step's grants can take.  (In the
    // asynchronous mode the free list belongs to the boundary chains, which run one after the other: the
    // decision step reads it itself.)
    const int free_top0 = *p.free_top;
    if (in && isb && bnd_idx < free_top0) p.free_peek[1 + bnd_idx] = p.free_stack[free_top0 - 1 - bnd_idx];
    if (threadIdx.x == 0) p.free_peek[0] = free_top0;
  }
  if (threadIdx.x == 0) p.hdr[HDR_STEP] += 1;
}

__global__ void gp_admit_kernel(GpDev p, int r, int share_from, int n_shared, int n_tail, int P_target, int* status) {
  const int lane = threadIdx.x;
  const int need = P_target - n_shared;
  const int top = *p.free_top;
  // refusals in a fixed order: what is wrong with the arguments, then the slot, then the pages
  int st = GP_OK;
  if (n_shared > 0 && (!p.live[share_from] || p.n_pristine[share_from] < n_shared)) st = GP_ERR_INVALID;
  else if (r < 0) st = GP_ERR_NO_SLOT;
  else if (need > top || P_target > p.cap) st = GP_ERR_NO_PAGES;
  __syncwarp();
  if (st == GP_OK) {
    int* table = p.page_table + (size_t)r * p.cap;
    for (int j = lane; j < n_shared; j += 32) {
      const int page = p.page_table[(size_t)share_from * p.cap + j];
      table[j] = page;
      atomicAdd(&p.refcount[page], 1);
    }
    for (int j = lane; j < need; j += 32) {
      const int page = p.free_stack[top - 1 - j];
      table[n_shared + j] = page;
      p.refcount[page] = 1;
    }
    __syncwarp();
    if (lane == 0) {
      const int n0 = n_shared * GP_PAGE + n_tail;
      *p.free_top = top - need;
      p.P[r] = P_target; p.n[r] = n0; p.pos[r] = n0; p.started[r] = 0; p.live[r] = 1;
      p.bstep[r] = GP_NEVER; p.last_act[r] = GP_ACT_NONE;
      p.n_pristine[r] = (n0 / p.blk) * p.sub;                 // only full pages of the method can be shared
    }
  }
  if (lane == 0) *status = st;
}

// copies the private part of a prompt into its pages: one thread per 16-byte chunk
__global__ void gp_ingest_kernel(GpDev p, int r, int n_shared, int n_tail, const __nv_bfloat16* k_tail,
                                 const __nv_bfloat16* v_tail) {
  const int CH = p.d / 8;
  const long long total = (long long)p.L * n_tail * p.Hkv * 2 * CH;
  const int row_bytes = p.d * 2;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % CH);
    long long t2 = idx / CH;
    const int isv = (int)(t2 % 2); t2 /= 2;
    const int h = (int)(t2 % p.Hkv); t2 /= p.Hkv;
    const int t = (int)(t2 % n_tail);
    const int l = (int)(t2 / n_tail);
    const __nv_bfloat16* src = (isv ? v_tail : k_tail) + (((size_t)l * n_tail + t) * p.Hkv + h) * p.d + c * 8;
    const int slot = n_shared * GP_PAGE + t;
    const int page = p.page_table[(size_t)r * p.cap + slot / GP_PAGE];
    const int s = slot % GP_PAGE;
    uint8_t* dst = reinterpret_cast<uint8_t*>(p.kv + gp_tile_off(p, l, page, h)) + isv * GP_PAGE * row_bytes +
                   s * row_bytes + ((c ^ (s & 7)) << 4);
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
    if (isv == 0 && c == 0) p.tok[gp_tok_off(p, l, page, h) + s] = slot;
  }
}

__global__ void gp_release_kernel(GpDev p, int r) {
  const int lane = threadIdx.x;
  const int Pr = p.P[r];
  const int* table = p.page_table + (size_t)r * p.cap;
  for (int j0 = 0; j0 < Pr; j0 += 32) {
    const int j = j0 + lane;
    bool freed = false;
    int page = -1;
    if (j < Pr) {
      page = table[j];
      freed = (atomicSub(&p.refcount[page], 1) == 1);
    }
    const unsigned mask = __ballot_sync(0xffffffffu, freed);
    int base = 0;
    if (lane == 0) base = *reinterpret_cast<volatile int*>(p.free_top);
    base = __shfl_sync(0xffffffffu, base, 0);
    if (freed) p.free_stack[base + __popc(mask & ((1u << lane) - 1u))] = page;
    __syncwarp();
    if (lane == 0 && mask) *reinterpret_cast<volatile int*>(p.free_top) = base + __popc(mask);
    __syncwarp();
  }
  if (lane == 0) {
    p.live[r] = 0; p.P[r] = 0; p.n[r] = 0; p.started[r] = 0; p.n_pristine[r] = 0; p.bstep[r] = GP_NEVER;
  }
}

// debug: token ids and un-swizzled K, V rows of one (layer, head) stream into the gather buffer
__global__ void gp_gather_kernel(GpDev p, int r, int l, int h, int n, int* tok_out, uint4* k_out, uint4* v_out) {
  const int CH = p.d / 8;
  const int row_bytes = p.d * 2;
  const long long total = (long long)n * 2 * CH;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % CH);
    const int isv = (int)((idx / CH) % 2);
    const int slot = (int)(idx / (2 * CH));
    const int page = p.page_table[(size_t)r * p.cap + slot / GP_PAGE];
    const int s = slot % GP_PAGE;
    const uint8_t* src = reinterpret_cast<const uint8_t*>(p.kv + gp_tile_off(p, l, page, h)) +
                         isv * GP_PAGE * row_bytes + s * row_bytes + ((c ^ (s & 7)) << 4);
    (isv ? v_out : k_out)[(size_t)slot * CH + c] = *reinterpret_cast<const uint4*>(src);
    if (isv == 0 && c == 0) tok_out[slot] = p.tok[gp_tok_off(p, l, page, h) + s];
  }
}

#define GP_CUDA(x)                      \
  do {                                  \
    if ((x) != cudaSuccess) return GP_ERR_CUDA; \
  } while (0)

void pool_free(gp_pool* pool) {
  if (pool->h_err) cudaFreeHost(pool->h_err);
  if (pool->fetch_stream) {
    cudaStreamDestroy(pool->fetch_stream);
    for (int i = 0; i < 2; ++i) { cudaEventDestroy(pool->ev_fetch[i]); cudaEventDestroy(pool->ev_used[i]); cudaEventDestroy(pool->ev_out[i]); }
  }
  delete pool;
}

// Asynchronous boundary mode: launches the boundary chain of the last decode step on `s` if it has not been
// launched yet (it normally rides behind the next step's attention kernel).  Everything that looks at the pool's
// pages, counters or free list from outside a decode step calls this first.
int flush_chain(gp_pool* pool, cudaStream_t s) {
  if (!pool->cfg.async_boundary || !pool->chain_pending) return GP_OK;
  const long long t = pool->serial - 1;                       // the step the chain belongs to
  const GpDev& d = (t & 1) ? pool->dev_alt : pool->dev;
  gp_launch_chain(d, d, 0, nullptr, (int)(t & 0x3fffffff), 1, pool->chain_grid, s, false);
  pool->chain_pending = 0;
  pool->launch_count += 1;
  return cudaGetLastError() == cudaSuccess ? GP_OK : GP_ERR_CUDA;
}

// the kernels' error bits, once the work that could set them has completed
int kernel_status(const gp_pool* pool) {
  return *reinterpret_cast<volatile const int*>(pool->h_err) ? GP_ERR_CUDA : GP_OK;
}

bool misaligned(const void* ptr, uintptr_t a) { return (reinterpret_cast<uintptr_t>(ptr) & (a - 1)) != 0; }

int check_req(gp_pool* pool, int32_t req) {
  if (!pool) return GP_ERR_INVALID;
  if (req < 0 || req >= pool->cfg.max_requests || !pool->live[req]) return GP_ERR_INVALID;
  return GP_OK;
}

}  // namespace

// ===================================================================================================
// C ABI
// ===================================================================================================
extern "C" {

int gp_config_default(gp_config* cfg) {
  if (!cfg) return GP_ERR_INVALID;
  memset(cfg, 0, sizeof(*cfg));
  cfg->page_size = GP_PAGE;
  cfg->max_requests = 512;
  cfg->recent_window = GP_PAGE;
  cfg->kv_shard_count = 1;
  cfg->k_loc = GP_PAGE / 4;          // a quarter of the page; the paper's 64 at its page size of 256
  cfg->beta_s = 0.9;
  cfg->beta_l = 0.999;
  cfg->top_p = 0.99;
  cfg->tau = 0.0;
  cfg->rope_theta = 0.0;
  cfg->policy = GP_POLICY_DEMAND;
  cfg->policy_seed = 0;
  cfg->p_compress = 0.7;
  cfg->shrink_below = -0.005;
  cfg->min_capacity = 1024;
  return GP_OK;
}

size_t gp_pool_bytes(const gp_config* cfg) {
  if (!valid_config(cfg)) return 0;
  return make_layout(*cfg).total;
}

int gp_pool_create(const gp_config* cfg, void* dev_blob, size_t bytes, int device, gp_pool** out) {
  if (!out) return GP_ERR_INVALID;
  *out = nullptr;
  if (!valid_config(cfg) || !dev_blob || ((uintptr_t)dev_blob & 255)) return GP_ERR_INVALID;
  const Layout L = make_layout(*cfg);
  if (bytes < L.total) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(device));
  gp_pool* pool = new (std::nothrow) gp_pool();
  if (!pool) return GP_ERR_STATE;
  pool->cfg = *cfg;
  pool->device = device;
  pool->blob = dev_blob;
  pool->bytes = bytes;
  pool->live.assign(cfg->max_requests, 0);
  pool->profiling = 0;
  pool->early_plan = 0;
  pool->first_plain = 0;
  pool->step_open = 0; pool->step_n_req = 0; pool->step_layers_done = 0;
  pool->step_layer_seen.assign(cfg->n_layers, 0);
  pool->h_err = nullptr;
  pool->launch_count = 0;
  pool->serial = 0;
  memset(pool->ms, 0, sizeof(pool->ms));
  memset(pool->launches, 0, sizeof(pool->launches));
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { pool_free(pool); return GP_ERR_CUDA; }
  pool->num_sms = prop.multiProcessorCount;
  pool->attn_grid = pool->num_sms * gp_attention_ctas_per_sm(cfg->head_dim);

  uint8_t* base = static_cast<uint8_t*>(dev_blob);
  GpDev& d = pool->dev;
  d.L = cfg->n_layers; d.Hq = cfg->n_q_heads; d.Hkv = cfg->n_kv_heads; d.G = cfg->n_q_heads / cfg->n_kv_heads;
  d.sub = cfg->page_size / GP_PAGE; d.blk = cfg->page_size;
  d.d = cfg->head_dim; d.M = cfg->max_requests; d.cap = cfg->max_pages_per_req * d.sub; d.k_loc = cfg->k_loc;
  d.chunk_pages = chunk_pages_setting(); d.max_rc = L.max_rc;
  d.bchunk_pages = bchunk_pages_setting();
  d.n_pages = cfg->n_pages * d.sub; d.max_batch_tokens = L.max_batch_tokens;
  d.max_boundary_tokens = L.max_boundary_tokens;
  d.async = cfg->async_boundary;
  d.spin_limit = GP_SPIN_LIMIT;
  d.withhold = 0;
  d.z_stride = (L.max_boundary_tokens + GP_PAGE - 1) / GP_PAGE * GP_PAGE;
  d.beta_s = cfg->beta_s; d.beta_l = cfg->beta_l; d.top_p = cfg->top_p; d.tau = cfg->tau; d.rope_theta = cfg->rope_theta;
  d.policy = cfg->policy; d.policy_seed = (unsigned long long)(unsigned)cfg->policy_seed; d.p_compress = cfg->p_compress;
  d.shrink_below = cfg->shrink_below;
  {
    const long long mp = (cfg->min_capacity + GP_PAGE - 1) / GP_PAGE;      // (P - 1) b >= min_capacity, and P >= 3
    d.min_pages_after_shrink = (int)(mp > (1 << 21) ? (1 << 21) : (mp < 2 * d.sub ? 2 * d.sub : mp));
  }
  d.p_fix = (unsigned long long)llrint(cfg->top_p * 4611686018427387904.0);
  d.kv = reinterpret_cast<__nv_bfloat16*>(base + L.kv);
  d.tok = reinterpret_cast<int*>(base + L.tok);
  d.refcount = reinterpret_cast<int*>(base + L.refcount);
  d.free_stack = reinterpret_cast<int*>(base + L.free_stack);
  int* words = reinterpret_cast<int*>(base + L.words);
  d.free_top = words + 0;
  {
    void* herr = nullptr; void* derr = nullptr;
    if (cudaHostAlloc(&herr, 64, cudaHostAllocMapped) != cudaSuccess ||
        cudaHostGetDevicePointer(&derr, herr, 0) != cudaSuccess) {
      if (herr) cudaFreeHost(herr);
      pool_free(pool);
      return GP_ERR_CUDA;
    }
    memset(herr, 0, 64);
    pool->h_err = static_cast<int*>(herr);
    d.err = static_cast<int*>(derr);
  }
  pool->d_status = words + 2;
  d.hdr = words + 64;
  d.page_table = reinterpret_cast<int*>(base + L.page_table);
  d.shadow = reinterpret_cast<int*>(base + L.shadow);
  int* reqi = reinterpret_cast<int*>(base + L.reqi);
  const int M = cfg->max_requests;
  d.P = reqi; d.n = reqi + M; d.started = reqi + 2 * M; d.sum_par = reqi + 3 * M;
  d.live = reqi + 4 * M; d.n_pristine = reqi + 5 * M; d.bstep = reqi + 6 * M; d.last_act = reqi + 7 * M;
  d.pos = reinterpret_cast<long long*>(base + L.pos);
  d.summ = reinterpret_cast<double*>(base + L.summ);
  d.Kx = reinterpret_cast<int*>(base + L.Kx);
  d.Hx = reinterpret_cast<double*>(base + L.Hx);
  d.metric = cfg->demand_metric;
  d.delta = reinterpret_cast<double*>(base + L.delta);
  d.rcx = reinterpret_cast<int*>(base + L.rc);
  d.mc_list = reinterpret_cast<int4*>(base + L.mc_list);
  d.bnd_info = reinterpret_cast<int4*>(base + L.bnd_info);
  d.bnd_acc = reinterpret_cast<int*>(base + L.bnd_acc);
  d.unit_ready = reinterpret_cast<int*>(base + L.unit_ready);
  d.shard_sums = reinterpret_cast<int*>(base + L.shard_sums);
  d.units_total = cfg->n_layers * cfg->n_kv_heads * cfg->kv_shard_count;
  d.free_peek = reinterpret_cast<int*>(base + L.free_peek);
  d.cmp_info = reinterpret_cast<int4*>(base + L.cmp_info);
  d.zbuf = reinterpret_cast<double*>(base + L.zbuf);
  d.qtil = reinterpret_cast<double*>(base + L.qtil);
  d.zstat = reinterpret_cast<double*>(base + L.zstat);
  d.evict = reinterpret_cast<int*>(base + L.evict);
  d.evict2 = reinterpret_cast<int*>(base + L.evict2);
  d.cflags = reinterpret_cast<int*>(base + L.cflags);
  d.rope_cs = reinterpret_cast<double*>(base + L.rope_cs);
  d.partials = reinterpret_cast<float*>(base + L.partials);
  d.scores = reinterpret_cast<double*>(base + L.scores);
  d.counters = reinterpret_cast<long long*>(base + L.counters);
  gp_attention_setup(d);
  gp_boundary_setup(d, pool->num_sms, &pool->sel_grid, &pool->compact_grid);
  pool->dev_alt = d;
  pool->chain_pending = 0;
  pool->last_stream = nullptr;
  if (cfg->async_boundary) {
    GpDev& a = pool->dev_alt;
    a.hdr = words + 128;
    a.bnd_info = reinterpret_cast<int4*>(base + L.bnd_info2);
    a.bnd_acc = reinterpret_cast<int*>(base + L.bnd_acc2);
    a.zbuf = reinterpret_cast<double*>(base + L.zbuf2);
    a.zstat = reinterpret_cast<double*>(base + L.zstat2);
    a.rcx = reinterpret_cast<int*>(base + L.rc2);
    a.mc_list = reinterpret_cast<int4*>(base + L.mc_list2);
    a.qtil = reinterpret_cast<double*>(base + L.qtil2);
    a.rope_cs = reinterpret_cast<double*>(base + L.rope_cs2);
    // the chain kernel runs beside the attention kernel on the room it leaves: `slots` of its thread blocks
    int slots = cfg->async_slots > 0 ? cfg->async_slots : 64;
    if (slots > pool->attn_grid / 2) slots = pool->attn_grid / 2;
    pool->attn_grid_async = pool->attn_grid - slots;
    pool->chain_grid = slots;
  }
  pool->attn_grid_ov = pool->attn_grid;
  pool->chain_grid_ov = 0;
  // One kernel behind the attention kernel pays while a step's boundary work is a few hundred jobs: it saves a kernel
  // boundary and starts its jobs while the attention kernel drains (64 requests x 8 units: 68 us per step against
  // 75).  With thousands of units the compaction moves hundreds of megabytes and wants the four-kernel path's larger
  // compaction grid (36 layers x 256 residents: 4.8 ms against 5.2; 256 requests x 8 units: 0.49 against 0.52).
  const bool fused_auto = (long long)cfg->max_requests * cfg->n_layers * cfg->n_kv_heads <= 1024;
  if (!cfg->async_boundary && (cfg->overlap_slots == -2 || (cfg->overlap_slots == 0 && fused_auto))) {
    pool->chain_grid_ov = pool->sel_grid;          // the whole grid, behind the attention kernel's
  } else if (!cfg->async_boundary && cfg->overlap_slots > 0) {
    int slots = cfg->overlap_slots;
    if (slots > pool->attn_grid / 2) slots = pool->attn_grid / 2;
    pool->attn_grid_ov = pool->attn_grid - slots;
    pool->chain_grid_ov = slots;
  }
  pool->dev.report_units = pool->dev_alt.report_units = pool->chain_grid_ov > 0;
  pool->dbg = base + L.dbg;
  pool->qn = reinterpret_cast<__nv_bfloat16*>(base + L.qn);
  pool->kn = reinterpret_cast<__nv_bfloat16*>(base + L.kn);
  if (cfg->host_staging) {
    pool->st_ids = reinterpret_cast<int*>(base + L.st_ids);
    pool->st_q = base + L.st_q; pool->st_k = base + L.st_k; pool->st_v = base + L.st_v;
    pool->st2_ids = reinterpret_cast<int*>(base + L.st2_ids);
    pool->st2_q = base + L.st2_q; pool->st2_k = base + L.st2_k; pool->st2_v = base + L.st2_v;
    pool->st_out = reinterpret_cast<float*>(base + L.st_out);
    pool->st_act = reinterpret_cast<int*>(base + L.st_act);
  } else {
    pool->st_ids = nullptr; pool->st_q = pool->st_k = pool->st_v = nullptr; pool->st_out = nullptr; pool->st_act = nullptr;
  }
  // Stale pages are read (masked) by the attention kernel, so they must hold finite numbers.
  if (cudaMemset(dev_blob, 0, L.total) != cudaSuccess) { pool_free(pool); return GP_ERR_CUDA; }
  gp_init_kernel<<<1024, 256>>>(d);
  pool->launch_count++;
  for (int i = 0; i <= GP_N_KERNELS; ++i) {
    if (cudaEventCreate(&pool->ev[i]) != cudaSuccess) { pool_free(pool); return GP_ERR_CUDA; }
  }
  if (cudaDeviceSynchronize() != cudaSuccess) { pool_free(pool); return GP_ERR_CUDA; }
  *out = pool;
  return GP_OK;
}

int gp_pool_destroy(gp_pool* pool) {
  if (!pool) return GP_ERR_INVALID;
  cudaSetDevice(pool->device);
  cudaDeviceSynchronize();
  for (int i = 0; i <= GP_N_KERNELS; ++i) cudaEventDestroy(pool->ev[i]);
  pool_free(pool);
  return GP_OK;
}

int gp_request_add(gp_pool* pool, int32_t share_from, int32_t n_shared_pages, const void* k_tail, const void* v_tail,
                   int32_t n_tail, int32_t initial_pages, void* stream, int32_t* out_req) {
  if (!pool || !out_req || n_tail < 0 || n_shared_pages < 0 || initial_pages < 0) return GP_ERR_INVALID;
  if (n_tail > 0 && (!k_tail || !v_tail)) return GP_ERR_INVALID;
  *out_req = -1;
  if (pool->step_open) return GP_ERR_STATE;      // the open step's plan holds a snapshot of the free list
  if (n_shared_pages > 0 && check_req(pool, share_from) != GP_OK) return GP_ERR_INVALID;
  const gp_config& c = pool->cfg;
  int slot = -1;
  for (int i = 0; i < c.max_requests; ++i)
    if (!pool->live[i]) { slot = i; break; }
  if (slot < 0 && n_shared_pages == 0) return GP_ERR_NO_SLOT;
  const int sub = c.page_size / GP_PAGE;
  const long long n_prompt = (long long)n_shared_pages * c.page_size + n_tail;
  long long P = n_prompt / c.page_size + 1;
  if (initial_pages > P) P = initial_pages;
  // with shared pages the donor's count of shareable pages lives on the device: the kernel below gives the
  // refusals in the documented order (invalid arguments, no slot, no pages)
  if (P > c.max_pages_per_req && n_shared_pages == 0) return GP_ERR_NO_PAGES;
  if (P > c.max_pages_per_req) P = (long long)c.max_pages_per_req + 1;      // still refused, and fits an int
  GP_CUDA(cudaSetDevice(pool->device));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (flush_chain(pool, s) != GP_OK) return GP_ERR_CUDA;       // the free list belongs to the last step's boundary chain first
  // the kernels count in physical pages
  gp_admit_kernel<<<1, 32, 0, s>>>(pool->dev, slot, share_from, n_shared_pages * sub, n_tail, (int)(P * sub), pool->d_status);
  pool->launch_count++;
  int st = GP_ERR_CUDA;
  GP_CUDA(cudaMemcpyAsync(&st, pool->d_status, sizeof(int), cudaMemcpyDeviceToHost, s));
  GP_CUDA(cudaStreamSynchronize(s));
  if (st != GP_OK) return st;
  if (n_tail > 0) {
    const long long total = (long long)c.n_layers * n_tail * c.n_kv_heads * 2 * (c.head_dim / 8);
    int grid = (int)((total + 255) / 256);
    if (grid > 148 * 16) grid = 148 * 16;
    gp_ingest_kernel<<<grid, 256, 0, s>>>(pool->dev, slot, n_shared_pages * sub, n_tail,
                                         static_cast<const __nv_bfloat16*>(k_tail),
                                         static_cast<const __nv_bfloat16*>(v_tail));
    pool->launch_count++;
    GP_CUDA(cudaStreamSynchronize(s));     // the caller may free the prompt buffers on return
  }
  pool->live[slot] = 1;
  *out_req = slot;
  return GP_OK;
}

// CTA 0 plans (when plan_on); the others update the query summaries of the units [lh0, lh0 + lh_n)
static void launch_plan(gp_pool* pool, const int32_t* ids, int32_t n_req, int32_t* actions, const void* q, int plan_on,
                        int lh0, int lh_n, cudaStream_t s, bool pdl, bool by_layer = false, const GpDev* dev = nullptr,
                        int attn_grid = 0, const GpNorm* norm = nullptr) {
  const GpDev& d = dev ? *dev : pool->dev;
  const int upc = 32 / (2 * d.G);                            // units a CTA takes per pass (one warp per row)
  const long long want = ((long long)n_req * lh_n + upc - 1) / upc;
  const long long room = 2LL * pool->num_sms - 1;            // two 1024-thread CTAs per SM, one wave
  const int prep = (int)(want < room ? want : room);
  gp_launch(gp_plan_kernel, 1 + prep, GP_PLAN_THREADS, 0, s, pdl, d, ids, n_req, actions,
            static_cast<const __nv_bfloat16*>(q), plan_on, lh0, lh_n, d.chunk_pages, d.bchunk_pages,
            by_layer ? d.Hkv : d.L * d.Hkv, attn_grid ? attn_grid : pool->attn_grid, (int)(pool->serial & 0x3fffffff),
            norm ? *norm : GpNorm{nullptr, nullptr, 0.0, nullptr, nullptr, nullptr});
}

int gp_decode_step(gp_pool* pool, const int32_t* dev_req_ids, int32_t n_req, const void* q, const void* k,
                   const void* v, void* out, int32_t* dev_actions, void* stream) {
  if (!pool || n_req < 0 || n_req > pool->cfg.max_requests) return GP_ERR_INVALID;
  if (pool->step_open) return GP_ERR_STATE;
  if (n_req == 0) return GP_OK;
  if (!dev_req_ids || !q || !k || !v || !out || !dev_actions) return GP_ERR_INVALID;
  // the kernels move query, key and value rows with 16-byte copies and write `out` in 8-byte pieces
  if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(out, 16) ||
      misaligned(dev_req_ids, 4) || misaligned(dev_actions, 4)) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(pool->device));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool prof = pool->profiling != 0;
  const bool pdl = !prof;                      // events between the kernels need them serialised the plain way
  const int serial = (int)(pool->serial & 0x3fffffff);
  if (!pool->cfg.async_boundary) {
    const GpDev& d = pool->dev;
    const int LH = d.L * d.Hkv;
    if (prof) cudaEventRecord(pool->ev[0], s);
    // first_plain: the kernel before the plan on the stream is not one of this library's (the host entry point's
    // fetch of the inputs): no programmatic dependence on it
    if (pool->chain_grid_ov > 0) {
      // Three kernels.  The boundary work of the step (selection jobs, decisions, compaction, then the merge of the
      // split outputs) is one kernel behind the attention kernel.  Its thread blocks take their places as that
      // kernel's leave (or, with overlap_slots > 0, run beside it on slots its grid leaves free), and a selection job
      // starts as soon as the attention kernel has reported its unit's summary logits complete.
      launch_plan(pool, dev_req_ids, n_req, dev_actions, q, pool->early_plan ? 2 : 1, 0, LH, s, pdl && !pool->first_plain, false,
                  nullptr, pool->attn_grid_ov);
      if (prof) cudaEventRecord(pool->ev[1], s);
      gp_launch_attention(d, dev_req_ids, n_req, q, k, v, static_cast<float*>(out), pool->attn_grid_ov, s, pdl, 0, LH, 0);
      if (prof) cudaEventRecord(pool->ev[2], s);
      gp_launch_chain(d, d, n_req, static_cast<float*>(out), serial, 1, pool->chain_grid_ov, s, pdl, dev_req_ids, dev_actions,
                      pool->actions_copy);
      if (prof) { cudaEventRecord(pool->ev[3], s); cudaEventRecord(pool->ev[4], s); }    // the last interval stays empty
      pool->launch_count += 3;
    } else {
      // Four kernels, one after the other (overlap_slots = -1): the selection and compaction kernels of the
      // layer-by-layer step
      launch_plan(pool, dev_req_ids, n_req, dev_actions, q, pool->early_plan ? 2 : 1, 0, LH, s, pdl && !pool->first_plain);
      if (prof) cudaEventRecord(pool->ev[1], s);
      gp_launch_attention(d, dev_req_ids, n_req, q, k, v, static_cast<float*>(out), pool->attn_grid, s, pdl, 0, LH, 0);
      if (prof) cudaEventRecord(pool->ev[2], s);
      gp_launch_boundary(d, dev_req_ids, n_req, dev_actions, static_cast<float*>(out), pool->sel_grid, pool->compact_grid, s,
                         prof ? pool->ev[3] : nullptr, pdl, serial);
      if (prof) cudaEventRecord(pool->ev[4], s);
      pool->launch_count += GP_N_KERNELS;
    }
  } else {
    // Asynchronous boundary work, all on the caller's stream: plan and attention of this step, then one kernel
    // with the boundary chain of the step before (working sets, decisions, compaction), which runs beside the
    // attention kernel, ends after it and then merges this step's split outputs.  Step t uses scratch set t mod 2.
    const int par = (int)(pool->serial & 1);
    const GpDev& d = par ? pool->dev_alt : pool->dev;
    const GpDev& dprev = par ? pool->dev : pool->dev_alt;
    const int LH = d.L * d.Hkv;
    if (prof) cudaEventRecord(pool->ev[0], s);
    // no early planning here: the plan reads the pages and slots of the requests that return from their step out,
    // which the chain kernel of the step before (the kernel before this one on the stream) has just written
    launch_plan(pool, dev_req_ids, n_req, dev_actions, q, 1, 0, LH, s, pdl && !pool->first_plain, false, &d, pool->attn_grid_async);
    if (prof) cudaEventRecord(pool->ev[1], s);
    gp_launch_attention(d, dev_req_ids, n_req, q, k, v, static_cast<float*>(out), pool->attn_grid_async, s, pdl, 0, LH, 0);
    if (prof) cudaEventRecord(pool->ev[2], s);
    // the decisions of the step before set pages and slots of requests that sit this step out: nothing else of
    // this step looks at those words
    gp_launch_chain(dprev, d, n_req, static_cast<float*>(out), (int)((pool->serial - 1) & 0x3fffffff),
                    pool->chain_pending, pool->chain_grid, s, pdl);
    if (prof) { cudaEventRecord(pool->ev[3], s); cudaEventRecord(pool->ev[4], s); }
    pool->chain_pending = 1;
    pool->last_stream = s;
    pool->launch_count += 3;
  }
  pool->serial += 1;
  GP_CUDA(cudaGetLastError());
  if (prof) {
    GP_CUDA(cudaEventSynchronize(pool->ev[GP_N_KERNELS]));
    for (int i = 0; i < GP_N_KERNELS; ++i) {
      float t = 0.f;
      GP_CUDA(cudaEventElapsedTime(&t, pool->ev[i], pool->ev[i + 1]));
      pool->ms[i] += t;
      pool->launches[i] += 1;
    }
  }
  return GP_OK;
}

int gp_async_join(gp_pool* pool, void* stream) {
  if (!pool) return GP_ERR_INVALID;
  if (!pool->cfg.async_boundary) return GP_OK;
  GP_CUDA(cudaSetDevice(pool->device));
  return flush_chain(pool, static_cast<cudaStream_t>(stream));
}

int gp_boundary_outcome(gp_pool* pool, int32_t req, int32_t* action, int64_t* step) {
  const int st = check_req(pool, req);
  if (st != GP_OK) return st;
  GP_CUDA(cudaSetDevice(pool->device));
  if (flush_chain(pool, pool->last_stream) != GP_OK) return GP_ERR_CUDA;
  GP_CUDA(cudaDeviceSynchronize());
  int a = 0, b = 0;
  GP_CUDA(cudaMemcpy(&a, pool->dev.last_act + req, 4, cudaMemcpyDeviceToHost));
  GP_CUDA(cudaMemcpy(&b, pool->dev.bstep + req, 4, cudaMemcpyDeviceToHost));
  if (b == GP_NEVER) a = GP_ACT_NONE;
  if (action) *action = a;
  if (step) *step = b == GP_NEVER ? -1 : (int64_t)((pool->serial & ~0x3fffffffLL) | (long long)b);
  return GP_OK;
}

// ---- the same step, layer by layer: a model's forward pass has layer l + 1's query only after layer l's
// attention output ---------------------------------------------------------------------------------------
int gp_step_begin(gp_pool* pool, const int32_t* dev_req_ids, int32_t n_req, int32_t* dev_actions, void* stream) {
  if (!pool || n_req < 0 || n_req > pool->cfg.max_requests) return GP_ERR_INVALID;
  if (pool->step_open || pool->cfg.async_boundary) return GP_ERR_STATE;
  if (n_req == 0) return GP_OK;
  if (!dev_req_ids || !dev_actions || misaligned(dev_req_ids, 4) || misaligned(dev_actions, 4)) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(pool->device));
  launch_plan(pool, dev_req_ids, n_req, dev_actions, nullptr, 1, 0, 0, static_cast<cudaStream_t>(stream), true, true);
  pool->launch_count += 1;
  pool->step_open = 1;
  pool->step_n_req = n_req;
  pool->step_layers_done = 0;
  pool->step_layer_seen.assign(pool->cfg.n_layers, 0);
  GP_CUDA(cudaGetLastError());
  return GP_OK;
}

int gp_attn_layer(gp_pool* pool, int32_t layer, const int32_t* dev_req_ids, int32_t n_req, const void* q, const void* k,
                  const void* v, void* out, void* stream) {
  if (!pool || pool->step_open != 1 || n_req != pool->step_n_req) return pool && pool->step_open != 1 ? GP_ERR_STATE : GP_ERR_INVALID;
  if (layer < 0 || layer >= pool->cfg.n_layers || !dev_req_ids || !q || !k || !v || !out) return GP_ERR_INVALID;
  if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(out, 16) || misaligned(dev_req_ids, 4))
    return GP_ERR_INVALID;
  if (pool->step_layer_seen[layer]) return GP_ERR_STATE;          // every layer once
  GP_CUDA(cudaSetDevice(pool->device));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const GpDev& d = pool->dev;
  // The kernels index their per-step tensors as [layer][request][head][d]: a layer's own tensors are handed over
  // as the base such an array would have (the kernels only touch this layer's part of it).
  const size_t qs = (size_t)layer * n_req * d.Hq * d.d, ks = (size_t)layer * n_req * d.Hkv * d.d;
  const __nv_bfloat16* qb = reinterpret_cast<const __nv_bfloat16*>(reinterpret_cast<uintptr_t>(q) - qs * 2);
  const __nv_bfloat16* kb = reinterpret_cast<const __nv_bfloat16*>(reinterpret_cast<uintptr_t>(k) - ks * 2);
  const __nv_bfloat16* vb = reinterpret_cast<const __nv_bfloat16*>(reinterpret_cast<uintptr_t>(v) - ks * 2);
  float* ob = reinterpret_cast<float*>(reinterpret_cast<uintptr_t>(out) - qs * 4);
  const int lh0 = layer * d.Hkv, lh_n = d.Hkv;
  launch_plan(pool, dev_req_ids, n_req, nullptr, qb, 0, lh0, lh_n, s, true);
  gp_launch_attention(d, dev_req_ids, n_req, qb, kb, vb, ob, pool->attn_grid, s, true, lh0, lh_n, -1);
  gp_launch_merge(d, n_req, ob, lh0, lh_n, pool->num_sms, s, true);
  pool->launch_count += 3;
  pool->step_layers_done += 1;
  pool->step_layer_seen[layer] = 1;
  GP_CUDA(cudaGetLastError());
  return GP_OK;
}

int gp_attn_layer_qknorm(gp_pool* pool, int32_t layer, const int32_t* dev_req_ids, int32_t n_req, const void* q_raw,
                         const void* k_raw, const void* v, const float* q_weight, const float* k_weight, double eps, void* out,
                         void* stream) {
  if (!pool || pool->step_open != 1 || n_req != pool->step_n_req) return pool && pool->step_open != 1 ? GP_ERR_STATE : GP_ERR_INVALID;
  if (layer < 0 || layer >= pool->cfg.n_layers || !dev_req_ids || !q_raw || !k_raw || !v || !out || !q_weight || !k_weight)
    return GP_ERR_INVALID;
  if (misaligned(q_raw, 16) || misaligned(k_raw, 16) || misaligned(v, 16) || misaligned(out, 16) || misaligned(dev_req_ids, 4) ||
      misaligned(q_weight, 4) || misaligned(k_weight, 4) || !(eps >= 0.0))
    return GP_ERR_INVALID;
  if (pool->step_layer_seen[layer]) return GP_ERR_STATE;          // every layer once
  GP_CUDA(cudaSetDevice(pool->device));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const GpDev& d = pool->dev;
  const size_t qs = (size_t)layer * n_req * d.Hq * d.d, ks = (size_t)layer * n_req * d.Hkv * d.d;
  auto shifted = [](const void* ptr, size_t bytes) { return reinterpret_cast<uintptr_t>(ptr) - bytes; };
  const __nv_bfloat16* qb = reinterpret_cast<const __nv_bfloat16*>(shifted(q_raw, qs * 2));
  const __nv_bfloat16* vb = reinterpret_cast<const __nv_bfloat16*>(shifted(v, ks * 2));
  float* ob = reinterpret_cast<float*>(shifted(out, qs * 4));
  GpNorm nm;
  nm.wq = q_weight; nm.wk = k_weight; nm.eps = eps;
  nm.k_raw = reinterpret_cast<const __nv_bfloat16*>(shifted(k_raw, ks * 2));
  nm.qn = reinterpret_cast<__nv_bfloat16*>(shifted(pool->qn, qs * 2));
  nm.kn = reinterpret_cast<__nv_bfloat16*>(shifted(pool->kn, ks * 2));
  const int lh0 = layer * d.Hkv, lh_n = d.Hkv;
  launch_plan(pool, dev_req_ids, n_req, nullptr, qb, 0, lh0, lh_n, s, true, false, nullptr, 0, &nm);
  gp_launch_attention(d, dev_req_ids, n_req, nm.qn, nm.kn, vb, ob, pool->attn_grid, s, true, lh0, lh_n, -1);
  gp_launch_merge(d, n_req, ob, lh0, lh_n, pool->num_sms, s, true);
  pool->launch_count += 3;
  pool->step_layers_done += 1;
  pool->step_layer_seen[layer] = 1;
  GP_CUDA(cudaGetLastError());
  return GP_OK;
}

int gp_step_end(gp_pool* pool, const int32_t* dev_req_ids, int32_t n_req, int32_t* dev_actions, void* stream) {
  if (!pool || pool->step_open != 1) return pool ? GP_ERR_STATE : GP_ERR_INVALID;
  if (n_req != pool->step_n_req || !dev_req_ids || !dev_actions) return GP_ERR_INVALID;
  if (pool->step_layers_done != pool->cfg.n_layers) return GP_ERR_STATE;       // layers missing: run them, or gp_step_abort
  GP_CUDA(cudaSetDevice(pool->device));
  gp_launch_boundary(pool->dev, dev_req_ids, n_req, dev_actions, nullptr,
                     pool->sel_grid, pool->compact_grid,
                     static_cast<cudaStream_t>(stream), nullptr, true, (int)(pool->serial & 0x3fffffff));
  pool->serial += 1;
  pool->launch_count += 2;
  pool->step_open = 0;
  GP_CUDA(cudaGetLastError());
  return GP_OK;
}

int gp_step_abort(gp_pool* pool) {
  if (!pool) return GP_ERR_INVALID;
  if (pool->step_open != 1) return GP_ERR_STATE;        // (a step begun with gp_decode_step_local has to be finished)
  // Nothing of an open step is committed before gp_step_end: the requests' counters are untouched, rows appended
  // by the layers that ran lie beyond the occupied slots, and the summaries went to the buffer not in use.
  pool->step_open = 0;
  return GP_OK;
}

// ---- the step of a pool that holds a part of the model's KV heads --------------------------------------------
int gp_decode_step_local(gp_pool* pool, const int32_t* dev_req_ids, int32_t n_req, const void* q, const void* k,
                         const void* v, void* out, int32_t* dev_actions, void* stream) {
  if (!pool || n_req < 0 || n_req > pool->cfg.max_requests) return GP_ERR_INVALID;
  if (pool->step_open || pool->cfg.async_boundary) return GP_ERR_STATE;
  if (n_req == 0) return GP_OK;
  if (!dev_req_ids || !q || !k || !v || !out || !dev_actions) return GP_ERR_INVALID;
  if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(out, 16) ||
      misaligned(dev_req_ids, 4) || misaligned(dev_actions, 4)) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(pool->device));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const GpDev& d = pool->dev;
  const int LH = d.L * d.Hkv;
  const int serial = (int)(pool->serial & 0x3fffffff);
  launch_plan(pool, dev_req_ids, n_req, dev_actions, q, 1, 0, LH, s, true);
  gp_launch_attention(d, dev_req_ids, n_req, q, k, v, static_cast<float*>(out), pool->attn_grid, s, true, 0, LH, 0);
  gp_launch_select_only(d, dev_req_ids, n_req, dev_actions, static_cast<float*>(out), pool->sel_grid, s, true, serial);
  pool->launch_count += 3;
  pool->step_open = 2;                           // between the two halves the pool takes nothing else
  pool->step_n_req = n_req;
  GP_CUDA(cudaGetLastError());
  return GP_OK;
}

int gp_shard_sums(gp_pool* pool, int32_t** dev_sums, int64_t* n_ints) {
  if (!pool || !dev_sums || !n_ints) return GP_ERR_INVALID;
  *dev_sums = pool->dev.shard_sums;
  *n_ints = 2LL * pool->cfg.max_requests;
  return GP_OK;
}

int gp_decode_step_finish(gp_pool* pool, const int32_t* dev_req_ids, int32_t n_req, int32_t* dev_actions, void* stream) {
  if (!pool) return GP_ERR_INVALID;
  if (pool->step_open != 2) return GP_ERR_STATE;
  if (n_req != pool->step_n_req || !dev_req_ids || !dev_actions) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(pool->device));
  gp_launch_decide_compact(pool->dev, dev_req_ids, n_req, dev_actions, pool->compact_grid, static_cast<cudaStream_t>(stream),
                           (int)(pool->serial & 0x3fffffff));
  pool->serial += 1;
  pool->launch_count += 2;
  pool->step_open = 0;
  GP_CUDA(cudaGetLastError());
  return GP_OK;
}

// The step's inputs, read from page-locked mapped host memory over the bus by one kernel: the request ids word
// by word, queries, keys and values in 16-byte pieces, every piece its own load, all in flight together (four
// separate copies cost their set-up four times).
__global__ void gp_fetch_inputs_kernel(int* __restrict__ d_ids, const int* __restrict__ s_ids, int n_ids,
                                       uint4* __restrict__ d1, const uint4* __restrict__ s1, long long n1,
                                       uint4* __restrict__ d2, const uint4* __restrict__ s2, long long n2,
                                       uint4* __restrict__ d3, const uint4* __restrict__ s3, long long n3) {
  const long long total = n1 + n2 + n3;
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (tid < n_ids) d_ids[tid] = s_ids[tid];
  for (long long i = tid; i < total; i += (long long)gridDim.x * blockDim.x) {
    if (i < n1) d1[i] = s1[i];
    else if (i < n1 + n2) d2[i - n1] = s2[i - n1];
    else d3[i - n1 - n2] = s3[i - n1 - n2];
  }
}

extern "C" int gp_decode_step_host_wait(gp_pool* pool);
static int host_step(gp_pool* pool, const int32_t* host_req_ids, int32_t n_req, const void* q, const void* k,
                     const void* v, void* out, int32_t* actions, void* stream, bool wait) {
  if (!pool || n_req < 0 || n_req > pool->cfg.max_requests) return GP_ERR_INVALID;
  if (!pool->st_ids || pool->step_open) return GP_ERR_STATE;
  if (n_req == 0) return GP_OK;
  if (!host_req_ids || !q || !k || !v || !out || !actions) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(pool->device));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const gp_config& c = pool->cfg;
  const size_t qb = (size_t)c.n_layers * n_req * c.n_q_heads * c.head_dim * 2;
  const size_t kb = (size_t)c.n_layers * n_req * c.n_kv_heads * c.head_dim * 2;
  // Inputs: from mapped page-locked buffers one kernel fetches all four over the bus into one of two staging sets.
  // When the caller issues steps ahead (gp_decode_step_host_async) the fetch runs on a stream of its own, beside
  // the kernels of the step before it: it waits until the step that last used the set has read it, and the step
  // waits for its fetch.  The call that waits for its step fetches on the caller's stream (nothing to overlap
  // with).  Pageable memory: four copies on the caller's stream.
  const int set = (int)(pool->host_steps & 1);
  bool staged_async = false;                 // inputs by the copy engine on the side stream (the call that does not wait)
  int* st_ids = set ? pool->st2_ids : pool->st_ids;
  void* st_q = set ? pool->st2_q : pool->st_q;
  void* st_k = set ? pool->st2_k : pool->st_k;
  void* st_v = set ? pool->st2_v : pool->st_v;
  {
    void *mi = nullptr, *mq = nullptr, *mk = nullptr, *mv = nullptr;
    const bool mapped = ((uintptr_t)host_req_ids % 4 == 0) && ((uintptr_t)q % 16 == 0) && ((uintptr_t)k % 16 == 0) &&
                        ((uintptr_t)v % 16 == 0) &&
                        cudaHostGetDevicePointer(&mi, const_cast<int32_t*>(host_req_ids), 0) == cudaSuccess &&
                        cudaHostGetDevicePointer(&mq, const_cast<void*>(q), 0) == cudaSuccess &&
                        cudaHostGetDevicePointer(&mk, const_cast<void*>(k), 0) == cudaSuccess &&
                        cudaHostGetDevicePointer(&mv, const_cast<void*>(v), 0) == cudaSuccess;
    if (mapped && wait) {
      const long long pieces = (long long)(qb + 2 * kb) / 16;         // a row is 128 or 256 bytes: whole pieces
      int grid = (int)((pieces + 255) / 256);
      if (grid > pool->num_sms * 8) grid = pool->num_sms * 8;
      if (grid * 256 < n_req) grid = (n_req + 255) / 256;
      gp_fetch_inputs_kernel<<<grid, 256, 0, s>>>(st_ids, static_cast<const int*>(mi), n_req,
                                                 static_cast<uint4*>(st_q), static_cast<const uint4*>(mq), (long long)qb / 16,
                                                 static_cast<uint4*>(st_k), static_cast<const uint4*>(mk), (long long)kb / 16,
                                                 static_cast<uint4*>(st_v), static_cast<const uint4*>(mv), (long long)kb / 16);
      pool->launch_count++;
    } else if (mapped) {
      if (!pool->fetch_stream) {
        GP_CUDA(cudaStreamCreateWithFlags(&pool->fetch_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
          GP_CUDA(cudaEventCreateWithFlags(&pool->ev_fetch[i], cudaEventDisableTiming));
          GP_CUDA(cudaEventCreateWithFlags(&pool->ev_used[i], cudaEventDisableTiming));
          GP_CUDA(cudaEventCreateWithFlags(&pool->ev_out[i], cudaEventDisableTiming));
          GP_CUDA(cudaEventRecord(pool->ev_used[i], s));
          GP_CUDA(cudaEventRecord(pool->ev_out[i], s));
        }
      }
      cudaStream_t fs = pool->fetch_stream;
      GP_CUDA(cudaStreamWaitEvent(fs, pool->ev_used[set], 0));
      // Copies by the copy engine here, not the fetch kernel: they run beside the step before, whose attention
      // kernel fills every SM's registers; a kernel that reads over the bus for 15 us held some of them and kept
      // that step's attention thread blocks from starting (11 us per step).  The copies' set-up time, which is
      // what the fetch kernel saves the call that waits, is hidden here.
      GP_CUDA(cudaMemcpyAsync(st_ids, host_req_ids, (size_t)n_req * 4, cudaMemcpyHostToDevice, fs));
      GP_CUDA(cudaMemcpyAsync(st_q, q, qb, cudaMemcpyHostToDevice, fs));
      GP_CUDA(cudaMemcpyAsync(st_k, k, kb, cudaMemcpyHostToDevice, fs));
      GP_CUDA(cudaMemcpyAsync(st_v, v, kb, cudaMemcpyHostToDevice, fs));
      GP_CUDA(cudaEventRecord(pool->ev_fetch[set], fs));
      GP_CUDA(cudaStreamWaitEvent(s, pool->ev_fetch[set], 0));
      staged_async = true;
    } else {
      (void)cudaGetLastError();                    // pageable memory: not an error
      GP_CUDA(cudaMemcpyAsync(st_ids, host_req_ids, (size_t)n_req * 4, cudaMemcpyHostToDevice, s));
      GP_CUDA(cudaMemcpyAsync(st_q, q, qb, cudaMemcpyHostToDevice, s));
      GP_CUDA(cudaMemcpyAsync(st_k, k, kb, cudaMemcpyHostToDevice, s));
      GP_CUDA(cudaMemcpyAsync(st_v, v, kb, cudaMemcpyHostToDevice, s));
    }
  }
  pool->host_steps += 1;
  // Outputs: when the caller's buffers are page-locked and mapped (the usual pinned allocation), the kernels
  // write them over the bus while they run and nothing is left to copy when the step ends.  (The same was tried
  // for the inputs and was slower: rows read over the bus by the kernels stall the pipelines that wait for them.)
  void* d_out = nullptr;
  void* d_act = nullptr;
  const bool direct = cudaHostGetDevicePointer(&d_out, out, 0) == cudaSuccess &&
                      cudaHostGetDevicePointer(&d_act, actions, 0) == cudaSuccess;
  if (!direct) (void)cudaGetLastError();           // pageable memory: not an error, the staged path takes over
  // (Results through a staging set and the copy engine on a third stream, beside the next step, were tried for the
  // call that does not wait: a megabyte takes the copy engine and the event that reports it 60 us, longer than the
  // host may lag behind when it reads every step's results before it issues the step after the next: 92 us per
  // step against 78 with the kernels writing the rows over the bus themselves.)
  float* st_out = pool->st_out;
  int* st_act = pool->st_act;
  if (staged_async && pool->host_async_issued - pool->host_waited >= 2) {          // two calls outstanding: the older first
    const int st0 = gp_decode_step_host_wait(pool);
    if (st0 != GP_OK) return st0;
  }
  // The inputs arrive by the fetch kernel or the copies above, which end before the plan kernel starts: that
  // kernel is launched the plain way here (not as a programmatic dependent of the fetch kernel, whose stores it
  // reads), so planning ahead of its wait, which is then no wait at all, is safe whatever the option says.
  const int early = pool->early_plan;
  pool->early_plan = 1;
  pool->first_plain = 1;
  // The actions: the plan kernel writes them all and the decisions overwrite some; written straight to host memory
  // they made the plan kernel wait for the bus.  With the boundary work in one kernel they stay on the device and
  // that kernel copies them to the caller's array once they are final (beside its compaction).
  const bool act_late = direct && !pool->cfg.async_boundary && pool->chain_grid_ov > 0;
  pool->actions_copy = act_late ? static_cast<int32_t*>(d_act) : nullptr;
  const int st = gp_decode_step(pool, st_ids, n_req, st_q, st_k, st_v,
                                direct ? d_out : static_cast<void*>(st_out),
                                direct && !act_late ? static_cast<int32_t*>(d_act) : st_act, stream);
  pool->actions_copy = nullptr;
  pool->early_plan = early;
  pool->first_plain = 0;
  if (st != GP_OK) return st;
  if (pool->fetch_stream) GP_CUDA(cudaEventRecord(pool->ev_used[set], s));       // the set may be fetched into again
  if (!direct) {
    GP_CUDA(cudaMemcpyAsync(out, st_out, qb * 2, cudaMemcpyDeviceToHost, s));
    GP_CUDA(cudaMemcpyAsync(actions, st_act, (size_t)n_req * 4, cudaMemcpyDeviceToHost, s));
  }
  if (staged_async) {                          // what gp_decode_step_host_wait waits for: this call's work on `stream`
    GP_CUDA(cudaEventRecord(pool->ev_out[set], s));
    pool->host_async_set[pool->host_async_issued & 1] = set;
    pool->host_async_issued += 1;
  }
  if (!wait) return GP_OK;
  GP_CUDA(cudaStreamSynchronize(s));
  return kernel_status(pool);
}

int gp_decode_step_host(gp_pool* pool, const int32_t* host_req_ids, int32_t n_req, const void* q, const void* k,
                        const void* v, void* out, int32_t* actions, void* stream) {
  return host_step(pool, host_req_ids, n_req, q, k, v, out, actions, stream, true);
}

int gp_decode_step_host_async(gp_pool* pool, const int32_t* host_req_ids, int32_t n_req, const void* q, const void* k,
                              const void* v, void* out, int32_t* actions, void* stream) {
  return host_step(pool, host_req_ids, n_req, q, k, v, out, actions, stream, false);
}

int gp_decode_step_host_wait(gp_pool* pool) {
  if (!pool) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(pool->device));
  if (pool->host_waited < pool->host_async_issued) {
    GP_CUDA(cudaEventSynchronize(pool->ev_out[pool->host_async_set[pool->host_waited & 1]]));
    pool->host_waited += 1;
  } else {
    GP_CUDA(cudaDeviceSynchronize());        // nothing of that kind outstanding: whatever else the pool has in flight
  }
  return kernel_status(pool);
}

int gp_pool_status(gp_pool* pool, int32_t* error_bits) {
  if (!pool) return GP_ERR_INVALID;
  const int e = *reinterpret_cast<volatile const int*>(pool->h_err);
  if (error_bits) *error_bits = e;
  return e ? GP_ERR_CUDA : GP_OK;
}

int gp_release(gp_pool* pool, int32_t req, void* stream) {
  const int st = check_req(pool, req);
  if (st != GP_OK) return st;
  if (pool->step_open) return GP_ERR_STATE;      // the open step's plan holds a snapshot of the free list
  GP_CUDA(cudaSetDevice(pool->device));
  if (flush_chain(pool, static_cast<cudaStream_t>(stream)) != GP_OK) return GP_ERR_CUDA;
  gp_release_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(pool->dev, req);
  pool->launch_count++;
  pool->live[req] = 0;
  GP_CUDA(cudaGetLastError());
  return GP_OK;
}

const char* gp_strerror(int status) {
  switch (status) {
    case GP_OK: return "ok";
    case GP_ERR_INVALID: return "invalid argument or request id";
    case GP_ERR_NO_SLOT: return "no free request slot";
    case GP_ERR_NO_PAGES: return "not enough free pages or per-request cap exceeded";
    case GP_ERR_CUDA: return "CUDA error or internal kernel error";
    case GP_ERR_STATE: return "call not possible in this state";
    case GP_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of the no-allocation entry point";
    default: return "unknown status";
  }
}

// ---- introspection ---------------------------------------------------------------------------------
int gp_debug_request(gp_pool* pool, int32_t req, int32_t* P, int32_t* n, int64_t* pos, int32_t* page_table) {
  const int st = check_req(pool, req);
  if (st != GP_OK) return st;
  GP_CUDA(cudaSetDevice(pool->device));
  if (flush_chain(pool, pool->last_stream) != GP_OK) return GP_ERR_CUDA;
  GP_CUDA(cudaDeviceSynchronize());
  int Pv = 0, nv = 0; long long pv = 0;
  GP_CUDA(cudaMemcpy(&Pv, pool->dev.P + req, 4, cudaMemcpyDeviceToHost));
  GP_CUDA(cudaMemcpy(&nv, pool->dev.n + req, 4, cudaMemcpyDeviceToHost));
  GP_CUDA(cudaMemcpy(&pv, pool->dev.pos + req, 8, cudaMemcpyDeviceToHost));
  if (P) *P = Pv / (pool->cfg.page_size / GP_PAGE);
  if (n) *n = nv;
  if (pos) *pos = pv;
  if (page_table && Pv > 0)
  {
    // pages of the method: the group of tiles that starts at table entry j * sub (see gp_debug_pool)
    const int sub = pool->cfg.page_size / GP_PAGE;
    std::vector<int> tiles((size_t)Pv);
    GP_CUDA(cudaMemcpy(tiles.data(), pool->dev.page_table + (size_t)req * pool->dev.cap, (size_t)Pv * 4, cudaMemcpyDeviceToHost));
    for (int j = 0; j < Pv / sub; ++j) page_table[j] = tiles[(size_t)j * sub] / sub;
  }
  return GP_OK;
}

int gp_debug_state(gp_pool* pool, int32_t* P, int32_t* n) {
  if (!pool) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(pool->device));
  if (flush_chain(pool, pool->last_stream) != GP_OK) return GP_ERR_CUDA;
  GP_CUDA(cudaDeviceSynchronize());
  const int M = pool->cfg.max_requests;
  const size_t nb = (size_t)M * 4;
  if (P) GP_CUDA(cudaMemcpy(P, pool->dev.P, nb, cudaMemcpyDeviceToHost));
  if (n) GP_CUDA(cudaMemcpy(n, pool->dev.n, nb, cudaMemcpyDeviceToHost));
  if (P) for (int i = 0; i < M; ++i) P[i] /= pool->cfg.page_size / GP_PAGE;
  return GP_OK;
}

static int gather_stream(gp_pool* pool, int32_t req, int32_t layer, int32_t kv_head, int* n_out) {
  const int st = check_req(pool, req);
  if (st != GP_OK) return st;
  if (layer < 0 || layer >= pool->cfg.n_layers || kv_head < 0 || kv_head >= pool->cfg.n_kv_heads) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(pool->device));
  if (flush_chain(pool, pool->last_stream) != GP_OK) return GP_ERR_CUDA;
  GP_CUDA(cudaDeviceSynchronize());
  int nv = 0;
  GP_CUDA(cudaMemcpy(&nv, pool->dev.n + req, 4, cudaMemcpyDeviceToHost));
  *n_out = nv;
  if (nv == 0) return GP_OK;
  const size_t cap_tok = (size_t)pool->cfg.max_pages_per_req * pool->cfg.page_size;
  int* tok = reinterpret_cast<int*>(pool->dbg);
  uint4* kk = reinterpret_cast<uint4*>(pool->dbg + cap_tok * 4);
  uint4* vv = reinterpret_cast<uint4*>(pool->dbg + cap_tok * 4 + cap_tok * pool->cfg.head_dim * 2);
  gp_gather_kernel<<<148, 256>>>(pool->dev, req, layer, kv_head, nv, tok, kk, vv);
  pool->launch_count++;
  if (flush_chain(pool, pool->last_stream) != GP_OK) return GP_ERR_CUDA;
  GP_CUDA(cudaDeviceSynchronize());
  return GP_OK;
}

int gp_debug_retained(gp_pool* pool, int32_t req, int32_t layer, int32_t kv_head, int32_t* token_ids) {
  if (!token_ids) return GP_ERR_INVALID;
  int n = 0;
  const int st = gather_stream(pool, req, layer, kv_head, &n);
  if (st != GP_OK) return st;
  if (n > 0) GP_CUDA(cudaMemcpy(token_ids, pool->dbg, (size_t)n * 4, cudaMemcpyDeviceToHost));
  return GP_OK;
}

int gp_debug_kv(gp_pool* pool, int32_t req, int32_t layer, int32_t kv_head, void* k_rows, void* v_rows) {
  int n = 0;
  const int st = gather_stream(pool, req, layer, kv_head, &n);
  if (st != GP_OK) return st;
  const size_t cap_tok = (size_t)pool->cfg.max_pages_per_req * pool->cfg.page_size;
  const size_t rowb = (size_t)pool->cfg.head_dim * 2;
  if (n > 0 && k_rows) GP_CUDA(cudaMemcpy(k_rows, pool->dbg + cap_tok * 4, n * rowb, cudaMemcpyDeviceToHost));
  if (n > 0 && v_rows)
    GP_CUDA(cudaMemcpy(v_rows, pool->dbg + cap_tok * 4 + cap_tok * rowb, n * rowb, cudaMemcpyDeviceToHost));
  return GP_OK;
}

int gp_debug_summaries(gp_pool* pool, int32_t req, double* out) {
  const int st = check_req(pool, req);
  if (st != GP_OK) return st;
  if (!out) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(pool->device));
  if (flush_chain(pool, pool->last_stream) != GP_OK) return GP_ERR_CUDA;
  GP_CUDA(cudaDeviceSynchronize());
  const gp_config& c = pool->cfg;
  int par = 0;
  GP_CUDA(cudaMemcpy(&par, pool->dev.sum_par + req, 4, cudaMemcpyDeviceToHost));
  const size_t per = (size_t)2 * c.n_q_heads * c.head_dim;
  for (int l = 0; l < c.n_layers; ++l)
    GP_CUDA(cudaMemcpy(out + (size_t)l * per, pool->dev.summ + (((size_t)l * c.max_requests + req) * 2 + par) * per,
                       per * 8, cudaMemcpyDeviceToHost));
  return GP_OK;
}

int gp_debug_boundary(gp_pool* pool, int32_t req, int32_t* K_S, int32_t* K_L, double* delta) {
  const int st = check_req(pool, req);
  if (st != GP_OK) return st;
  GP_CUDA(cudaSetDevice(pool->device));
  if (flush_chain(pool, pool->last_stream) != GP_OK) return GP_ERR_CUDA;
  GP_CUDA(cudaDeviceSynchronize());
  const int LH = pool->cfg.n_layers * pool->cfg.n_kv_heads;
  std::vector<int> kx((size_t)LH * 2);
  GP_CUDA(cudaMemcpy(kx.data(), pool->dev.Kx + (size_t)req * LH * 2, (size_t)LH * 8, cudaMemcpyDeviceToHost));
  for (int i = 0; i < LH; ++i) {
    if (K_S) K_S[i] = kx[2 * i];
    if (K_L) K_L[i] = kx[2 * i + 1];
  }
  if (delta) GP_CUDA(cudaMemcpy(delta, pool->dev.delta + req, 8, cudaMemcpyDeviceToHost));
  return GP_OK;
}

int gp_debug_entropy(gp_pool* pool, int32_t req, double* H_S, double* H_L) {
  const int st = check_req(pool, req);
  if (st != GP_OK) return st;
  if (pool->cfg.demand_metric != GP_METRIC_ENTROPY) return GP_ERR_STATE;
  GP_CUDA(cudaSetDevice(pool->device));
  if (flush_chain(pool, pool->last_stream) != GP_OK) return GP_ERR_CUDA;
  GP_CUDA(cudaDeviceSynchronize());
  const int LH = pool->cfg.n_layers * pool->cfg.n_kv_heads;
  std::vector<double> hx((size_t)LH * 2);
  GP_CUDA(cudaMemcpy(hx.data(), pool->dev.Hx + (size_t)req * LH * 2, (size_t)LH * 16, cudaMemcpyDeviceToHost));
  for (int i = 0; i < LH; ++i) {
    if (H_S) H_S[i] = hx[2 * i];
    if (H_L) H_L[i] = hx[2 * i + 1];
  }
  return GP_OK;
}

int gp_debug_pool(gp_pool* pool, int64_t* n_free, int32_t* refcounts, int64_t counters[12]) {
  if (!pool) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(pool->device));
  if (flush_chain(pool, pool->last_stream) != GP_OK) return GP_ERR_CUDA;
  GP_CUDA(cudaDeviceSynchronize());
  int top = 0;
  GP_CUDA(cudaMemcpy(&top, pool->dev.free_top, 4, cudaMemcpyDeviceToHost));
  const int err = *reinterpret_cast<volatile const int*>(pool->h_err);
  if (n_free) *n_free = top / (pool->cfg.page_size / GP_PAGE);
  if (refcounts) {
    // One count per page of the method.  Its 16-token tiles are taken from the free list, shared and returned
    // together and in whole aligned groups (the list starts in tile order and every pop and push is a multiple of
    // the group), so page i is tiles [i * sub, (i + 1) * sub) and its count is that of its first tile.
    const int sub = pool->cfg.page_size / GP_PAGE;
    std::vector<int> ref((size_t)pool->dev.n_pages);
    GP_CUDA(cudaMemcpy(ref.data(), pool->dev.refcount, ref.size() * 4, cudaMemcpyDeviceToHost));
    for (long long i = 0; i < pool->cfg.n_pages; ++i) refcounts[i] = ref[(size_t)i * sub];
  }
  if (counters) {
    long long c[12];
    GP_CUDA(cudaMemcpy(c, pool->dev.counters, 96, cudaMemcpyDeviceToHost));
    for (int i = 0; i < 12; ++i) counters[i] = c[i];
    counters[4] /= pool->cfg.page_size / GP_PAGE;          // copy-on-write: counted per 16-token tile, reported per page
    counters[7] = err;
  }
  return GP_OK;
}

int gp_test_withhold(gp_pool* pool, int32_t what, int32_t spin_limit) {
  if (!pool || what < 0 || what > 31 || spin_limit < 0) return GP_ERR_INVALID;
  GpDev* views[2] = {&pool->dev, &pool->dev_alt};
  for (GpDev* v : views) {
    v->withhold = what;
    v->spin_limit = spin_limit > 0 ? (unsigned)spin_limit : GP_SPIN_LIMIT;
  }
  return GP_OK;
}

int gp_set_early_plan(gp_pool* pool, int32_t enable) {
  if (!pool) return GP_ERR_INVALID;
  pool->early_plan = enable ? 1 : 0;
  return GP_OK;
}

int gp_set_profiling(gp_pool* pool, int32_t enable) {
  if (!pool) return GP_ERR_INVALID;
  pool->profiling = enable ? 1 : 0;
  memset(pool->ms, 0, sizeof(pool->ms));
  memset(pool->launches, 0, sizeof(pool->launches));
  return GP_OK;
}

int gp_get_kernel_times(gp_pool* pool, float* ms, int64_t* launches) {
  if (!pool) return GP_ERR_INVALID;
  GP_CUDA(cudaSetDevice(pool->device));
  if (flush_chain(pool, pool->last_stream) != GP_OK) return GP_ERR_CUDA;
  GP_CUDA(cudaDeviceSynchronize());
  for (int i = 0; i < GP_N_KERNELS; ++i) {
    if (ms) ms[i] = pool->ms[i];
    if (launches) launches[i] = pool->launches[i];
  }
  memset(pool->ms, 0, sizeof(pool->ms));
  memset(pool->launches, 0, sizeof(pool->launches));
  return GP_OK;
}

int64_t gp_launch_count(gp_pool* pool) { return pool ? pool->launch_count : 0; }

}  // extern "C"
