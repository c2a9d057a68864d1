// Capacity-boundary work (Sec. 3.2 - 3.3, App. D.1, App. D.2), every step, behind the attention kernel.
// That kernel leaves, for every (request at a boundary, layer, KV head) unit and both calibrated summaries,
// exp(logit - the page's maximum logit) of every candidate key, and per 16-token page the maximum and the sum of
// those exponentials.  The work on them, in the order of its dependences:
//
//   selection jobs    per unit, three independent jobs, one CTA each: per-head softmax over the candidate
//                     set and group mean -> a^S or a^L and its working-set size K^S or K^L (Eq. 7); and,
//                     speculatively, the b slots a compression would evict (Eq. 9, Eq. 10).  Under the
//                     Shrink policy a fourth job lists the 2b slots a Shrink would evict (Eq. 13).
//   decisions         by the CTA that finishes its jobs last: Eq. 8 per request, the action (grow, compress,
//                     shrink), the device allocator: grants first, then copy-on-write targets, each in ascending
//                     request id.
//   compaction        per compressing unit: stable in-place compaction into (P-1) b slots ((P-2) b at a Shrink),
//                     writing to copy-on-write targets where the source page is shared.  Work is claimed from a
//                     ticket counter, a chunk of 64 source slots at a time (a chunk publishes "my sources are
//                     read" before the next chunk may overwrite their tail) or, with many units, a unit at a
//                     time.  The last CTA swaps in the target pages, drops the references to the replaced ones
//                     and returns the last page of every request that shrank.
//   merge             of the partial attention outputs of requests that were split over several work items.
//
// It comes in two shapes that run the same device functions:
//   gp_chain_kernel                       all of it in one kernel (the deciding CTA tells the others through a flag):
//                                         behind the attention kernel of its own step, with every job waiting for the
//                                         attention kernel's report that its unit is complete (synchronous mode), or
//                                         beside the attention kernel of the next step (asynchronous mode);
//   gp_bsel_kernel, gp_compact_kernel     selection + decisions + merge, then compaction, as kernels of their own
//   (and gp_decide_kernel)                (large pools, the layer-by-layer step; with the KV heads spread over several
//                                         pools the decisions wait for the sums of all pools in a kernel of their own).
//
// Everything that decides an integer outcome is fp64.  Top-p counting and the eviction cut work on the
// IEEE bit patterns of the (non-negative) scores: one pass into a two-level histogram (4096 fine bins under
// 256 coarse ones) when the scores' top bits are uniform, else a radix descent, 11 bits per level; the
// histograms live in shared memory, and the top-p mass is accumulated in 2^62 fixed point with integer
// atomics, so the result does not depend on the order in which threads add.
#include "../../include/growpage.h"
#include "gp_dev.cuh"

namespace {

constexpr int NBINS = 2048;
constexpr int NBINS_PAD = NBINS + NBINS / 8;     // bins are stored at b + (b >> 3): a thread's 8 consecutive bins and
#define HIDX(b) ((b) + ((b) >> 3))              // its neighbours' then fall into different banks
constexpr double TWO62 = 4611686018427387904.0;
constexpr int SEL_T = 256;           // threads of the selection kernel
constexpr int SEL_NW = SEL_T / 32;
constexpr int SEL_CAP = 6144;        // candidate tokens whose scores are staged in shared memory
constexpr int CT = 256;              // threads of the compaction kernel
constexpr int MOVE_TOK = GP_MOVE_TOK;     // source slots per compaction chunk
constexpr int CMP_SHRINK = 1 << 30;       // flag on a compressing request's boundary index: the action is a Shrink

__device__ __forceinline__ unsigned long long to_fix(double a) {
  return (unsigned long long)__double2ll_rn(a * TWO62);
}

struct PairCU { unsigned c; unsigned long long s; };

// exclusive suffix sum over the block: sum of the values of threads with a higher id
template <int BT>
__device__ __forceinline__ PairCU block_suffix_excl(unsigned c, unsigned long long s, unsigned* wc,
                                                    unsigned long long* wsum) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned ic = c; unsigned long long is = s;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    unsigned tc = __shfl_down_sync(0xffffffffu, ic, off);
    unsigned long long ts = __shfl_down_sync(0xffffffffu, is, off);
    if (lane + off < 32) { ic += tc; is += ts; }
  }
  if (lane == 0) { wc[warp] = ic; wsum[warp] = is; }
  __syncthreads();
  PairCU r; r.c = ic - c; r.s = is - s;
  for (int w = warp + 1; w < BT / 32; ++w) { r.c += wc[w]; r.s += wsum[w]; }
  __syncthreads();
  return r;
}
// exclusive prefix count over the block
template <int BT>
__device__ __forceinline__ unsigned block_prefix_excl(unsigned c, unsigned* wc) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned ic = c;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    unsigned tc = __shfl_up_sync(0xffffffffu, ic, off);
    if (lane >= off) ic += tc;
  }
  if (lane == 31) wc[warp] = ic;
  __syncthreads();
  unsigned r = ic - c;
  for (int w = 0; w < warp; ++w) r += wc[w];
  __syncthreads();
  return r;
}

__device__ __constant__ int kWidths[6] = {11, 11, 11, 11, 11, 8};   // 63 bits below the sign

// 64-bit add into a (low, high) pair of 32-bit shared-memory words with two native atomics; the pair is
// exact once all adds have landed (the carry travels with the high word's add).
__device__ __forceinline__ void add64_split(unsigned* lo, unsigned* hi, unsigned long long x) {
  const unsigned xl = (unsigned)x, xh = (unsigned)(x >> 32);
  const unsigned old = atomicAdd(lo, xl);
  const unsigned carry = (old + xl) < old ? 1u : 0u;
  if (xh + carry) atomicAdd(hi, xh + carry);
}

// Eq. 7: smallest k such that the k largest of a[0..n) sum to at least p.
template <int BT>
__device__ __noinline__ int top_p_count(const GpDev& p, const double* a, int n, unsigned long long p_fix, unsigned* hcnt,
                           unsigned long long* hsum64, unsigned* wc, unsigned long long* wsum, long long* s_res) {
  unsigned* hlo = reinterpret_cast<unsigned*>(hsum64);
  unsigned* hhi = hlo + NBINS_PAD;
  const int tid = threadIdx.x;
  unsigned long long prefix = 0;
  unsigned cnt_above = 0;
  unsigned long long sum_above = 0;
  int shift = 63;
  int bin_star = 0;
  for (int lvl = 0; lvl < 6; ++lvl) {
    const int w = kWidths[lvl];
    shift -= w;
    const int nb = 1 << w;
    for (int i = tid; i < nb + (nb >> 3); i += BT) { hcnt[i] = 0; hlo[i] = 0; hhi[i] = 0; }
    if (tid == 0) s_res[0] = -1;
    __syncthreads();
    for (int i = tid; i < n; i += BT) {
      const double v = a[i];
      const unsigned long long key = (unsigned long long)__double_as_longlong(v);
      if (lvl == 0 || (key >> (shift + w)) == prefix) {
        const int bin = (int)((key >> shift) & (unsigned long long)(nb - 1));
        atomicAdd(&hcnt[HIDX(bin)], 1u);
        add64_split(&hlo[HIDX(bin)], &hhi[HIDX(bin)], to_fix(v));
      }
    }
    __syncthreads();
    const int per = nb / BT > 0 ? nb / BT : 1;
    const int lo = tid * per, hi = lo + per;     // this thread's bins [lo, hi)
    unsigned c = 0; unsigned long long s = 0;
    if (lo < nb) for (int b = lo; b < hi; ++b) { c += hcnt[HIDX(b)]; s += ((unsigned long long)hhi[HIDX(b)] << 32) + hlo[HIDX(b)]; }
    PairCU ex = block_suffix_excl<BT>(c, s, wc, wsum);
    if (lo < nb) {
      unsigned long long run_s = sum_above + ex.s;
      unsigned run_c = cnt_above + ex.c;
      for (int b = hi - 1; b >= lo; --b) {
        const unsigned long long before = run_s;
        run_s += ((unsigned long long)hhi[HIDX(b)] << 32) + hlo[HIDX(b)];
        if (before < p_fix && run_s >= p_fix) { s_res[0] = b; s_res[1] = run_c; s_res[2] = (long long)before; }
        run_c += hcnt[HIDX(b)];
      }
    }
    __syncthreads();
    if (s_res[0] < 0) return n;                  // rounding kept the total below p: everything
    bin_star = (int)s_res[0];
    cnt_above = (unsigned)s_res[1];
    sum_above = (unsigned long long)s_res[2];
    const unsigned cstar = hcnt[HIDX(bin_star)];
    __syncthreads();
    if (cstar == 1) return (int)cnt_above + 1;
    prefix = (prefix << w) | (unsigned long long)bin_star;
  }
  // all bits fixed: the bin holds copies of one value
  const unsigned c = hcnt[HIDX(bin_star)];
  const unsigned long long f = (((unsigned long long)hhi[HIDX(bin_star)] << 32) + hlo[HIDX(bin_star)]) / c;
  unsigned long long j = (p_fix - sum_above + f - 1) / f;
  if (j < 1) j = 1;
  if (j > c) j = c;
  __syncthreads();
  return (int)cnt_above + (int)j;
}

// ------------------------------------------------------------------------------------------------------
// fast path: one pass fills a 4096-bin histogram and its 256-bin summary; a one-warp sort finishes
// ------------------------------------------------------------------------------------------------------
// Scores of a candidate set are probabilities of similar magnitude: bits 62..58 of their IEEE patterns are
// nearly always the same (the softmax pass reports whether they are).  Then bits 57..46 (low exponent bits and
// the top of the mantissa) order the scores finely enough that the crossing point falls into a bin with a
// handful of members.  The 256-bin summary (bits 57..50) is scanned by the block, one bin per thread; the 16
// fine bins under the crossing summary bin by half a warp; the members of the crossing fine bin are sorted by
// one warp.  When the top bits differ or the bin is crowded, the callers fall back on the general radix
// descent above.
constexpr int FBINS = 4096;
constexpr int FB_PAD = FBINS + FBINS / 16;       // plane stride (the general routine pads its bins)
constexpr int CBINS = 256;                       // summary bins: 16 fine bins each, one per thread
constexpr int FSHIFT = 46;
static_assert(CBINS <= SEL_T, "one summary bin per thread");

struct FastHist {
  unsigned* cnt; unsigned* lo; unsigned* hi;       // [FBINS] members, and their fixed-point mass in two halves
  unsigned* ccnt; unsigned* clo; unsigned* chi;    // [CBINS] the same per summary bin
};

__device__ __forceinline__ void fast_hist_zero(const FastHist& H, bool with_mass) {
  const uint4 z = make_uint4(0, 0, 0, 0);
  for (int i = threadIdx.x; i < FBINS / 4; i += SEL_T) {
    reinterpret_cast<uint4*>(H.cnt)[i] = z;
    if (with_mass) { reinterpret_cast<uint4*>(H.lo)[i] = z; reinterpret_cast<uint4*>(H.hi)[i] = z; }
  }
  if (threadIdx.x < CBINS) {
    H.ccnt[threadIdx.x] = 0;
    if (with_mass) { H.clo[threadIdx.x] = 0; H.chi[threadIdx.x] = 0; }
  }
}

// sorts (v, tag) across the 32 lanes: descending v when DESC, else ascending v with larger tag first among
// equal v
template <bool DESC>
__device__ __forceinline__ void warp_sort(double& v, int& tag) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
    for (int j = k >> 1; j > 0; j >>= 1) {
      const double ov = __shfl_xor_sync(0xffffffffu, v, j);
      const int ot = __shfl_xor_sync(0xffffffffu, tag, j);
      // "first" = the element that belongs earlier in the final order
      const bool mine_first = DESC ? (v > ov || (v == ov && tag < ot)) : (v < ov || (v == ov && tag > ot));
      const bool want_first = (((lane & k) == 0) == ((lane & j) == 0));
      if (mine_first != want_first) { v = ov; tag = ot; }
    }
  }
}

// Eq. 7 on the fast path (histograms already zeroed, s_res[0] = -1, *s_cnt = 0); returns -1 when the general
// routine has to take over
__device__ int top_p_fast(const GpDev& p, const double* a, int n, unsigned long long p_fix, const FastHist& H,
                          unsigned* wc, unsigned long long* wsum, long long* s_res, double* list, int* s_cnt) {
  const int tid = threadIdx.x;
  for (int i = tid; i < n; i += SEL_T) {
    const double v = a[i];
    const int bin = (int)(((unsigned long long)__double_as_longlong(v) >> FSHIFT) & (FBINS - 1));
    const unsigned long long f = to_fix(v);
    atomicAdd(&H.cnt[bin], 1u);
    add64_split(&H.lo[bin], &H.hi[bin], f);
    atomicAdd(&H.ccnt[bin >> 4], 1u);
    add64_split(&H.clo[bin >> 4], &H.chi[bin >> 4], f);
  }
  __syncthreads();
  {                                               // summary level: thread t owns bin t; higher bins = larger scores
    const unsigned c = tid < CBINS ? H.ccnt[tid] : 0u;
    const unsigned long long m = tid < CBINS ? ((unsigned long long)H.chi[tid] << 32) + H.clo[tid] : 0ull;
    const PairCU ex = block_suffix_excl<SEL_T>(c, m, wc, wsum);
    if (tid < CBINS && ex.s < p_fix && ex.s + m >= p_fix) { s_res[0] = tid; s_res[1] = ex.c; s_res[2] = (long long)ex.s; }
  }
  __syncthreads();
  if (s_res[0] < 0) return n;                    // rounding kept the total below p: everything
  if (tid < 32) {                                // fine level: lane j owns the (j+1)-th highest bin of the 16
    const int cb = (int)s_res[0];
    const int fb = cb * 16 + 15 - (tid & 15);
    const unsigned c = tid < 16 ? H.cnt[fb] : 0u;
    const unsigned long long m = tid < 16 ? ((unsigned long long)H.hi[fb] << 32) + H.lo[fb] : 0ull;
    unsigned ic = c; unsigned long long im = m;
#pragma unroll
    for (int off = 1; off < 16; off <<= 1) {
      const unsigned tc = __shfl_up_sync(0xffffffffu, ic, off);
      const unsigned long long tm = __shfl_up_sync(0xffffffffu, im, off);
      if (tid >= off) { ic += tc; im += tm; }
    }
    const unsigned long long before = (unsigned long long)s_res[2] + im - m;
    if (tid < 16 && before < p_fix && before + m >= p_fix) {
      s_res[4] = fb; s_res[5] = s_res[1] + (long long)(ic - c); s_res[6] = (long long)before; s_res[7] = c;
    }
  }
  __syncthreads();
  const int bstar = (int)s_res[4];
  const unsigned cnt_above = (unsigned)s_res[5];
  const unsigned long long sum_above = (unsigned long long)s_res[6];
  const unsigned cstar = (unsigned)s_res[7];
  if (cstar == 1) return (int)cnt_above + 1;
  if (cstar > 32) return -1;
  for (int i = tid; i < n; i += SEL_T) {
    const double v = a[i];
    if ((int)(((unsigned long long)__double_as_longlong(v) >> FSHIFT) & (FBINS - 1)) == bstar) list[atomicAdd(s_cnt, 1)] = v;
  }
  __syncthreads();
  if (tid < 32) {
    double v = tid < (int)cstar ? list[tid] : -1.0;
    int tag = tid;
    warp_sort<true>(v, tag);
    unsigned long long inc = tid < (int)cstar ? to_fix(v) : 0ull;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const unsigned long long o = __shfl_up_sync(0xffffffffu, inc, off);
      if (tid >= off) inc += o;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, tid < (int)cstar && sum_above + inc >= p_fix);
    if (tid == 0) s_res[3] = (long long)cnt_above + (hit ? __ffs(hit) : (int)cstar);
  }
  __syncthreads();
  return (int)s_res[3];
}

// Eq. 10 global cut on the fast path (counts already zeroed, s_res[0] = -1, s_cnt[0..1] = 0): lists the ne
// (b, or 2b for a Shrink) evicted slots in ev[] (unsorted) and returns true, or returns false when the general routine has to take
// over.  `a` holds Eq. 9 scores, `loc` the block-local quota bits (those slots are never evicted).
__device__ bool evict_fast(const double* a, int nC, const unsigned* loc, const FastHist& H, unsigned* wc, long long* s_res,
                           double* list, int* list_slot, int* s_cnt, int* ev, const unsigned ne) {
  const int tid = threadIdx.x;
  for (int i = tid; i < nC; i += SEL_T) {
    if (!((loc[i >> 5] >> (i & 31)) & 1u)) {
      const int bin = (int)(((unsigned long long)__double_as_longlong(a[i]) >> FSHIFT) & (FBINS - 1));
      atomicAdd(&H.cnt[bin], 1u);
      atomicAdd(&H.ccnt[bin >> 4], 1u);
    }
  }
  __syncthreads();
  {                                               // summary level, ascending: the b lowest scores go
    const unsigned c = tid < CBINS ? H.ccnt[tid] : 0u;
    const unsigned ex = block_prefix_excl<SEL_T>(c, wc);
    if (tid < CBINS && ex < ne && ex + c >= ne) { s_res[0] = tid; s_res[1] = ex; }
  }
  __syncthreads();
  if (s_res[0] < 0) return false;
  if (tid < 32) {
    const int fb = (int)s_res[0] * 16 + (tid & 15);
    const unsigned c = tid < 16 ? H.cnt[fb] : 0u;
    unsigned ic = c;
#pragma unroll
    for (int off = 1; off < 16; off <<= 1) {
      const unsigned tc = __shfl_up_sync(0xffffffffu, ic, off);
      if (tid >= off) ic += tc;
    }
    const unsigned before = (unsigned)s_res[1] + ic - c;
    if (tid < 16 && before < ne && before + c >= ne) { s_res[4] = fb; s_res[5] = before; s_res[6] = c; }
  }
  __syncthreads();
  const int bstar = (int)s_res[4];
  const int cnt_below = (int)s_res[5], cstar = (int)s_res[6];
  const bool exact = (cnt_below + cstar == (int)ne);
  if (!exact && cstar > 32) return false;
  for (int i = tid; i < nC; i += SEL_T) {
    if (!((loc[i >> 5] >> (i & 31)) & 1u)) {
      const int bin = (int)(((unsigned long long)__double_as_longlong(a[i]) >> FSHIFT) & (FBINS - 1));
      if (bin < bstar || (exact && bin == bstar)) ev[atomicAdd(&s_cnt[0], 1)] = i;
      else if (bin == bstar) { const int at = atomicAdd(&s_cnt[1], 1); list[at] = a[i]; list_slot[at] = i; }
    }
  }
  __syncthreads();
  if (!exact && tid < 32) {                      // the lowest scores of the bin, later slots first among equals
    double v = tid < cstar ? list[tid] : INFINITY;
    int slot = tid < cstar ? list_slot[tid] : -1;
    warp_sort<false>(v, slot);
    if (tid < (int)ne - cnt_below) ev[cnt_below + tid] = slot;
  }
  __syncthreads();
  return true;
}

// Eq. 10 global cut, general routine (radix descent over the score bits): lists the ne evicted slots in ev[]
__device__ __noinline__ void evict_general(const GpDev& p, const double* a, int nC, const unsigned* loc, unsigned* hcnt,
                                           unsigned* wc, long long* s_res, int* s_i, int* ev, const unsigned ne) {
  const int tid = threadIdx.x;
      __syncthreads();
    unsigned long long prefix = 0;
  unsigned cnt_below = 0;
  unsigned long long thr = 0;        // evict keys strictly below thr ...
  unsigned long long tie_key = 0;    // ... and need_eq of the highest slots whose key equals tie_key
  int need_eq = 0;
  {
    int shift = 63;
    bool done = false;
    for (int lvl = 0; lvl < 6 && !done; ++lvl) {
      const int w = kWidths[lvl];
      shift -= w;
      const int nb = 1 << w;
      for (int i = tid; i < nb + (nb >> 3); i += SEL_T) hcnt[i] = 0;
      if (tid == 0) s_res[0] = -1;
      __syncthreads();
      for (int i = tid; i < nC; i += SEL_T) {
        if (!((loc[i >> 5] >> (i & 31)) & 1u)) {
          const unsigned long long key = (unsigned long long)__double_as_longlong(a[i]);
          if (lvl == 0 || (key >> (shift + w)) == prefix)
            atomicAdd(&hcnt[HIDX((int)((key >> shift) & (unsigned long long)(nb - 1)))], 1u);
        }
      }
      __syncthreads();
      const int per = nb / SEL_T > 0 ? nb / SEL_T : 1;
      const int lo = tid * per, hi = lo + per;
      unsigned c = 0;
      if (lo < nb) for (int b = lo; b < hi; ++b) c += hcnt[HIDX(b)];
      const unsigned ex = block_prefix_excl<SEL_T>(c, wc);
      if (lo < nb) {
        unsigned run = cnt_below + ex;
        for (int b = lo; b < hi; ++b) {
          const unsigned before = run;
          run += hcnt[HIDX(b)];
          if (before < ne && run >= ne) { s_res[0] = b; s_res[1] = before; }
        }
      }
      __syncthreads();
      if (s_res[0] < 0) {                                  // fewer than b candidates: cannot happen
        if (tid == 0) atomicOr(p.err, GP_E_BOUNDS);
        break;
      }
      const int bin_star = (int)s_res[0];
      cnt_below = (unsigned)s_res[1];
      const unsigned cstar = hcnt[HIDX(bin_star)];
      __syncthreads();
      prefix = (prefix << w) | (unsigned long long)bin_star;
      if (cnt_below + cstar == ne) {        // the bin fits exactly: no tie to break
        thr = (prefix + 1ull) << shift;
        done = true;
      }
    }
    if (!done) {                                           // equal scores straddle the cut
      thr = prefix;
      tie_key = prefix;
      need_eq = (int)ne - (int)cnt_below;
    }
  }
  for (int i = tid; i < nC; i += SEL_T) {
    if (!((loc[i >> 5] >> (i & 31)) & 1u)) {
      const unsigned long long key = (unsigned long long)__double_as_longlong(a[i]);
      if (key < thr) { const int at = atomicAdd(&s_i[0], 1); if (at < (int)ne) ev[at] = i; }
    }
  }
  __syncthreads();
  if (tid == 0) {
    int cntv = s_i[0];
    for (int i = nC - 1; i >= 0 && need_eq > 0; --i) {     // rare: older (lower) slots win ties
      if (!((loc[i >> 5] >> (i & 31)) & 1u)) {
        const unsigned long long key = (unsigned long long)__double_as_longlong(a[i]);
        if (key == tie_key) { if (cntv < (int)ne) ev[cntv] = i; ++cntv; --need_eq; }
      }
    }
    if (cntv != (int)ne) atomicOr(p.err, GP_E_BOUNDS);
  }
}

// ------------------------------------------------------------------------------------------------------
// decision + allocator, run by the last CTA of the selection kernel
// ------------------------------------------------------------------------------------------------------
__device__ void decide_and_allocate(const GpDev& p, const int* req_ids, int n_req, int n_bnd, int* actions, int* s_arr,
                                    int serial, bool from_sums = false) {
  // from_sums: the sums of K^S and K^L come from shard_sums (summed over the pools that hold the model's other KV
  // heads) instead of this pool's own accumulators
  // In the asynchronous boundary mode this runs beside the next decode step: it touches only the requests at
  // this step's boundary (which sit that step out), reads the free list itself (the boundary chains run one
  // after the other and nothing else takes or returns pages meanwhile) and reports through last_act only
  // (`actions` is null: the caller's array belongs to a step that has ended).
  int* s_want = s_arr;
  int* s_ksh = s_arr + GP_MAX_REQ;
  int* s_P = s_arr + 2 * GP_MAX_REQ;
  int* s_order = s_arr + 3 * GP_MAX_REQ;
  int* s_req = s_arr + 4 * GP_MAX_REQ;
  int* s_base = s_arr + 5 * GP_MAX_REQ;
  int* s_bi = s_arr + 6 * GP_MAX_REQ;
  int* s_free = s_arr + 7 * GP_MAX_REQ;      // the free pages the grants of this step can take, top first
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarp = blockDim.x >> 5;
  // everything the decisions need arrives in one round trip: the jobs summed K^S and K^L per request, a job
  // counted its shared pages, and the plan kernel copied the top of the free list
  const int LH = p.L * p.Hkv;
  const int n_active = p.hdr[HDR_N_ACTIVE];
  int top0 = 0;
  if (n_bnd > 0) {
    top0 = p.async ? __ldcg(p.free_top) : __ldcg(p.free_peek);
    for (int e = tid; e < n_bnd; e += blockDim.x) {
      const int4 inf = p.bnd_info[2 * e];
      int4 acc = __ldcg(reinterpret_cast<const int4*>(p.bnd_acc) + e);
      if (from_sums) { acc.x = __ldcg(p.shard_sums + 2 * e); acc.y = __ldcg(p.shard_sums + 2 * e + 1); }
      s_free[e] = p.async ? (e < top0 ? __ldcg(p.free_stack + top0 - 1 - e) : 0) : __ldcg(p.free_peek + 1 + e);
      const int r = inf.y, Pr = inf.z;
      const int nC = (Pr - p.sub) * GP_PAGE;                // |C_t| of Eq. 7: history minus the newest page of the method
      // Eq. 8 with a common |C|: Delta = (sum K^S - sum K^L) / (N |C|), one division of exact integers
      double delta = 0.0;
      int want = 1;
      if (nC > 0) {
        delta = (double)((long long)acc.x - (long long)acc.y) / ((double)p.units_total * (double)nC);
        if (p.metric == GP_METRIC_ENTROPY) {
          // the same mean with H / ln |C| in the place of K / |C|, summed unit by unit in (layer, head) order
          const double* hx = p.Hx + (size_t)r * LH * 2;
          double accd = 0.0;
          for (int u2 = 0; u2 < LH; ++u2) accd += __ldcg(hx + 2 * u2) - __ldcg(hx + 2 * u2 + 1);
          delta = nC > 1 ? accd / ((double)LH * log((double)nC)) : 0.0;
        }
        want = delta > p.tau;
        if (p.policy == 1) {                                  // the reversed reading of the demand signal
          want = !want;
        } else if (p.policy == 2) {                           // frequency-matched random control
          unsigned long long zz = p.policy_seed + 0x9E3779B97F4A7C15ull * (unsigned long long)(r + 1) +
                                  0xBF58476D1CE4E5B9ull * (unsigned long long)inf.w;
          zz = (zz ^ (zz >> 30)) * 0xBF58476D1CE4E5B9ull;
          zz = (zz ^ (zz >> 27)) * 0x94D049BB133111EBull;
          zz ^= zz >> 31;
          want = !((double)(zz >> 11) * (1.0 / 9007199254740992.0) < p.p_compress);
        } else if (p.policy == GP_POLICY_SHRINK) {            // Eq. 13: the third action, where it is admissible
          if (!want && delta < p.shrink_below && Pr - p.sub >= p.min_pages_after_shrink) want = 16;
        }
      }
      p.delta[r] = delta;
      // pages and slots as the step left them (full); the allocator below changes what the decision changes.  In
      // the asynchronous mode the plan of the step in between leaves these two words of a held request alone.
      p.P[r] = Pr; p.n[r] = Pr * GP_PAGE;
      s_want[e] = want; s_ksh[e] = acc.z; s_P[e] = Pr; s_req[e] = r; s_bi[e] = inf.x;
    }
  }
  if (tid == 0) {
    atomicAdd(reinterpret_cast<unsigned long long*>(p.counters + 5), 1ull);
    atomicAdd(reinterpret_cast<unsigned long long*>(p.counters + 6), (unsigned long long)n_active);
    p.hdr[HDR_WORK_CMP] = 0;
    if (n_bnd == 0) { p.hdr[HDR_N_CMP] = 0; p.hdr[HDR_N_CITEM] = 0; p.hdr[HDR_N_COW] = 0; }
  }
  if (n_bnd == 0) return;
  __syncthreads();
  for (int e = tid; e < n_bnd; e += blockDim.x) {
    int rank = 0;
    for (int f = 0; f < n_bnd; ++f) rank += (s_req[f] < s_req[e]);
    s_order[rank] = e;
  }
  __syncthreads();
  auto report = [&](int bi, int r, int act) {
    if (actions) actions[bi] = act;
    p.last_act[r] = act;
  };
  if (tid == 0) {                                        // sequential allocator: shared memory only
    int top = top0;
    int n_cmp = 0, chunks = 0;
    unsigned long long grow = 0, comp = 0, fall = 0, stall = 0, cow = 0, scored = 0, shr = 0;
    const int sub = p.sub;
    for (int k = 0; k < n_bnd; ++k) {                    // pass 1: grants, ascending request id
      const int e = s_order[k];
      const int r = s_req[e], Pr = s_P[e], bi = s_bi[e];
      scored += (unsigned long long)(Pr - sub) * GP_PAGE;
      if ((s_want[e] & 1) && Pr + sub <= p.cap && top >= sub) {
        // one page of the method: `sub` tiles from the top of the free list
        for (int t = 0; t < sub; ++t) {
          const int page = (sub == 1 && !p.async) ? s_free[top0 - top] : p.free_stack[top - 1];
          --top;
          p.refcount[page] = 1;
          p.page_table[(size_t)r * p.cap + Pr + t] = page;
        }
        p.P[r] = Pr + sub;
        report(bi, r, GP_ACT_GROW);
        s_want[e] |= 2;
        ++grow;
      } else if (Pr == sub) {
        report(bi, r, GP_ACT_STALLED);
        s_want[e] |= 4;
        ++stall;
      }
    }
    for (int k = 0; k < n_bnd; ++k) {                    // pass 2: copy-on-write targets
      const int e = s_order[k];
      if (s_want[e] & 6) continue;
      const int r = s_req[e], bi = s_bi[e];
      if (s_ksh[e] > top) {
        report(bi, r, GP_ACT_STALLED);
        ++stall;
        continue;
      }
      s_base[e] = top;
      top -= s_ksh[e];
      cow += s_ksh[e];
      const bool shrink = (s_want[e] & 16) != 0;
      p.cmp_info[n_cmp] = make_int4(r, s_P[e], e | (shrink ? CMP_SHRINK : 0), chunks);
      chunks += (s_P[e] * GP_PAGE + MOVE_TOK - 1) / MOVE_TOK;
      ++n_cmp;
      if (s_want[e] & 1) { report(bi, r, GP_ACT_COMPRESS_FALLBACK); ++fall; }
      else if (shrink) { report(bi, r, GP_ACT_SHRINK); ++shr; }
      else { report(bi, r, GP_ACT_COMPRESS); ++comp; }
      // a compression frees one page worth of slots; a Shrink frees two and gives the last page back (the
      // compaction kernel returns it once nothing reads it any more)
      p.n[r] = (s_P[e] - (shrink ? 2 : 1) * sub) * GP_PAGE;
      if (shrink) p.P[r] = s_P[e] - sub;
      p.n_pristine[r] = 0;
      s_want[e] |= 8;
    }
    p.cmp_info[n_cmp] = make_int4(0, 0, 0, chunks);
    if (top < 0) atomicOr(p.err, GP_E_FREELIST);
    *p.free_top = top;
    p.hdr[HDR_N_CMP] = n_cmp;
    p.hdr[HDR_N_CITEM] = chunks * LH;
    p.hdr[HDR_N_COW] = (int)(cow + shr);           // page-table work left for the compaction kernel's last CTA
    unsigned long long* cn = reinterpret_cast<unsigned long long*>(p.counters);
    if (grow) atomicAdd(cn + 0, grow);
    if (comp) atomicAdd(cn + 1, comp);
    if (fall) atomicAdd(cn + 2, fall);
    if (stall) atomicAdd(cn + 3, stall);
    if (cow) atomicAdd(cn + 4, cow);
    if (shr) atomicAdd(cn + 10, shr);
    atomicAdd(cn + 9, scored);
  }
  __syncthreads();
  for (int e = warp; e < n_bnd; e += nwarp) {             // fill in the targets, in table order
    if (!(s_want[e] & 8) || s_ksh[e] == 0) continue;
    const int r = s_req[e], Pr = s_P[e], base = s_base[e];
    const int* table = p.page_table + (size_t)r * p.cap;
    int* shadow = p.shadow + (size_t)r * p.cap;
    int running = 0;
    for (int j0 = 0; j0 < Pr - p.sub; j0 += 32) {
      const int j = j0 + lane;
      const bool sh = j < Pr - p.sub && p.refcount[table[j]] > 1;
      const unsigned mask = __ballot_sync(0xffffffffu, sh);
      if (sh) {
        const int newp = p.free_stack[base - 1 - (running + __popc(mask & ((1u << lane) - 1u)))];
        shadow[j] = newp;
        p.refcount[newp] = 1;
      }
      running += __popc(mask);
    }
  }
}

// one copy of the fp64 exponential in the image: the selection jobs run once per launch, so what they cost
// is mostly the fetching of their instructions
__device__ __noinline__ double exp_once(double x) { return exp(x); }
// factor of a page and column when the factors' table does not fit (very large candidate sets)
__device__ __noinline__ double factor_slow(const double* zs_entry, double M) { return exp(__ldcg(zs_entry) - M); }

// L2 loads the compiler may not sink towards their first use: the selection jobs issue all loads of a phase
// together and only then wait (a plain load is free to drift past the block barriers in between)
__device__ __forceinline__ double2 ld_early2(const double* ptr) {
  double2 v;
  asm volatile("ld.global.cg.v2.f64 {%0, %1}, [%2];" : "=d"(v.x), "=d"(v.y) : "l"(ptr));
  return v;
}

// max or sum over the block of one value per thread, separately for each of `ncols` interleaved columns
// (thread t belongs to column t % ncols); fixed shuffle tree, so the sum does not depend on timing
template <bool IS_MAX>
__device__ __forceinline__ void column_reduce(double v, int ncols, double* red, double* result) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int off = ncols; off < 32; off <<= 1) {
    const double o = __shfl_xor_sync(0xffffffffu, v, off);
    v = IS_MAX ? fmax(v, o) : v + o;
  }
  if (lane < ncols) red[warp * 16 + lane] = v;
  __syncthreads();
  if (threadIdx.x < ncols) {
    double r = red[threadIdx.x];
    for (int w = 1; w < SEL_T / 32; ++w) r = IS_MAX ? fmax(r, red[w * 16 + threadIdx.x]) : r + red[w * 16 + threadIdx.x];
    result[threadIdx.x] = r;
  }
  __syncthreads();
}

// Per-head softmax over C and the group mean (Sec. 3.2), then a^S, a^L or s = max(a^S, a^L) (Eq. 9) of every
// candidate into a[].  The attention kernel left, per 16-token page t and column c, the page's maximum logit
// m_tc and s_tc = sum of exp(z - m_tc), and per token x = exp(z - m_tc).  With M_c the maximum over pages and
// f_tc = exp(m_tc - M_c):  softmax = x f_tc / Z_c,  Z_c = sum_t s_tc f_tc.  So this pass takes one exponential
// per page and column instead of one per token and column; the factors f_tc sit in shared memory (F, f_cap
// entries; when the candidate set has more page-columns than that, they are recomputed per token).
// All loads of the prologue (page partials and the first batch of x) are issued together.
template <int GG>
__device__ __noinline__ bool job_softmax(const GpDev& p, const double* __restrict__ x, size_t view_stride,
                                         const double* __restrict__ zs, double* __restrict__ a, int nC, int task,
                                         double* red, double* sM, double* sZ, double* F, int f_cap) {
  constexpr int G2 = 2 * GG;
  constexpr int U = 4;                                   // 16-byte loads per thread and view in flight
  constexpr int KEEP = 2;                                // page partials per thread held in registers
  constexpr int LPT = GG >= 2 ? GG / 2 : 1;              // lanes that share a token (two columns each)
  const int tid = threadIdx.x;
  const int nview = task == 2 ? 2 : 1;
  const int ncols = nview * GG;
  const int col0 = task == 1 ? GG : 0;
  const int myc = tid % ncols;                           // SEL_T is a multiple of ncols
  const int mycol = col0 + myc;
  const int ntile = nC / GP_PAGE;
  const int t0 = tid / ncols, tstep = SEL_T / ncols;
  const bool table = ntile * ncols <= f_cap;
  const int nv = nC * GG / 2;                            // 16-byte pieces of one view: consecutive lanes, consecutive pieces
  const double* xb = x + (task == 1 ? view_stride : 0);
  double2 keep[KEEP];
#pragma unroll
  for (int k = 0; k < KEEP; ++k) {
    const int t = t0 + k * tstep;
    keep[k] = make_double2(-INFINITY, 0.0);
    if (t < ntile) keep[k] = ld_early2(zs + ((size_t)t * G2 + mycol) * 2);
  }
  double2 xv[2][U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int k = tid + u * SEL_T;
    xv[0][u] = xv[1][u] = make_double2(0.0, 0.0);
    if (k < nv) {
      xv[0][u] = ld_early2(xb + 2 * (size_t)k);
      if (task == 2) xv[1][u] = ld_early2(xb + view_stride + 2 * (size_t)k);
    }
  }
  double m = fmax(keep[0].x, keep[1].x);
  for (int t = t0 + KEEP * tstep; t < ntile; t += tstep) m = fmax(m, __ldcg(zs + ((size_t)t * G2 + mycol) * 2));
  column_reduce<true>(m, ncols, red, sM);
  const double mc = sM[myc];
  double acc = 0.0;
#pragma unroll
  for (int k = 0; k < KEEP; ++k) {
    const int t = t0 + k * tstep;
    if (t < ntile) {
      const double f = exp_once(keep[k].x - mc);
      acc += keep[k].y * f;
      if (table) F[t * ncols + myc] = f;
    }
  }
  for (int t = t0 + KEEP * tstep; t < ntile; t += tstep) {
    const double2 ms = __ldcg(reinterpret_cast<const double2*>(zs + ((size_t)t * G2 + mycol) * 2));
    const double f = exp_once(ms.x - mc);
    acc += ms.y * f;
    if (table) F[t * ncols + myc] = f;
  }
  column_reduce<false>(acc, ncols, red, sZ);
  if (tid < ncols) sZ[tid] = 1.0 / ((double)GG * sZ[tid]);     // group mean and normaliser in one factor
  __syncthreads();
  unsigned top_bits = 0;
  for (int k0 = tid; k0 - tid < nv; k0 += U * SEL_T) {   // uniform trip count: the shuffles below need whole warps
    if (k0 != tid) {
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int k = k0 + u * SEL_T;
        xv[0][u] = xv[1][u] = make_double2(0.0, 0.0);
        if (k < nv) {
          xv[0][u] = __ldcg(reinterpret_cast<const double2*>(xb + 2 * (size_t)k));
          if (task == 2) xv[1][u] = __ldcg(reinterpret_cast<const double2*>(xb + view_stride + 2 * (size_t)k));
        }
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int k = k0 + u * SEL_T;
      const bool on = k < nv;
      const int flat = 2 * (on ? k : 0);
      const int tok = flat / GG, g = flat % GG;           // GG = 1: tokens tok and tok + 1 (same page), column 0
      const int t = tok / GP_PAGE;
      double part[2][2];                                  // [view][element of the piece]
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        part[q][0] = part[q][1] = 0.0;
        if (q < nview && on) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int c = q * GG + (GG == 1 ? 0 : g + e); // column of this job: index into F, sM, sZ
            const double f = table ? F[t * ncols + c] : factor_slow(zs + ((size_t)t * G2 + col0 + c) * 2, sM[c]);
            part[q][e] = (e == 0 ? xv[q][u].x : xv[q][u].y) * f * sZ[c];
          }
        }
      }
      if (GG == 1) {
        if (on) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const double s0 = task == 2 ? fmax(part[0][e], part[1][e]) : part[0][e];       // Eq. 9
            a[tok + e] = s0;
            top_bits |= 1u << (unsigned)(((unsigned long long)__double_as_longlong(s0) >> 58) & 31ull);
          }
        }
      } else {
        double sv0 = part[0][0] + part[0][1], sv1 = part[1][0] + part[1][1];
#pragma unroll
        for (int o = 1; o < LPT; o <<= 1) {
          sv0 += __shfl_xor_sync(0xffffffffu, sv0, o);
          sv1 += __shfl_xor_sync(0xffffffffu, sv1, o);
        }
        if (on && g == 0) {
          const double s0 = task == 2 ? fmax(sv0, sv1) : sv0;                              // Eq. 9
          a[tok] = s0;
          top_bits |= 1u << (unsigned)(((unsigned long long)__double_as_longlong(s0) >> 58) & 31ull);
        }
      }
    }
  }
  // bits 62..58 of every score, as a set: the fast selection path needs them all equal.  (The block-wide
  // barrier reductions combine predicates, not words, so the sets are OR-ed by hand: per warp, then over the
  // warps through shared memory; `red` is free here.)
  top_bits = __reduce_or_sync(0xffffffffu, top_bits);
  unsigned* sets = reinterpret_cast<unsigned*>(red);
  if ((tid & 31) == 0) sets[tid >> 5] = top_bits;
  __syncthreads();
  unsigned all_bits = 0;
#pragma unroll
  for (int w = 0; w < SEL_NW; ++w) all_bits |= sets[w];
  __syncthreads();
  return __popc(all_bits) == 1;
}

// Attention outputs of requests that were split over several work items: merges the items' partial results
// (running maximum in the log2 domain, sum of exponentials, unnormalised output) into the output row.  The
// calling CTA takes merges first, first + stride, ...
__device__ __noinline__ void merge_partials(const GpDev& p, int n_req, float* __restrict__ out, int n_mc, int n_rc,
                                            int first_item, int stride, int lh0, int lh_n) {
  const int G = p.G, D = p.d;
  const int PSTRIDE = G * (D + 2);
  for (long long mi = first_item; mi < (long long)n_mc * lh_n; mi += stride) {       // units [lh0, lh0 + lh_n)
    const int4 mc = p.mc_list[mi / lh_n];
    const int lh = lh0 + (int)(mi % lh_n), l = lh / p.Hkv, h = lh % p.Hkv;
    const int bi = mc.x, nch = mc.z;
    const float* first = p.partials + ((size_t)lh * n_rc + mc.y) * PSTRIDE;
    float* orow = out + (((size_t)l * n_req + bi) * p.Hq + h * G) * D;
    for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
      const int g = idx / D, dc = idx % D;
      const float* pg = first + g * (D + 2);
      float M = -INFINITY, acc = 0.f, ls = 0.f;
      for (int c0 = 0; c0 < nch; c0 += 4) {               // four items' values in flight together
        float m[4], lv[4], vv[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float* pc = pg + (size_t)(c0 + k) * PSTRIDE;
          const bool on = c0 + k < nch;
          m[k] = on ? __ldcg(pc + D) : -INFINITY;
          lv[k] = on ? __ldcg(pc + D + 1) : 0.f;
          vv[k] = on ? __ldcg(pc + dc) : 0.f;
        }
        const float Mn = fmaxf(fmaxf(M, fmaxf(m[0], m[1])), fmaxf(m[2], m[3]));
        const float sc = exp2f(M - Mn);
        acc *= sc; ls *= sc;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float w = exp2f(m[k] - Mn);
          acc += w * vv[k];
          ls += w * lv[k];
        }
        M = Mn;
      }
      orow[idx] = acc / ls;
    }
  }
}

// ------------------------------------------------------------------------------------------------------
// working sets + speculative eviction list; three independent jobs per unit (four under the Shrink policy: its
// list of 2b evictions), one CTA each; the last CTA decides
// ------------------------------------------------------------------------------------------------------
struct SelGeom {
  static constexpr size_t BUF_BYTES = SEL_CAP * sizeof(double);
  static constexpr size_t H_BYTES = (size_t)FB_PAD * 12;
  static constexpr size_t MISC_BYTES = SEL_NW * 8 + SEL_NW * 4 + 8 * 8 + 2 * GP_MAX_BLK * 4 + 16 * 4 + (SEL_NW * 16 + 32) * 8 + 32 * 8 + 32 * 4 + 3 * CBINS * 4;
};

// shared memory of the selection kernel
struct SelSmem {
  double* sbuf;                      // [SEL_CAP] a^S, a^L or s
  unsigned* hcnt;                    // histogram planes; the softmax factors F share them before the bins are used
  unsigned long long* hsum;
  unsigned long long* wsum;          // [SEL_NW]
  unsigned* wc;                      // [SEL_NW]
  long long* s_res;                  // [8]
  int* ev;                           // [2 * GP_MAX_BLK] evicted slots of the job
  int* s_i;                          // [16]
  double* red;                       // [SEL_NW][16]
  double* sM;                        // [16]
  double* sZ;                        // [16]
  double* flist;                     // [32] members of the crossing bin
  int* flist_slot;                   // [32]
  unsigned* loc;                     // [cap*b/32 + 1] block-local picks, one bit per candidate
  FastHist H;
};
constexpr int SEL_F_CAP = (int)(SelGeom::H_BYTES / sizeof(double));

__device__ __forceinline__ SelSmem sel_smem_at(uint8_t* smem) {      // smem: 256-byte aligned, gp_bsel_smem bytes
  SelSmem S;
  S.sbuf = reinterpret_cast<double*>(smem);
  S.hcnt = reinterpret_cast<unsigned*>(smem + SelGeom::BUF_BYTES);
  S.hsum = reinterpret_cast<unsigned long long*>(S.hcnt + FB_PAD);           // two u32 planes (low, high)
  S.wsum = S.hsum + FB_PAD;
  S.wc = reinterpret_cast<unsigned*>(S.wsum + SEL_NW);
  S.s_res = reinterpret_cast<long long*>(S.wc + SEL_NW);
  S.ev = reinterpret_cast<int*>(S.s_res + 8);
  S.s_i = S.ev + 2 * GP_MAX_BLK;
  S.red = reinterpret_cast<double*>(S.s_i + 16);
  S.sM = S.red + SEL_NW * 16;
  S.sZ = S.sM + 16;
  S.flist = S.sZ + 16;
  S.flist_slot = reinterpret_cast<int*>(S.flist + 32);
  unsigned* coarse = reinterpret_cast<unsigned*>(S.flist_slot + 32);           // [3][CBINS] summary bins
  S.loc = coarse + 3 * CBINS;
  S.H.cnt = S.hcnt; S.H.lo = reinterpret_cast<unsigned*>(S.hsum); S.H.hi = S.H.lo + FB_PAD;
  S.H.ccnt = coarse; S.H.clo = coarse + CBINS; S.H.chi = coarse + 2 * CBINS;
  return S;
}

// One selection job of a boundary unit: per-head softmax over the candidate set and the group mean from the
// attention kernel's per-page partials (`z`, `zs`), then either the working-set size of one view (task 0: K^S,
// 1: K^L; Eq. 7) or the `ne` slots a compression would evict (task 2; Eq. 9, Eq. 10).  The outputs go to Kout / acc
// (the request's running sum for Eq. 8) and evout.
__device__ __forceinline__ void sel_job(const GpDev& p, const SelSmem& S, const double* z, size_t view_stride, const double* zs,
                                     double* a, int nC, int task, int ne, int* Kout, int* acc, int* evout, double* Hout) {
  const int tid = threadIdx.x;
  if (task == 2) for (int i = tid; i < (nC + 31) / 32; i += SEL_T) S.loc[i] = 0;
  if (tid == 0) { S.s_res[0] = -1; S.s_i[0] = 0; S.s_i[5] = 0; S.s_i[6] = 0; S.s_i[7] = 0; }
  bool uniform;
  double* F = reinterpret_cast<double*>(S.hcnt);
  switch (p.G) {
    case 1: uniform = job_softmax<1>(p, z, view_stride, zs, a, nC, task, S.red, S.sM, S.sZ, F, SEL_F_CAP); break;
    case 2: uniform = job_softmax<2>(p, z, view_stride, zs, a, nC, task, S.red, S.sM, S.sZ, F, SEL_F_CAP); break;
    case 4: uniform = job_softmax<4>(p, z, view_stride, zs, a, nC, task, S.red, S.sM, S.sZ, F, SEL_F_CAP); break;
    default: uniform = job_softmax<8>(p, z, view_stride, zs, a, nC, task, S.red, S.sM, S.sZ, F, SEL_F_CAP); break;
  }
  if (task < 2 && p.metric == GP_METRIC_ENTROPY) {
    // the ablation's other metric: H = -sum a ln a of the view, summed in a fixed order (per thread over its
    // strided candidates, then a fixed tree), so that the same input gives the same bits on every run
    __syncthreads();
    double hsum = 0.0;
    for (int i = tid; i < nC; i += SEL_T) { const double v = a[i]; if (v > 0.0) hsum -= v * log(v); }
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) hsum += __shfl_xor_sync(0xffffffffu, hsum, o2);
    if ((tid & 31) == 0) S.red[tid >> 5] = hsum;
    __syncthreads();
    if (tid == 0) {
      double tot = 0.0;
      for (int w = 0; w < SEL_NW; ++w) tot += S.red[w];
      Kout[task] = 0;
      Hout[task] = tot;
    }
    __syncthreads();
    return;
  }
  fast_hist_zero(S.H, task < 2);                   // the factors' table shared this memory
  if (task < 2) {
    __syncthreads();
    // ---- Eq. 7 -------------------------------------------------------------------------------------------
    int K = uniform ? top_p_fast(p, a, nC, p.p_fix, S.H, S.wc, S.wsum, S.s_res, S.flist, &S.s_i[5]) : -1;
    if (K < 0) { __syncthreads(); K = top_p_count<SEL_T>(p, a, nC, p.p_fix, S.hcnt, S.hsum, S.wc, S.wsum, S.s_res); }
    if (tid == 0) {
      Kout[task] = K;
      atomicAdd(acc + task, K);                    // Eq. 8 needs only the sums over layers and heads
    }
    return;
  }
  // ---- Eq. 10, block-local quota: the k' best slots of every block of C (score desc, slot asc); a block is a
  // page of the method, the last one short when the protected window is smaller than the page -----------------
  const int blk = p.blk;
  const int nblk = (nC + blk - 1) / blk;
  const int K_t = nC - ne;
  const int kq = min(p.k_loc, K_t / nblk);
  if (kq > 0) {
    for (int i = tid; i < nC; i += SEL_T) {
      const double s = a[i];
      int rank = 0;
      if (blk == GP_PAGE) {
        const int b0 = i & ~15;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const double sj = a[b0 + j];
          rank += (sj > s) || (sj == s && (b0 + j) < i);
        }
      } else {
        const int b0 = (i / blk) * blk, b1 = min(b0 + blk, nC);
        for (int j = b0; j < b1; ++j) {
          const double sj = a[j];
          rank += (sj > s) || (sj == s && j < i);
        }
      }
      if (rank < kq) atomicOr(&S.loc[i >> 5], 1u << (i & 31));
    }
  }
  __syncthreads();
  // ---- global cut: the b lowest of the rest are evicted (score asc, slot desc) --------------------------------
  if (!uniform || !evict_fast(a, nC, S.loc, S.H, S.wc, S.s_res, S.flist, S.flist_slot, &S.s_i[6], S.ev, (unsigned)ne))
    evict_general(p, a, nC, S.loc, S.hcnt, S.wc, S.s_res, S.s_i, S.ev, (unsigned)ne);
  __syncthreads();
  for (int t = tid; t < ne; t += SEL_T) {                    // the evicted slots in ascending order, by rank
    const int mine = S.ev[t];
    int rank = 0;
    for (int j = 0; j < ne; ++j) rank += (S.ev[j] < mine);
    evout[rank] = mine;
  }
}

// Rarely taken tails of the selection kernel's last thread block, kept out of line so that they do not weigh on the
// register allocation of the jobs.
// Layer-by-layer step: the requests' counters move on at the end of the step (a whole-step launch does it where
// the attention kernel appends the token): one token further, the summary buffers swapped.  The first work item of
// a request names it once.
__device__ __noinline__ void advance_counters(const GpDev& p, int n_rc) {
  for (int idx = threadIdx.x; idx < n_rc; idx += blockDim.x) {
    const int* d = p.rcx + (size_t)idx * GP_DESC_INTS;
    if (d[4] == 0) {
      const int r = d[1];
      p.n[r] += 1; p.pos[r] += 1; p.started[r] = 1; p.sum_par[r] ^= 1;
    }
  }
  __syncthreads();
}
// A pool that holds a part of the model's KV heads: its sums of K^S and K^L per boundary request, zero past them
__device__ __noinline__ void publish_shard_sums(const GpDev& p, int n_bnd) {
  for (int e = threadIdx.x; e < p.M; e += blockDim.x) {
    p.shard_sums[2 * e] = e < n_bnd ? __ldcg(p.bnd_acc + 4 * e) : 0;
    p.shard_sums[2 * e + 1] = e < n_bnd ? __ldcg(p.bnd_acc + 4 * e + 1) : 0;
  }
}

template <bool SHR>      // SHR: the pool runs the Shrink policy (a fourth job per unit)
__global__ void __launch_bounds__(SEL_T, 2)
gp_bsel_kernel(const __grid_constant__ GpDev p, const int* __restrict__ req_ids, int n_req, int* __restrict__ actions,
               float* __restrict__ out, int serial, int decide) {
  // decide == 0: the step of a pool that holds a part of the model's KV heads: the last thread block only hands
  // out the sums of K^S and K^L per boundary request; the decisions follow in a kernel of their own once the
  // sums of all parts are added up
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((256u - (smem_u32(smem_raw) & 255u)) & 255u);
  SelSmem S = sel_smem_at(smem);
  int* s_i = S.s_i;
  // the decision scratch aliases the score staging area: it is used after the last item only

  const int tid = threadIdx.x;
  const int LH = p.L * p.Hkv;
  const int G = p.G, G2 = 2 * p.G;
  constexpr int NT = SHR ? 4 : 3;                           // jobs per unit: K^S, K^L, eviction list(s)
  // What the plan kernel wrote (counts, boundary records) is read before the wait for the attention kernel: the
  // plan kernel had completed before any CTA of the attention kernel let this grid be scheduled, and the
  // attention kernel does not touch these words; the loads go to the L2 (an L1 line could date from the step
  // before).  The first item's record is fetched before the number of items is known (same round trip); slots
  // of bnd_info past the count hold stale but readable data that is then not used.
  int4 inf_first = make_int4(0, 0, 0, 0), inf2_first = inf_first;
  {
    const int b0 = (int)(blockIdx.x / (NT * LH));
    if (b0 < p.M) { inf_first = __ldcg(p.bnd_info + 2 * b0); inf2_first = __ldcg(p.bnd_info + 2 * b0 + 1); }
  }
  const int n_bnd = __ldcg(p.hdr + HDR_N_BND);
  const int n_mc = out ? __ldcg(p.hdr + HDR_N_MC) : 0, n_rc = __ldcg(p.hdr + HDR_N_RC);   // out == null: already merged layer by layer
  const long long items = (long long)n_bnd * LH * NT;
  gp_pdl_wait();
  gp_pdl_launch_dependents();

  // CTAs without a job merge the split requests' attention partials while the others work; when fewer than a
  // quarter of the CTAs are idle, everybody merges after the jobs instead
  const long long n_busy = items + n_bnd < (long long)gridDim.x ? items + n_bnd : (long long)gridDim.x;
  const int n_idle = (int)gridDim.x - (int)n_busy;
  const bool idle_merge = n_idle * 4 >= (int)gridDim.x;
  if (idle_merge && (long long)blockIdx.x >= n_busy)
    merge_partials(p, n_req, out, n_mc, n_rc, (int)blockIdx.x - (int)n_busy, n_idle, 0, LH);

  for (long long item = blockIdx.x; item < items + n_bnd; item += gridDim.x) {
    if (item >= items) {
      // pages of C that other requests share: each needs a copy-on-write target if this request compresses
      const int e = (int)(item - items);
      if (tid < 32) {
        const int4 inf = p.bnd_info[2 * e];
        const int* table = p.page_table + (size_t)inf.y * p.cap;
        int ksh = 0;
        for (int j = tid; j < inf.z - p.sub; j += 32) ksh += (p.refcount[table[j]] > 1);
#pragma unroll
        for (int o2 = 16; o2 > 0; o2 >>= 1) ksh += __shfl_xor_sync(0xffffffffu, ksh, o2);
        if (tid == 0) p.bnd_acc[4 * e + 2] = ksh;
      }
      continue;
    }
    const long long u = item / NT;
    const int job = (int)(item % NT);               // 0: K^S, 1: K^L, 2: eviction list, 3: a Shrink's eviction list
    const int task = job < 2 ? job : 2;
    const int ne = (SHR && job == 3) ? 2 * p.blk : p.blk;        // slots a compression (a Shrink) frees
    const int bidx = (int)(u / LH), lh = (int)(u % LH);
    const int l = lh / p.Hkv, h = lh % p.Hkv;
    const bool is_first = item == (long long)blockIdx.x;
    const int4 inf = is_first ? inf_first : p.bnd_info[2 * bidx];          // {slot in the batch, request, P}
    const int4 inf2 = is_first ? inf2_first : p.bnd_info[2 * bidx + 1];    // {offset into the logit scratch}
    const int r = inf.y, Pr = inf.z;
    const long long off = (long long)(unsigned)inf2.x | ((long long)inf2.y << 32);
    // two supports (they coincide when the page is 16 tokens): the working sets of Eq. 7 leave out the newest page
    // of the method, the eviction candidates of Eq. 10 only the protected window, the newest 16-token tile
    const int nC_d = (Pr - p.sub) * GP_PAGE, nC_e = (Pr - 1) * GP_PAGE;
    const int nC = task < 2 ? nC_d : nC_e;
    int* Kout = p.Kx + (((size_t)r * p.L + l) * p.Hkv + h) * 2;
    int* evout = (SHR && job == 3) ? p.evict2 + (size_t)u * 2 * p.blk : p.evict + (size_t)u * p.blk;
    __syncthreads();
    if (nC_d == 0) {                         // one page of the method: nothing to estimate from, nothing to evict
      if (tid == 0 && task < 2) Kout[task] = 0;
      continue;
    }
    if (SHR && job == 3 && Pr - p.sub < p.min_pages_after_shrink) continue;      // this boundary cannot be a Shrink
    const size_t view_stride = (size_t)p.z_stride * G;
    const double* z = p.zbuf + (size_t)lh * 2 * view_stride + (size_t)off * G;   // [2 views][nC][G] exp(logit - page max)
    const double* zs = p.zstat + ((size_t)lh * (p.max_boundary_tokens / GP_PAGE) + off / GP_PAGE) * G2 * 2;
    double* a = nC <= SEL_CAP ? S.sbuf : p.scores + ((size_t)job * LH + lh) * p.max_boundary_tokens + off;
    sel_job(p, S, z, view_stride, zs, a, nC, task, ne, Kout, p.bnd_acc + 4 * bidx, evout,
              p.Hx + (((size_t)r * p.L + l) * p.Hkv + h) * 2);
  }

  // ---- the last CTA takes the decisions ----------------------------------------------------------------------
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    const int prev = atomicAdd(&p.hdr[HDR_DONE_SEL], 1);
    s_i[2] = (prev == (int)gridDim.x - 1);
    if (prev == (int)gridDim.x - 1) p.hdr[HDR_DONE_SEL] = 0;
  }
  __syncthreads();
  if (s_i[2]) {
    __threadfence();
    if (!out) advance_counters(p, n_rc);
    if (decide) decide_and_allocate(p, req_ids, n_req, n_bnd, actions, reinterpret_cast<int*>(S.sbuf), serial);
    else publish_shard_sums(p, n_bnd);
  }

  if (!idle_merge) merge_partials(p, n_req, out, n_mc, n_rc, (int)gridDim.x - 1 - (int)blockIdx.x, (int)gridDim.x, 0, LH);
}

// merges the partial outputs of the split requests for the units [lh0, lh0 + lh_n): the per-layer entry point
// needs a layer's output complete before the next layer's query exists
__global__ void __launch_bounds__(256)
gp_merge_kernel(const __grid_constant__ GpDev p, int n_req, float* __restrict__ out, int lh0, int lh_n) {
  // the kernel after this one may be scheduled at once: it waits for this grid's end where it needs to, and this
  // grid ends after the attention kernel (the wait below), so completion stays transitive
  gp_pdl_launch_dependents();
  gp_pdl_wait();
  merge_partials(p, n_req, out, p.hdr[HDR_N_MC], p.hdr[HDR_N_RC], (int)blockIdx.x, (int)gridDim.x, lh0, lh_n);
}

// ------------------------------------------------------------------------------------------------------
// compaction
// ------------------------------------------------------------------------------------------------------
// shared memory of the compaction
struct CmpSmem {
  int4* s_info;      // [GP_MAX_REQ + 1] compressing requests: {request, P, boundary index, first chunk}
  int* ev;           // [2 * GP_MAX_BLK] slots the unit's compression (or Shrink) evicts
  int* s_i;          // [8]
  int* s_dst;        // [MOVE_TOK] per source slot of the chunk: destination slot (-1: stays or goes)
  int* s_spage;      // [MOVE_TOK] source page
  int* s_dpage;      // [MOVE_TOK] destination page
};
constexpr size_t CMP_SMEM_BYTES = (GP_MAX_REQ + 1) * 16 + (2 * GP_MAX_BLK + 8 + 3 * MOVE_TOK) * 4;
__device__ __forceinline__ CmpSmem cmp_smem_at(uint8_t* base) {       // base: 16-byte aligned, CMP_SMEM_BYTES
  CmpSmem C;
  C.s_info = reinterpret_cast<int4*>(base);
  C.ev = reinterpret_cast<int*>(base + (GP_MAX_REQ + 1) * 16);
  C.s_i = C.ev + 2 * GP_MAX_BLK;
  C.s_dst = C.s_i + 8;
  C.s_spage = C.s_dst + MOVE_TOK;
  C.s_dpage = C.s_spage + MOVE_TOK;
  return C;
}

// The compaction of a step, run by every CTA of the calling grid (CT threads): work is claimed from the ticket
// counter until none is left; the last CTA to finish swaps in the copy-on-write targets.  What a ticket stands for
// depends on how much there is.  A few units (one layer, a handful of requests at their boundary): one 64-slot chunk
// of a unit per ticket, so that all thread blocks have work; a chunk says when its sources are read, and waits for
// that word from the chunks before it whose sources its destinations reach.  Units for every thread block twice
// over: one unit per ticket, its chunks in ascending order by the same thread block (a chunk's destinations lie
// below the next chunk's sources, and program order puts every chunk's reads before the next chunk's writes), which
// saves the ticket, the eviction list and the waits per chunk and skips the chunks below the first evicted slot.
template <int D, bool SHR>
__device__ __forceinline__ void compact_body(const GpDev& p, const CmpSmem& C, int serial) {
  constexpr int CH = D / 8;
  constexpr int ROW_BYTES = D * 2;
  constexpr int PIECES = MOVE_TOK * 2 * CH / CT;        // 16-byte pieces per thread per chunk
  int4* s_info = C.s_info;
  int* ev = C.ev;
  int* s_i = C.s_i;
  int* s_dst = C.s_dst;
  int* s_spage = C.s_spage;
  int* s_dpage = C.s_dpage;

  const int tid = threadIdx.x, lane = tid & 31;
  const int LH = p.L * p.Hkv;
  // the first round trip fetches everything at once: the header, the list of compressing requests (its first
  // CT entries before their count is known; entries past the count are never looked at) and the first ticket
  if (tid == 0) { s_i[0] = atomicAdd(&p.hdr[HDR_WORK_CMP], 1); s_i[3] = 0; }
  if (tid <= p.M) s_info[tid] = p.cmp_info[tid];
  const int n_cmp = p.hdr[HDR_N_CMP];
  const int n_items = p.hdr[HDR_N_CITEM];
  const int n_cow = p.hdr[HDR_N_COW];
  // unique per decode step of the pool (the chunk flags are never cleared): the host's step count in the
  // asynchronous mode, where the two scratch sets count on their own; otherwise the counter the plan kernel keeps
  // on the device, so that a step replayed from a CUDA graph gets a stamp of its own
  const int stamp = p.async ? serial + 1 : p.hdr[HDR_STEP];
  for (int i = tid + CT; i <= n_cmp; i += CT) s_info[i] = p.cmp_info[i];

  const bool by_unit = (p.withhold & GP_TEST_COMPACT_BY_UNIT) || (long long)n_cmp * LH >= 2LL * (long long)gridDim.x;
  const int n_work = by_unit ? n_cmp * LH : n_items;
  for (bool first = true;; first = false) {
    __syncthreads();
    if (!first) {
      if (tid == 0) s_i[0] = atomicAdd(&p.hdr[HDR_WORK_CMP], 1);
      __syncthreads();
    }
    const int item = s_i[0];
    if (item >= n_work) break;
    // ticket -> (compressing request, layer/head) and the chunks it covers; chunks of a unit are consecutive and
    // ascending in the item numbering the flags go by
    int lo, lh, j_begin, j_end;
    if (by_unit) {
      lo = item / LH; lh = item % LH;
      j_begin = 0; j_end = s_info[lo + 1].w - s_info[lo].w;
    } else {
      lo = 0;
      int hi = n_cmp;
      while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (LH * s_info[mid].w <= item) lo = mid; else hi = mid; }
      const int nchunk = s_info[lo + 1].w - s_info[lo].w;
      const int rem = item - LH * s_info[lo].w;
      lh = rem / nchunk; j_begin = rem % nchunk; j_end = j_begin + 1;
    }
    const int4 inf = s_info[lo];
    const int l = lh / p.Hkv, h = lh % p.Hkv;
    const int r = inf.x;
    const int Pr = inf.y;
    const int* table = p.page_table + (size_t)r * p.cap;
    const int* shadow = p.shadow + (size_t)r * p.cap;
    const int n_src = Pr * GP_PAGE;
    // second round trip: the eviction list and, for every source slot of the chunk, its page and its
    // copy-on-write target
    const bool shrink = SHR && (inf.z & CMP_SHRINK) != 0;
    const int e_bnd = inf.z & (CMP_SHRINK - 1);
    const int ne = shrink ? 2 * p.blk : p.blk;             // slots freed: one page of the method, two at a Shrink
    for (int t = tid; t < ne; t += CT)
      ev[t] = shrink ? p.evict2[((size_t)e_bnd * LH + lh) * 2 * p.blk + t] : p.evict[((size_t)e_bnd * LH + lh) * p.blk + t];
    if (by_unit && n_cow == 0) {
      // nothing is shared in this step: slots below the first evicted one stay where they are
      __syncthreads();
      if (tid < 32) {
        int mn = 0x7fffffff;
        for (int t = tid; t < ne; t += 32) mn = min(mn, ev[t]);
#pragma unroll
        for (int o2 = 16; o2 > 0; o2 >>= 1) mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, o2));
        if (tid == 0) s_i[5] = mn / MOVE_TOK;
      }
      __syncthreads();
      j_begin = s_i[5];
    }
   for (int j = j_begin; j < j_end; ++j) {
    if (j != j_begin) __syncthreads();                   // the chunk before has left the shared arrays
    const int c0 = j * MOVE_TOK;
    int t0 = 0, s0 = -1;
    const int my_i = c0 + tid;                             // the slot this thread plans (first MOVE_TOK threads)
    if (tid < MOVE_TOK && my_i < n_src) {
      const int pg = my_i / GP_PAGE;
      t0 = table[pg]; s0 = shadow[pg];
    }
    __syncthreads();
    int tokv = 0, tok_dst = -1, tok_page = 0;
    if (tid < MOVE_TOK) {
      int ds = -1, dpage = 0;
      if (my_i < n_src) {
        int sh = 0; bool evicted = false;
        if (ne == GP_PAGE) {
#pragma unroll
          for (int e2 = 0; e2 < GP_PAGE; ++e2) { sh += (ev[e2] < my_i); evicted |= (ev[e2] == my_i); }
        } else {
          for (int e2 = 0; e2 < ne; ++e2) { sh += (ev[e2] < my_i); evicted |= (ev[e2] == my_i); }
        }
        const int pg = my_i / GP_PAGE;
        const bool cow = (pg < Pr - 1) && (s0 >= 0);
        if (!evicted && (sh > 0 || cow)) {
          ds = my_i - sh;
          // the destination tile: as many tiles down as evicted slots lie before this one (third round trip,
          // from the L2, only for slots that move across a tile boundary)
          const int dpg = ds / GP_PAGE;
          if (dpg == pg) dpage = s0 >= 0 ? s0 : t0;
          else { const int sd = shadow[dpg]; dpage = sd >= 0 ? sd : table[dpg]; }
          tokv = p.tok[gp_tok_off(p, l, t0, h) + (my_i % GP_PAGE)];
          tok_dst = ds; tok_page = dpage;
        }
      }
      s_dst[tid] = ds; s_spage[tid] = t0; s_dpage[tid] = dpage;
    }
    __syncthreads();

    // A thread's pieces of a chunk: piece k2 belongs to slot tl0 + k2 * TLS of the chunk, and is the same 16 bytes of
    // its row every time (K or V, physical piece cp); a page's tile of this unit lies page_stride bytes after the
    // one of the page before.
    constexpr int PPS = 2 * CH, TLS = CT / PPS;
    const int tl0 = tid / PPS, isv = (tid % PPS) / CH, cp = tid % CH;
    uint8_t* const unit_base = reinterpret_cast<uint8_t*>(p.kv + gp_tile_off(p, l, 0, h)) + isv * GP_PAGE * ROW_BYTES;
    const size_t page_stride = (size_t)p.Hkv * 2 * GP_PAGE * ROW_BYTES;
    uint4 val[PIECES];
#pragma unroll
    for (int k2 = 0; k2 < PIECES; ++k2) {
      const int tl = tl0 + k2 * TLS;
      val[k2] = make_uint4(0, 0, 0, 0);
      if (s_dst[tl] >= 0)
        val[k2] = *reinterpret_cast<const uint4*>(unit_base + (size_t)s_spage[tl] * page_stride +
                                                  ((c0 + tl) % GP_PAGE) * ROW_BYTES + (cp << 4));
    }
    // Touch every loaded value so that the loads have completed before the flag below is published: the
    // next chunk's CTA may overwrite the tail of this chunk's sources as soon as it sees the flag.
    unsigned touched = (unsigned)tokv;
#pragma unroll
    for (int k2 = 0; k2 < PIECES; ++k2) touched ^= val[k2].x ^ val[k2].y ^ val[k2].z ^ val[k2].w;
    if (touched == 0x9e3779b9u && c0 < 0) s_i[4] = 1;      // never true; keeps the dependency alive
    __syncthreads();
    if (tid == 0 && !by_unit) {
      // No fence on either side: the flag only says that loads have returned (they have: their values were
      // consumed above), and the stores below are issued after the flag has been seen.
      if (!((p.withhold & GP_WITHHOLD_CHUNK) && j == 0))               // (test support: see GP_WITHHOLD_CHUNK)
        *reinterpret_cast<volatile int*>(p.cflags + item) = stamp;      // "my sources are read"
      // my destinations reach back as far as a slot can move down, `ne` slots: into the sources of the chunks
      // before this one, all of which must have been read (tickets are handed out in order, so those chunks are
      // running or done)
      const int reach = (ne + MOVE_TOK - 1) / MOVE_TOK;
      for (int back = 1; back <= reach && back <= j; ++back) {
        volatile int* prev = reinterpret_cast<volatile int*>(p.cflags + item - back);
        unsigned it = 0;
        while (*prev != stamp && it < p.spin_limit) ++it;
        if (it >= p.spin_limit) atomicOr(p.err, GP_E_SPIN_CMP);
      }
    }
    __syncthreads();
#pragma unroll
    for (int k2 = 0; k2 < PIECES; ++k2) {
      const int tl = tl0 + k2 * TLS;
      const int ds = s_dst[tl];
      if (ds >= 0) {
        const int c = cp ^ ((c0 + tl) & 7);                 // the logical piece this thread holds (rows are swizzled by slot)
        *reinterpret_cast<uint4*>(unit_base + (size_t)s_dpage[tl] * page_stride + (ds % GP_PAGE) * ROW_BYTES +
                                  ((c ^ (ds & 7)) << 4)) = val[k2];
      }
    }
    if (tok_dst >= 0) {
      atomicAdd(&s_i[3], 1);
      p.tok[gp_tok_off(p, l, tok_page, h) + (tok_dst % GP_PAGE)] = tokv;
    }
   }
  }
  __syncthreads();
  if (tid == 0 && s_i[3] > 0)
    atomicAdd(reinterpret_cast<unsigned long long*>(p.counters + 8), (unsigned long long)s_i[3]);

  // ---- the last CTA swaps in the copy-on-write targets and drops the old references (App. D.2), and hands
  // back the last page of every request that shrank (Eq. 13) ---------------------------------------------
  if (n_cow == 0) return;                                 // nothing was shared and nobody shrank
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int prev = atomicAdd(&p.hdr[HDR_DONE_CMP], 1);
    s_i[2] = (prev == (int)gridDim.x - 1);
    if (prev == (int)gridDim.x - 1) p.hdr[HDR_DONE_CMP] = 0;
  }
  __syncthreads();
  if (s_i[2] && tid < 32) {
    __threadfence();
    for (int ci = 0; ci < n_cmp; ++ci) {
      const int r = s_info[ci].x;
      const int Pr = s_info[ci].y;
      int* table = p.page_table + (size_t)r * p.cap;
      int* shadow = p.shadow + (size_t)r * p.cap;
      for (int j0 = 0; j0 < Pr - 1; j0 += 32) {
        const int j = j0 + lane;
        bool freed = false;
        int old = -1;
        if (j < Pr - 1 && shadow[j] >= 0) {
          old = table[j];
          table[j] = shadow[j];
          shadow[j] = -1;
          freed = (atomicSub(&p.refcount[old], 1) == 1);
        }
        const unsigned mask = __ballot_sync(0xffffffffu, freed);
        int base = 0;
        if (lane == 0) base = *reinterpret_cast<volatile int*>(p.free_top);
        base = __shfl_sync(0xffffffffu, base, 0);
        if (freed) p.free_stack[base + __popc(mask & ((1u << lane) - 1u))] = old;
        __syncwarp();
        if (lane == 0 && mask) *reinterpret_cast<volatile int*>(p.free_top) = base + __popc(mask);
        __syncwarp();
      }
      if (SHR && (s_info[ci].z & CMP_SHRINK) && lane == 0) {      // the page of the method the request no longer owns
        for (int t = p.sub; t >= 1; --t) {
          const int last = table[Pr - t];
          if (atomicSub(&p.refcount[last], 1) == 1) {
            const int top = *reinterpret_cast<volatile int*>(p.free_top);
            p.free_stack[top] = last;
            *reinterpret_cast<volatile int*>(p.free_top) = top + 1;
          }
        }
      }
      __syncwarp();
    }
  }
}


template <int D, bool SHR>
__global__ void __launch_bounds__(CT, 4)
gp_compact_kernel(const __grid_constant__ GpDev p, const int* __restrict__ req_ids, int n_req, int serial) {
  __shared__ __align__(16) uint8_t cmp_raw[CMP_SMEM_BYTES];
  gp_pdl_wait();
  gp_pdl_launch_dependents();
  compact_body<D, SHR>(p, cmp_smem_at(cmp_raw), serial);
}

// ------------------------------------------------------------------------------------------------------
// asynchronous boundary mode: the whole boundary chain of a step in one kernel, beside the next step's attention
// ------------------------------------------------------------------------------------------------------
// Launched right behind the attention kernel of step t + 1 as its programmatic dependent, this grid works on the
// boundary chain of step t: it does not wait for that attention kernel before it starts (everything it reads
// was complete before that kernel could start), runs the selection jobs, lets the last CTA to finish them
// decide and allocate, waits inside the grid for that (a bounded wait on a flag: the grid is sized to be
// resident at once, on the room the attention kernel leaves), compacts, and only then waits for the attention
// kernel to end; after that it merges the split requests' partial outputs of step t + 1.  The grid therefore
// ends after both, and the plan of step t + 2, its programmatic dependent, finds the pages and counters of the
// requests that sat step t + 1 out in their final state.  `p`: the view of step t (its scratch set, the copy of
// the counters its decisions go to); `pa`: the view of step t + 1 (for the merge).
template <int D, bool SHR>
__global__ void __launch_bounds__(SEL_T, 2)
gp_chain_kernel(const __grid_constant__ GpDev p, const __grid_constant__ GpDev pa, int n_req_merge, float* __restrict__ out_merge,
                int serial, int has_chain, const int* __restrict__ req_ids, int* __restrict__ actions,
                int* __restrict__ actions_copy) {
  // actions_copy: where the step's actions are wanted as well once they are final (the host entry points: the
  // caller's array in page-locked host memory; writing them there from the plan kernel made that kernel wait
  // for the bus)
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((256u - (smem_u32(smem_raw) & 255u)) & 255u);
  const int tid = threadIdx.x;
  const int LH = p.L * p.Hkv;
  // Synchronous mode (same_step): the chain belongs to the step whose attention kernel runs beside this grid.
  // A selection job then waits until the consumer warps of that kernel have reported the unit's summary logits
  // complete (the requests at their boundary come first in its deal), the decisions are reported through
  // `actions` as usual, and the next kernel on the stream may only be scheduled once the attention kernel has
  // ended (its early part reads counters that kernel advances).
  const bool same_step = !p.async;
  if (!same_step) gp_pdl_launch_dependents();
  if (has_chain) {
    SelSmem S = sel_smem_at(smem);
    int* s_i = S.s_i;
    const int G = p.G, G2 = 2 * p.G;
    constexpr int NT = SHR ? 4 : 3;
    const int n_bnd = __ldcg(p.hdr + HDR_N_BND);
    const long long items = (long long)n_bnd * LH * NT;
    for (long long item = blockIdx.x; item < items + n_bnd; item += gridDim.x) {
      if (item >= items) {
        const int e = (int)(item - items);
        if (tid < 32) {
          const int4 inf = p.bnd_info[2 * e];
          const int* table = p.page_table + (size_t)inf.y * p.cap;
          int ksh = 0;
          for (int j = tid; j < inf.z - p.sub; j += 32) ksh += (p.refcount[table[j]] > 1);
#pragma unroll
          for (int o2 = 16; o2 > 0; o2 >>= 1) ksh += __shfl_xor_sync(0xffffffffu, ksh, o2);
          if (tid == 0) p.bnd_acc[4 * e + 2] = ksh;
        }
        continue;
      }
      const long long u = item / NT;
      const int job = (int)(item % NT);
      const int task = job < 2 ? job : 2;
      const int ne = (SHR && job == 3) ? 2 * p.blk : p.blk;        // slots a compression (a Shrink) frees
      const int bidx = (int)(u / LH), lh = (int)(u % LH);
      const int l = lh / p.Hkv, h = lh % p.Hkv;
      const int4 inf = p.bnd_info[2 * bidx];
      const int4 inf2 = p.bnd_info[2 * bidx + 1];
      const int r = inf.y, Pr = inf.z;
      const long long off = (long long)(unsigned)inf2.x | ((long long)inf2.y << 32);
      // two supports (they coincide when the page is 16 tokens): the working sets of Eq. 7 leave out the newest page
    // of the method, the eviction candidates of Eq. 10 only the protected window, the newest 16-token tile
    const int nC_d = (Pr - p.sub) * GP_PAGE, nC_e = (Pr - 1) * GP_PAGE;
    const int nC = task < 2 ? nC_d : nC_e;
      int* Kout = p.Kx + (((size_t)r * p.L + l) * p.Hkv + h) * 2;
      int* evout = (SHR && job == 3) ? p.evict2 + (size_t)u * 2 * p.blk : p.evict + (size_t)u * p.blk;
      __syncthreads();
      if (nC_d == 0) {                         // one page of the method: nothing to estimate from, nothing to evict
        if (tid == 0 && task < 2) Kout[task] = 0;
        continue;
      }
      if (SHR && job == 3 && Pr - p.sub < p.min_pages_after_shrink) continue;
      if (same_step) {
        // every work item of the request reports once per consumer warp for this unit (bounded wait; the
        // attention kernel's thread blocks were all resident before this grid could be scheduled)
        if (tid == 0) {
          const volatile int* rdy = p.unit_ready + (size_t)bidx * LH + lh;
          unsigned it = 0;
          while (*rdy < inf2.z && it < p.spin_limit) { ++it; __nanosleep(200); }
          if (it >= p.spin_limit) atomicOr(p.err, GP_E_SPIN_SEL);
          __threadfence();
        }
        __syncthreads();
      }
      const size_t view_stride = (size_t)p.z_stride * G;
      const double* z = p.zbuf + (size_t)lh * 2 * view_stride + (size_t)off * G;
      const double* zs = p.zstat + ((size_t)lh * (p.max_boundary_tokens / GP_PAGE) + off / GP_PAGE) * G2 * 2;
      double* a = nC <= SEL_CAP ? S.sbuf : p.scores + ((size_t)job * LH + lh) * p.max_boundary_tokens + off;
      sel_job(p, S, z, view_stride, zs, a, nC, task, ne, Kout, p.bnd_acc + 4 * bidx, evout,
              p.Hx + (((size_t)r * p.L + l) * p.Hkv + h) * 2);
    }
    // ---- the last CTA to finish its jobs takes the decisions and tells the others ------------------------------
    const int stamp = same_step ? p.hdr[HDR_STEP] : serial + 1;
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      const int prev = atomicAdd(&p.hdr[HDR_DONE_SEL], 1);
      s_i[2] = (prev == (int)gridDim.x - 1);
      if (prev == (int)gridDim.x - 1) p.hdr[HDR_DONE_SEL] = 0;
    }
    __syncthreads();
    if (s_i[2]) {
      __threadfence();
      decide_and_allocate(p, req_ids, n_req_merge, n_bnd, same_step ? actions : nullptr, reinterpret_cast<int*>(S.sbuf), serial);
      __syncthreads();
      if (tid == 0 && !(p.withhold & GP_WITHHOLD_DECIDED)) {      // (test support: see GP_WITHHOLD_DECIDED)
        __threadfence();
        *reinterpret_cast<volatile int*>(p.hdr + HDR_DECIDED) = stamp;
      }
    } else if (tid == 0) {
      volatile int* flag = reinterpret_cast<volatile int*>(p.hdr + HDR_DECIDED);
      unsigned it = 0;
      while (*flag != stamp && it < p.spin_limit) { ++it; __nanosleep(100); }
      if (it >= p.spin_limit) atomicOr(p.err, GP_E_SPIN_CMP);
      __threadfence();
    }
    __syncthreads();
    if (same_step) {
      // The attention kernel of this step has ended by now (the decisions needed its last reports): the split
      // requests' outputs are merged first, and then the next kernel on the stream may be scheduled.  With early
      // planning that is the next step's plan, which so runs beside the compaction below: the decisions it reads
      // are taken, the attention kernel has moved the requests on, and the compaction reads nothing the plan writes
      // (the merge does: the lists of split requests, hence its place before).
      gp_pdl_wait();
      if (actions_copy && blockIdx.x == gridDim.x - 1)
        for (int i = tid; i < n_req_merge; i += SEL_T) actions_copy[i] = __ldcg(actions + i);
      if (out_merge) merge_partials(pa, n_req_merge, out_merge, pa.hdr[HDR_N_MC], pa.hdr[HDR_N_RC], (int)blockIdx.x, (int)gridDim.x, 0, LH);
      gp_pdl_launch_dependents();
    }
    // ---- compaction: its arrays take the place of the selection's -----------------------------------------------
    compact_body<D, SHR>(p, cmp_smem_at(smem), serial);
  }
  if (same_step) return;
  gp_pdl_wait();              // the attention kernel beside which this grid ran has ended
  if (out_merge) merge_partials(pa, n_req_merge, out_merge, pa.hdr[HDR_N_MC], pa.hdr[HDR_N_RC], (int)blockIdx.x, (int)gridDim.x, 0, LH);
}

// the decisions of a step whose sums of K^S and K^L were completed outside (KV heads spread over several pools)
__global__ void __launch_bounds__(SEL_T)
gp_decide_kernel(const __grid_constant__ GpDev p, const int* __restrict__ req_ids, int n_req, int* __restrict__ actions,
                 int serial) {
  __shared__ int s_arr[8 * GP_MAX_REQ];
  decide_and_allocate(p, req_ids, n_req, __ldcg(p.hdr + HDR_N_BND), actions, s_arr, serial, true);
}

}  // namespace

// the compaction kernel of a pool: head dimension, and whether the Shrink policy is on
static auto compact_kernel_of(const GpDev& p) -> void (*)(const GpDev, const int*, int, int) {
  const bool shr = p.policy == GP_POLICY_SHRINK;
  if (p.d == 128) return shr ? gp_compact_kernel<128, true> : gp_compact_kernel<128, false>;
  return shr ? gp_compact_kernel<64, true> : gp_compact_kernel<64, false>;
}

// shared memory of the selection kernel for a per-request page cap (its bitmap of block-local picks has one bit
// per candidate token)
size_t gp_bsel_smem_for_cap(long long cap) {
  return SelGeom::BUF_BYTES + SelGeom::H_BYTES + SelGeom::MISC_BYTES + ((size_t)cap * GP_PAGE / 32 + 2) * 4 + 512;
}
size_t gp_bsel_smem(const GpDev& p) { return gp_bsel_smem_for_cap(p.cap); }

// one-time setup for a pool: opts the selection kernel into its shared memory and sizes both grids to
// exactly one resident wave, so that no CTA waits for another to leave before it can start
void gp_boundary_setup(const GpDev& p, int num_sms, int* grid_sel, int* grid_compact) {
  const size_t sel_sm = gp_bsel_smem(p);
  const bool shr = p.policy == GP_POLICY_SHRINK;
  auto sel = shr ? gp_bsel_kernel<true> : gp_bsel_kernel<false>;
  cudaFuncSetAttribute(sel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sel_sm);
  {                                                  // the kernel with the whole boundary chain: same shared memory
    auto opt_in = [&](auto kern) { cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sel_sm); };
    if (p.d == 128) { if (shr) opt_in(gp_chain_kernel<128, true>); else opt_in(gp_chain_kernel<128, false>); }
    else { if (shr) opt_in(gp_chain_kernel<64, true>); else opt_in(gp_chain_kernel<64, false>); }
  }
  int occ = 0;
  cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, sel, SEL_T, sel_sm);
  *grid_sel = num_sms * (occ > 0 ? occ : 1);
  occ = 0;
  cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, compact_kernel_of(p), CT, 0);
  *grid_compact = num_sms * (occ > 0 ? occ : 1);
}

// asynchronous mode: the boundary chain of the step whose view is `p` (none when !has_chain), and afterwards the
// merge of the split requests' partial outputs of the step whose view is `pa` (none when out_merge is null)
void gp_launch_chain(const GpDev& p, const GpDev& pa, int n_req_merge, float* out_merge, int serial, int has_chain, int grid,
                     cudaStream_t s, bool pdl, const int* req_ids, int* actions, int* actions_copy) {
  const size_t sm = gp_bsel_smem(p);
  const bool shr = p.policy == GP_POLICY_SHRINK;
  auto launch = [&](auto kern) {
    gp_launch(kern, grid, SEL_T, sm, s, pdl, p, pa, n_req_merge, out_merge, serial, has_chain, req_ids, actions, actions_copy);
  };
  if (p.d == 128) { if (shr) launch(gp_chain_kernel<128, true>); else launch(gp_chain_kernel<128, false>); }
  else { if (shr) launch(gp_chain_kernel<64, true>); else launch(gp_chain_kernel<64, false>); }
}

void gp_launch_select_only(const GpDev& p, const int* req_ids, int n_req, int* actions, float* out, int grid_sel, cudaStream_t s,
                           bool pdl, int serial) {
  const size_t sel_sm = gp_bsel_smem(p);
  const bool shr = p.policy == GP_POLICY_SHRINK;
  gp_launch(shr ? gp_bsel_kernel<true> : gp_bsel_kernel<false>, grid_sel, SEL_T, sel_sm, s, pdl, p, req_ids, n_req, actions, out,
            serial, 0);
}

// plain launches: what comes before them on the stream (the caller's reduction of the sums) is not this library's
void gp_launch_decide_compact(const GpDev& p, const int* req_ids, int n_req, int* actions, int grid_compact, cudaStream_t s,
                              int serial) {
  gp_launch(gp_decide_kernel, 1, SEL_T, 0, s, false, p, req_ids, n_req, actions, serial);
  gp_launch(compact_kernel_of(p), grid_compact, CT, 0, s, true, p, req_ids, n_req, serial);
}

void gp_launch_merge(const GpDev& p, int n_req, float* out, int lh0, int lh_n, int grid, cudaStream_t s, bool pdl) {
  gp_launch(gp_merge_kernel, grid, 256, 0, s, pdl, p, n_req, out, lh0, lh_n);
}

void gp_launch_boundary(const GpDev& p, const int* req_ids, int n_req, int* actions, float* out, int grid_sel,
                        int grid_compact, cudaStream_t s, cudaEvent_t ev, bool pdl, int serial) {
  const size_t sel_sm = gp_bsel_smem(p);
  const bool shr = p.policy == GP_POLICY_SHRINK;
  // asynchronous mode: the kernel before this one on its stream belongs to another step (an event wait lies in
  // between): plain launch; the compaction kernel follows as a programmatic dependent as usual
  gp_launch(shr ? gp_bsel_kernel<true> : gp_bsel_kernel<false>, grid_sel, SEL_T, sel_sm, s, pdl && !p.async, p, req_ids,
            n_req, actions, out, serial, 1);
  if (ev) cudaEventRecord(ev, s);
  gp_launch(compact_kernel_of(p), grid_compact, CT, 0, s, pdl, p, req_ids, n_req, serial);
}
