// Capacity-boundary kernels (Sec. 3.2 - 3.3, App. D.1, App. D.2).
//
// gp_score_kernel   one CTA per (request at a boundary, layer, KV head):
//                   Eq. 12 calibration (+ RoPE at the current position), summary-induced attention
//                   a^S, a^L over the candidate set C (everything but the newest page), and the
//                   working-set sizes K^S, K^L of Eq. 7.  All in fp64: these values decide integer
//                   outcomes (set sizes, the retained set, grow or compress), which are compared
//                   bit for bit with a float64 reference.
// gp_compact_kernel one CTA per (compressing request, layer, KV head):
//                   Eq. 9 scores, Eq. 10 block-local + global selection, then the stable in-place
//                   compaction into (P-1) b slots, writing to copy-on-write targets where the source
//                   page is shared.  The last CTA to finish swaps in the target pages and drops the
//                   references to the replaced ones.
//
// Top-p counting and top-k selection are radix descents over the IEEE bit patterns of the
// (non-negative) scores: 11 bits per level, counts in shared-memory histograms.  The top-p mass is
// accumulated in 2^62 fixed point with integer atomics, so the result does not depend on the order
// in which threads add.
#include "gp_dev.cuh"

namespace {

constexpr int BT = 256;              // threads per CTA
constexpr int NBINS = 2048;
constexpr double TWO62 = 4611686018427387904.0;

__device__ __forceinline__ unsigned long long to_fix(double a) {
  return (unsigned long long)__double2ll_rn(a * TWO62);
}

struct PairCU { unsigned c; unsigned long long s; };

// exclusive suffix sum over the block: result = sum of the values of threads with a higher id
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

// Eq. 7: smallest k such that the k largest of a[0..n) sum to at least p.
__device__ int top_p_count(const double* __restrict__ a, int n, unsigned long long p_fix, unsigned* hcnt,
                           unsigned long long* hsum, unsigned* wc, unsigned long long* wsum, long long* s_res) {
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
    for (int i = tid; i < nb; i += BT) { hcnt[i] = 0; hsum[i] = 0; }
    if (tid == 0) s_res[0] = -1;
    __syncthreads();
    for (int i = tid; i < n; i += BT) {
      const double v = __ldcg(a + i);
      const unsigned long long key = (unsigned long long)__double_as_longlong(v);
      if (lvl == 0 || (key >> (shift + w)) == prefix) {
        const int bin = (int)((key >> shift) & (unsigned long long)(nb - 1));
        atomicAdd(&hcnt[bin], 1u);
        atomicAdd(&hsum[bin], to_fix(v));
      }
    }
    __syncthreads();
    const int per = nb / BT > 0 ? nb / BT : 1;
    const int lo = tid * per, hi = lo + per;     // this thread's bins [lo, hi)
    unsigned c = 0; unsigned long long s = 0;
    if (lo < nb) for (int b = lo; b < hi; ++b) { c += hcnt[b]; s += hsum[b]; }
    PairCU ex = block_suffix_excl(c, s, wc, wsum);
    if (lo < nb) {
      unsigned long long run_s = sum_above + ex.s;
      unsigned run_c = cnt_above + ex.c;
      for (int b = hi - 1; b >= lo; --b) {
        const unsigned long long before = run_s;
        run_s += hsum[b];
        if (before < p_fix && run_s >= p_fix) { s_res[0] = b; s_res[1] = run_c; s_res[2] = (long long)before; }
        run_c += hcnt[b];
      }
    }
    __syncthreads();
    if (s_res[0] < 0) return n;                  // rounding kept the total below p: everything
    bin_star = (int)s_res[0];
    cnt_above = (unsigned)s_res[1];
    sum_above = (unsigned long long)s_res[2];
    const unsigned cstar = hcnt[bin_star];
    __syncthreads();
    if (cstar == 1) return (int)cnt_above + 1;
    prefix = (prefix << w) | (unsigned long long)bin_star;
  }
  // all bits fixed: the bin holds copies of one value
  const unsigned c = hcnt[bin_star];
  const unsigned long long f = hsum[bin_star] / c;
  unsigned long long j = (p_fix - sum_above + f - 1) / f;
  if (j < 1) j = 1;
  if (j > c) j = c;
  __syncthreads();
  return (int)cnt_above + (int)j;
}

template <int D>
struct ScoreGeom {
  static constexpr int CH = D / 8;
  static constexpr int TILE_TOK = 128;
  static constexpr size_t QT_BYTES = 2 * 8 * D * sizeof(double);
  static constexpr size_t KT_BYTES = TILE_TOK * D * 2;
  static constexpr size_t H_BYTES = NBINS * 4 + NBINS * 8;
  static constexpr size_t RED_BYTES = (BT + 64) * 8 + 64 * 8;
  static constexpr size_t SMEM = QT_BYTES + KT_BYTES + H_BYTES + RED_BYTES + 256;
};

template <int D>
__global__ void __launch_bounds__(BT)
gp_score_kernel(const __grid_constant__ GpDev p, const int* __restrict__ req_ids, int n_req,
                const __nv_bfloat16* __restrict__ q) {
  using GEO = ScoreGeom<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((256u - (smem_u32(smem_raw) & 255u)) & 255u);
  double* qt = reinterpret_cast<double*>(smem);                               // [2][8][D]
  uint4* ktile = reinterpret_cast<uint4*>(smem + GEO::QT_BYTES);              // [128][CH]
  unsigned* hcnt = reinterpret_cast<unsigned*>(smem + GEO::QT_BYTES + GEO::KT_BYTES);
  unsigned long long* hsum = reinterpret_cast<unsigned long long*>(hcnt + NBINS);
  double* red = reinterpret_cast<double*>(hsum + NBINS);                      // [BT]
  double* sM = red + BT;                                                      // [16] maxima
  double* sZ = sM + 16;                                                       // [16] normalisers
  unsigned long long* wsum = reinterpret_cast<unsigned long long*>(sZ + 16);  // [8]
  unsigned* wc = reinterpret_cast<unsigned*>(wsum + 8);                       // [8]
  long long* s_res = reinterpret_cast<long long*>(wc + 8);                    // [4]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.G, LH = p.L * p.Hkv, G2 = 2 * p.G;
  const int n_bnd = p.hdr[HDR_N_BND];
  const long long units = (long long)n_bnd * LH;
  double* ws = p.score_ws + (size_t)blockIdx.x * ((size_t)p.cap * GP_PAGE) * G2;
  const double sqrt_d = sqrt((double)D);

  for (long long u = blockIdx.x; u < units; u += gridDim.x) {
    const int bidx = (int)(u / LH), lh = (int)(u % LH);
    const int l = lh / p.Hkv, h = lh % p.Hkv;
    const int bi = p.bnd_list[bidx];
    const int r = req_ids[bi];
    const int Pr = p.P[r];
    const int nC = (Pr - 1) * GP_PAGE;
    int* Kout = p.Kx + (((size_t)r * p.L + l) * p.Hkv + h) * 2;
    if (nC == 0) {
      if (tid == 0) { Kout[0] = 0; Kout[1] = 0; }
      continue;
    }
    const long long off = p.bnd_off[bi];
    double* aS = p.scores + ((size_t)lh) * p.max_batch_tokens + off;
    double* aL = p.scores + ((size_t)LH + lh) * p.max_batch_tokens + off;
    const int* table = p.page_table + (size_t)r * p.cap;
    __syncthreads();

    // ---- Eq. 12: per-head RMS calibration against this step's query, then RoPE at position t ----
    for (int vec = warp; vec < G2; vec += BT / 32) {
      const int x = vec / G, g = vec % G, head = h * G + g;
      const __nv_bfloat16* qrow = q + (((size_t)l * n_req + bi) * p.Hq + head) * D;
      const double* srow = p.summ + gp_summ_off(p, l, r, x, head);
      double sq = 0.0, ss = 0.0;
      for (int dd = lane; dd < D; dd += 32) {
        const double qv = (double)__bfloat162float(qrow[dd]);
        const double sv = srow[dd];
        sq += qv * qv;
        ss += sv * sv;
      }
#pragma unroll
      for (int o2 = 16; o2 > 0; o2 >>= 1) {
        sq += __shfl_xor_sync(0xffffffffu, sq, o2);
        ss += __shfl_xor_sync(0xffffffffu, ss, o2);
      }
      const double gamma = ss > 0.0 ? sqrt(sq / (double)D) / sqrt(ss / (double)D) : 1.0;
      double* dst = qt + (x * 8 + g) * D;
      for (int dd = lane; dd < D; dd += 32) dst[dd] = gamma * srow[dd];
      __syncwarp();
      if (p.rope_theta != 0.0) {
        const double* cs = p.rope_cs + (size_t)bi * (D / 2) * 2;
        for (int j = lane; j < D / 2; j += 32) {
          const double c = cs[2 * j], s = cs[2 * j + 1];
          const double x1 = dst[j], x2 = dst[j + D / 2];
          dst[j] = x1 * c - x2 * s;
          dst[j + D / 2] = x2 * c + x1 * s;
        }
      }
    }
    __syncthreads();

    // ---- pass 1: logits of every (token of C, view, head of the group) -------------------------------
    const int x = tid >> 7;                      // view handled by this thread: 0 short, 1 long
    const int rowi = tid & 127;
    double mx[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) mx[g] = -INFINITY;
    for (int t0 = 0; t0 < nC; t0 += GEO::TILE_TOK) {
      for (int i = tid; i < GEO::TILE_TOK * GEO::CH; i += BT) {
        const int rr = i / GEO::CH, pc = i % GEO::CH;
        const int tokn = t0 + rr;
        if (tokn < nC) {
          const int page = table[tokn / GP_PAGE];
          const uint4* src = reinterpret_cast<const uint4*>(p.kv + gp_tile_off(p, l, page, h)) +
                             (tokn % GP_PAGE) * GEO::CH + pc;
          ktile[i] = __ldg(src);
        }
      }
      __syncthreads();
      const int tokn = t0 + rowi;
      if (tokn < nC) {
        double acc[8];
#pragma unroll
        for (int g = 0; g < 8; ++g) acc[g] = 0.0;
        const int sw = rowi & 7;
#pragma unroll 2
        for (int c = 0; c < GEO::CH; ++c) {
          const uint4 kk = ktile[rowi * GEO::CH + (c ^ sw)];
          double kd[8];
          kd[0] = (double)bf16_lo_f(kk.x); kd[1] = (double)bf16_hi_f(kk.x);
          kd[2] = (double)bf16_lo_f(kk.y); kd[3] = (double)bf16_hi_f(kk.y);
          kd[4] = (double)bf16_lo_f(kk.z); kd[5] = (double)bf16_hi_f(kk.z);
          kd[6] = (double)bf16_lo_f(kk.w); kd[7] = (double)bf16_hi_f(kk.w);
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            if (g < G) {
              const double* qq = qt + (x * 8 + g) * D + c * 8;
#pragma unroll
              for (int e = 0; e < 8; ++e) acc[g] = fma(kd[e], qq[e], acc[g]);
            }
          }
        }
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          if (g < G) {
            const double z = acc[g] / sqrt_d;
            ws[(size_t)tokn * G2 + x * G + g] = z;
            mx[g] = fmax(mx[g], z);
          }
        }
      }
      __syncthreads();
    }
    // maxima per (view, head)
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      if (g < G) {
        double m = mx[g];
#pragma unroll
        for (int o2 = 16; o2 > 0; o2 >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o2));
        if (lane == 0) red[warp * 8 + g] = m;
      }
    }
    __syncthreads();
    if (tid < G2) {
      const int xx = tid / G, g = tid % G;
      double m = -INFINITY;
      for (int w = 0; w < 4; ++w) m = fmax(m, red[(xx * 4 + w) * 8 + g]);
      sM[tid] = m;
    }
    __syncthreads();

    // ---- pass 2: w = exp(z - max), normalisers ---------------------------------------------------------
    {
      const int col = tid % G2;
      const double m = sM[col];
      double zs = 0.0;
      const size_t entries = (size_t)nC * G2;
      for (size_t e2 = tid; e2 < entries; e2 += BT) {
        const double w = exp(ws[e2] - m);
        ws[e2] = w;
        zs += w;
      }
      red[tid] = zs;
      __syncthreads();
      if (tid < G2) {
        double z = 0.0;
        for (int k2 = tid; k2 < BT; k2 += G2) z += red[k2];
        sZ[tid] = z;
      }
      __syncthreads();
    }
    // ---- pass 3: a^x = mean over the group of the per-head softmaxes ----------------------------------
    for (int tokn = tid; tokn < nC; tokn += BT) {
      const double* wr = ws + (size_t)tokn * G2;
      double s0 = 0.0, s1 = 0.0;
      for (int g = 0; g < G; ++g) {
        s0 += wr[g] / sZ[g];
        s1 += wr[G + g] / sZ[G + g];
      }
      aS[tokn] = s0 / (double)G;
      aL[tokn] = s1 / (double)G;
    }
    __syncthreads();
    // ---- Eq. 7 -----------------------------------------------------------------------------------------
    const int KS = top_p_count(aS, nC, p.p_fix, hcnt, hsum, wc, wsum, s_res);
    const int KL = top_p_count(aL, nC, p.p_fix, hcnt, hsum, wc, wsum, s_res);
    if (tid == 0) { Kout[0] = KS; Kout[1] = KL; }
  }
}

// =====================================================================================================
template <int D>
__global__ void __launch_bounds__(BT)
gp_compact_kernel(const __grid_constant__ GpDev p, const int* __restrict__ req_ids, int n_req) {
  constexpr int CH = D / 8;
  constexpr int ROW_BYTES = D * 2;
  constexpr int MOVE_TOK = 64;                          // source slots per round
  constexpr int PIECES = MOVE_TOK * 2 * CH / BT;        // 16-byte pieces per thread per round
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((256u - (smem_u32(smem_raw) & 255u)) & 255u);
  unsigned* hcnt = reinterpret_cast<unsigned*>(smem);                          // [NBINS]
  double* stile = reinterpret_cast<double*>(hcnt + NBINS);                     // [BT]
  unsigned* wc = reinterpret_cast<unsigned*>(stile + BT);                      // [8]
  int* ev = reinterpret_cast<int*>(wc + 8);                                    // [16] evicted slots
  int* s_i = ev + 16;                                                          // [8] misc
  long long* s_res = reinterpret_cast<long long*>(s_i + 8);                    // [4]
  unsigned* loc = reinterpret_cast<unsigned*>(s_res + 4);                      // [cap*b/32] local-quota bits

  const int tid = threadIdx.x, lane = tid & 31;
  const int LH = p.L * p.Hkv;
  const int n_cmp = p.hdr[HDR_N_CMP];
  const long long units = (long long)n_cmp * LH;

  for (long long u = blockIdx.x; u < units; u += gridDim.x) {
    const int ci = (int)(u / LH), lh = (int)(u % LH);
    const int l = lh / p.Hkv, h = lh % p.Hkv;
    const int bi = p.cmp_list[ci];
    const int r = req_ids[bi];
    const int Pr = p.P[r];
    const int nC = (Pr - 1) * GP_PAGE;
    const int nblk = Pr - 1;
    const int K_t = nC - GP_PAGE;
    const int kq = min(p.k_loc, K_t / nblk);             // k' of Eq. 10
    const long long off = p.bnd_off[bi];
    const double* aS = p.scores + ((size_t)lh) * p.max_batch_tokens + off;
    const double* aL = p.scores + ((size_t)LH + lh) * p.max_batch_tokens + off;
    const int* table = p.page_table + (size_t)r * p.cap;
    const int* shadow = p.shadow + (size_t)r * p.cap;
    __syncthreads();

    // ---- block-local quota: the k' best slots of every page of C (score desc, slot asc) ---------------
    for (int i = tid; i < (nC + 31) / 32; i += BT) loc[i] = 0;
    if (tid == 0) { s_i[0] = 0; s_i[1] = 0x7fffffff; s_i[3] = 0; }
    __syncthreads();
    for (int t0 = 0; t0 < nC; t0 += BT) {
      const int tokn = t0 + tid;
      double s = 0.0;
      if (tokn < nC) s = fmax(__ldcg(aS + tokn), __ldcg(aL + tokn));     // Eq. 9
      stile[tid] = s;
      __syncthreads();
      if (tokn < nC && kq > 0) {
        const int b0 = tid & ~15;
        int rank = 0;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const double sj = stile[b0 + j];
          rank += (sj > s) || (sj == s && (b0 + j) < tid);
        }
        if (rank < kq) atomicOr(&loc[tokn >> 5], 1u << (tokn & 31));
      }
      __syncthreads();
    }
    // first page whose source is shared (copy-on-write): everything from there on is rewritten
    for (int j = tid; j < Pr - 1; j += BT)
      if (shadow[j] >= 0) atomicMin(&s_i[1], j * GP_PAGE);
    __syncthreads();

    // ---- global cut: evict the b lowest of the rest (score asc, slot desc) --------------------------------
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
        for (int i = tid; i < nb; i += BT) hcnt[i] = 0;
        if (tid == 0) s_res[0] = -1;
        __syncthreads();
        for (int i = tid; i < nC; i += BT) {
          if (!((loc[i >> 5] >> (i & 31)) & 1u)) {
            const unsigned long long key =
                (unsigned long long)__double_as_longlong(fmax(__ldcg(aS + i), __ldcg(aL + i)));
            if (lvl == 0 || (key >> (shift + w)) == prefix)
              atomicAdd(&hcnt[(int)((key >> shift) & (unsigned long long)(nb - 1))], 1u);
          }
        }
        __syncthreads();
        const int per = nb / BT > 0 ? nb / BT : 1;
        const int lo = tid * per, hi = lo + per;
        unsigned c = 0;
        if (lo < nb) for (int b = lo; b < hi; ++b) c += hcnt[b];
        const unsigned ex = block_prefix_excl(c, wc);
        if (lo < nb) {
          unsigned run = cnt_below + ex;
          for (int b = lo; b < hi; ++b) {
            const unsigned before = run;
            run += hcnt[b];
            if (before < (unsigned)GP_PAGE && run >= (unsigned)GP_PAGE) { s_res[0] = b; s_res[1] = before; }
          }
        }
        __syncthreads();
        if (s_res[0] < 0) {                                  // fewer than b candidates: cannot happen
          if (tid == 0) atomicOr(p.err, GP_E_BOUNDS);
          break;
        }
        const int bin_star = (int)s_res[0];
        cnt_below = (unsigned)s_res[1];
        const unsigned cstar = hcnt[bin_star];
        __syncthreads();
        prefix = (prefix << w) | (unsigned long long)bin_star;
        if (cnt_below + cstar == (unsigned)GP_PAGE) {        // the bin fits exactly: no tie to break
          thr = (prefix + 1ull) << shift;
          done = true;
        }
      }
      if (!done) {                                           // equal scores straddle the cut
        thr = prefix;
        tie_key = prefix;
        need_eq = GP_PAGE - (int)cnt_below;
      }
    }
    // ---- list the evicted slots --------------------------------------------------------------------------
    for (int i = tid; i < nC; i += BT) {
      if (!((loc[i >> 5] >> (i & 31)) & 1u)) {
        const unsigned long long key = (unsigned long long)__double_as_longlong(fmax(__ldcg(aS + i), __ldcg(aL + i)));
        if (key < thr) { const int at = atomicAdd(&s_i[0], 1); if (at < GP_PAGE) ev[at] = i; }
      }
    }
    __syncthreads();
    if (tid == 0) {
      int cntv = s_i[0];
      for (int i = nC - 1; i >= 0 && need_eq > 0; --i) {     // rare: older (lower) slots win ties
        if (!((loc[i >> 5] >> (i & 31)) & 1u)) {
          const unsigned long long key = (unsigned long long)__double_as_longlong(fmax(__ldcg(aS + i), __ldcg(aL + i)));
          if (key == tie_key) { if (cntv < GP_PAGE) ev[cntv] = i; ++cntv; --need_eq; }
        }
      }
      if (cntv != GP_PAGE) atomicOr(p.err, GP_E_BOUNDS);
      for (int a = 1; a < GP_PAGE; ++a) {                    // sort the 16 slots ascending
        const int key = ev[a];
        int b2 = a - 1;
        while (b2 >= 0 && ev[b2] > key) { ev[b2 + 1] = ev[b2]; --b2; }
        ev[b2 + 1] = key;
      }
    }
    __syncthreads();

    // ---- stable compaction: survivors of C in slot order, then the protected page ------------------------
    const int n_src = Pr * GP_PAGE;
    int start = min(ev[0], s_i[1]);
    start = (start / MOVE_TOK) * MOVE_TOK;
    for (int c0 = start; c0 < n_src; c0 += MOVE_TOK) {
      uint4 val[PIECES];
      int dst_slot[PIECES];
      int tokv = 0, tok_dst = -1;
#pragma unroll
      for (int k2 = 0; k2 < PIECES; ++k2) {
        const int piece = tid + k2 * BT;
        const int tl = piece / (2 * CH), pc = piece % (2 * CH);
        const int i = c0 + tl;
        dst_slot[k2] = -1;
        if (i < n_src) {
          int sh = 0; bool evicted = false;
#pragma unroll
          for (int e2 = 0; e2 < GP_PAGE; ++e2) { sh += (ev[e2] < i); evicted |= (ev[e2] == i); }
          const int pg = i / GP_PAGE;
          const bool cow = (pg < Pr - 1) && (shadow[pg] >= 0);
          if (!evicted && (sh > 0 || cow)) {
            const int isv = pc / CH, cp = pc % CH;
            const uint8_t* src = reinterpret_cast<const uint8_t*>(p.kv + gp_tile_off(p, l, table[pg], h)) +
                                 isv * GP_PAGE * ROW_BYTES + (i % GP_PAGE) * ROW_BYTES + (cp << 4);
            val[k2] = *reinterpret_cast<const uint4*>(src);
            // remember the logical chunk in the low bits of the destination code
            dst_slot[k2] = ((i - sh) << 5) | ((cp ^ (i & 7)) << 1) | isv;
          }
        }
      }
      if (tid < MOVE_TOK) {
        const int i = c0 + tid;
        if (i < n_src) {
          int sh = 0; bool evicted = false;
#pragma unroll
          for (int e2 = 0; e2 < GP_PAGE; ++e2) { sh += (ev[e2] < i); evicted |= (ev[e2] == i); }
          const int pg = i / GP_PAGE;
          const bool cow = (pg < Pr - 1) && (shadow[pg] >= 0);
          if (!evicted && (sh > 0 || cow)) {
            tokv = p.tok[gp_tok_off(p, l, table[pg], h) + (i % GP_PAGE)];
            tok_dst = i - sh;
          }
        }
      }
      __syncthreads();
#pragma unroll
      for (int k2 = 0; k2 < PIECES; ++k2) {
        if (dst_slot[k2] >= 0) {
          const int ds = dst_slot[k2] >> 5, c = (dst_slot[k2] >> 1) & 15, isv = dst_slot[k2] & 1;
          const int pg = ds / GP_PAGE;
          const int page = shadow[pg] >= 0 ? shadow[pg] : table[pg];
          uint8_t* dst = reinterpret_cast<uint8_t*>(p.kv + gp_tile_off(p, l, page, h)) + isv * GP_PAGE * ROW_BYTES +
                         (ds % GP_PAGE) * ROW_BYTES + ((c ^ (ds & 7)) << 4);
          *reinterpret_cast<uint4*>(dst) = val[k2];
        }
      }
      if (tok_dst >= 0) {
        atomicAdd(&s_i[3], 1);
        const int pg = tok_dst / GP_PAGE;
        const int page = shadow[pg] >= 0 ? shadow[pg] : table[pg];
        p.tok[gp_tok_off(p, l, page, h) + (tok_dst % GP_PAGE)] = tokv;
      }
      __syncthreads();
    }
    if (tid == 0) atomicAdd(reinterpret_cast<unsigned long long*>(p.counters + 8), (unsigned long long)s_i[3]);
  }

  // ---- the last CTA swaps in the copy-on-write targets and drops the old references (App. D.2) ----------
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
      const int r = req_ids[p.cmp_list[ci]];
      const int Pr = p.P[r];
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
    }
  }
}

}  // namespace

void gp_launch_score(const GpDev& p, const int* req_ids, int n_req, const void* q, cudaStream_t s) {
  const __nv_bfloat16* qq = static_cast<const __nv_bfloat16*>(q);
  if (p.d == 128) {
    auto kern = gp_score_kernel<128>;
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ScoreGeom<128>::SMEM);
    kern<<<p.score_grid, BT, ScoreGeom<128>::SMEM, s>>>(p, req_ids, n_req, qq);
  } else {
    auto kern = gp_score_kernel<64>;
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ScoreGeom<64>::SMEM);
    kern<<<p.score_grid, BT, ScoreGeom<64>::SMEM, s>>>(p, req_ids, n_req, qq);
  }
}

size_t gp_compact_smem(const GpDev& p) {
  return NBINS * 4 + BT * 8 + 8 * 4 + 16 * 4 + 8 * 4 + 4 * 8 + ((size_t)p.cap * GP_PAGE / 32 + 1) * 4 + 256 + 64;
}

void gp_launch_compact(const GpDev& p, const int* req_ids, int n_req, int grid, cudaStream_t s) {
  const size_t sm = gp_compact_smem(p);
  if (p.d == 128) {
    auto kern = gp_compact_kernel<128>;
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    kern<<<grid, BT, sm, s>>>(p, req_ids, n_req);
  } else {
    auto kern = gp_compact_kernel<64>;
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    kern<<<grid, BT, sm, s>>>(p, req_ids, n_req);
  }
}
