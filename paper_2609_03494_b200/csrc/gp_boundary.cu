// Capacity-boundary kernels (Sec. 3.2 - 3.3, App. D.1, App. D.2), launched every step after attention.
// The attention kernel has already left, for every (request at a boundary, layer, KV head) unit, the
// fp64 logits z of the two calibrated summaries against every candidate key.
//
//   gp_bsel_kernel    first merges the partial attention outputs of requests split over several work items;
//                     then, per unit: per-head softmax over the candidate set and group mean -> a^S, a^L;
//                     working-set sizes K^S, K^L (Eq. 7); and, speculatively, the b slots a compression
//                     would evict (Eq. 9, Eq. 10).  The last CTA to finish aggregates Eq. 8, decides grow
//                     or compress per request and runs the device allocator: grants first, then
//                     copy-on-write targets, each in ascending request id.
//   gp_compact_kernel per (compressing unit, chunk of 64 source slots): stable in-place compaction into
//                     (P-1) b slots, writing to copy-on-write targets where the source page is shared.
//                     Chunks are claimed in order from a ticket counter; a chunk publishes "my sources
//                     are read" before the next chunk may overwrite their tail.  The last CTA swaps in the
//                     target pages and drops the references to the replaced ones.
//
// Everything that decides an integer outcome is fp64.  Top-p counting and top-k selection are radix
// descents over the IEEE bit patterns of the (non-negative) scores, 11 bits per level, with histograms in
// shared memory; the top-p mass is accumulated in 2^62 fixed point with integer atomics, so the result
// does not depend on the order in which threads add.
#include "../../include/growpage.h"
#include "gp_dev.cuh"

namespace {

constexpr int NBINS = 2048;
constexpr int NBINS_PAD = NBINS + NBINS / 8;     // bins are stored at b + (b >> 3): a thread's 8 consecutive bins and
#define HIDX(b) ((b) + ((b) >> 3))              // its neighbours' then fall into different banks
constexpr double TWO62 = 4611686018427387904.0;
constexpr int SEL_T = 256;           // threads of the selection kernel
constexpr int SEL_CAP = 6144;        // candidate tokens whose scores are staged in shared memory
constexpr int CT = 256;              // threads of the compaction kernel
constexpr int MOVE_TOK = GP_MOVE_TOK;     // source slots per compaction chunk

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
__device__ int top_p_count(const GpDev& p, const double* a, int n, unsigned long long p_fix, unsigned* hcnt,
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
    const long long t_l0 = GP_T_NOW();
    (void)t_l0;
    for (int i = tid; i < nb + (nb >> 3); i += BT) { hcnt[i] = 0; hlo[i] = 0; hhi[i] = 0; }
    if (tid == 0) s_res[0] = -1;
    __syncthreads();
    const long long t_l1 = GP_T_NOW();
    (void)t_l1;
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
    const long long t_l2 = GP_T_NOW();
    (void)t_l2;
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
    if (tid == 0) { GP_T_ADD(30, 1); GP_T_ADD(12, t_l1 - t_l0); GP_T_ADD(13, t_l2 - t_l1); GP_T_ADD(14, GP_T_NOW() - t_l2); }
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
// decision + allocator, run by the last CTA of the selection kernel
// ------------------------------------------------------------------------------------------------------
__device__ void decide_and_allocate(const GpDev& p, const int* req_ids, int n_req, int* actions, int* s_arr) {
  int* s_want = s_arr;
  int* s_ksh = s_arr + GP_MAX_REQ;
  int* s_P = s_arr + 2 * GP_MAX_REQ;
  int* s_order = s_arr + 3 * GP_MAX_REQ;
  int* s_req = s_arr + 4 * GP_MAX_REQ;
  int* s_base = s_arr + 5 * GP_MAX_REQ;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarp = blockDim.x >> 5;
  const int n_bnd = p.hdr[HDR_N_BND];
  for (int i = tid; i < n_req; i += blockDim.x) {
    if (p.b_flags[i]) {
      const int r = req_ids[i];
      p.n[r] = p.b_nold[i] + 1;
      p.pos[r] += 1;
      p.started[r] = 1;
      p.sum_par[r] ^= 1;                                  // the attention kernel wrote the other buffer
    }
  }
  if (tid == 0) {
    p.counters[5] += 1;
    p.counters[6] += p.hdr[HDR_N_ACTIVE];
    p.hdr[HDR_N_CMP] = 0;
    p.hdr[HDR_N_CITEM] = 0;
    p.hdr[HDR_WORK_CMP] = 0;
  }
  if (n_bnd == 0) return;
  __syncthreads();
  const int LH = p.L * p.Hkv;
  for (int e = warp; e < n_bnd; e += nwarp) {
    const int bi = p.bnd_list[e];
    const int r = req_ids[bi];
    const int Pr = p.P[r];
    const int nC = (Pr - 1) * GP_PAGE;
    long long sS = 0, sL = 0;
    const int* kx = p.Kx + (size_t)r * LH * 2;
    for (int j = lane; j < LH; j += 32) { sS += kx[2 * j]; sL += kx[2 * j + 1]; }
    int ksh = 0;
    const int* table = p.page_table + (size_t)r * p.cap;
    for (int j = lane; j < Pr - 1; j += 32) ksh += (p.refcount[table[j]] > 1);
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) {
      sS += __shfl_xor_sync(0xffffffffu, sS, o2);
      sL += __shfl_xor_sync(0xffffffffu, sL, o2);
      ksh += __shfl_xor_sync(0xffffffffu, ksh, o2);
    }
    if (lane == 0) {
      // Eq. 8 with a common |C|: Delta = (sum K^S - sum K^L) / (N |C|), one division of exact integers
      double delta = 0.0;
      int want = 1;
      if (nC > 0) {
        delta = (double)(sS - sL) / ((double)LH * (double)nC);
        want = delta > p.tau;
      }
      p.delta[r] = delta;
      s_want[e] = want; s_ksh[e] = ksh; s_P[e] = Pr; s_req[e] = r;
    }
  }
  __syncthreads();
  for (int e = tid; e < n_bnd; e += blockDim.x) {
    int rank = 0;
    for (int f = 0; f < n_bnd; ++f) rank += (s_req[f] < s_req[e]);
    s_order[rank] = e;
  }
  __syncthreads();
  if (tid == 0) {
    int top = *p.free_top;
    int n_cmp = 0, chunks = 0;
    long long grow = 0, comp = 0, fall = 0, stall = 0, cow = 0, scored = 0;
    for (int k = 0; k < n_bnd; ++k) {                    // pass 1: grants
      const int e = s_order[k];
      const int r = s_req[e], Pr = s_P[e], bi = p.bnd_list[e];
      scored += (long long)(Pr - 1) * GP_PAGE;
      if ((s_want[e] & 1) && Pr < p.cap && top > 0) {
        const int page = p.free_stack[--top];
        p.refcount[page] = 1;
        p.page_table[(size_t)r * p.cap + Pr] = page;
        p.P[r] = Pr + 1;
        actions[bi] = GP_ACT_GROW;
        s_want[e] |= 2;
        ++grow;
      } else if (Pr == 1) {
        actions[bi] = GP_ACT_STALLED;
        s_want[e] |= 4;
        ++stall;
      }
    }
    for (int k = 0; k < n_bnd; ++k) {                    // pass 2: copy-on-write targets
      const int e = s_order[k];
      if (s_want[e] & 6) continue;
      const int r = s_req[e], bi = p.bnd_list[e];
      if (s_ksh[e] > top) {
        actions[bi] = GP_ACT_STALLED;
        ++stall;
        continue;
      }
      s_base[e] = top;
      top -= s_ksh[e];
      cow += s_ksh[e];
      p.cmp_list[n_cmp] = bi;
      p.cmp_bnd[n_cmp] = e;
      p.cmp_chunk0[n_cmp] = chunks;
      chunks += (s_P[e] * GP_PAGE + MOVE_TOK - 1) / MOVE_TOK;
      ++n_cmp;
      if (s_want[e] & 1) { actions[bi] = GP_ACT_COMPRESS_FALLBACK; ++fall; } else { actions[bi] = GP_ACT_COMPRESS; ++comp; }
      p.n[r] = (s_P[e] - 1) * GP_PAGE;
      p.n_pristine[r] = 0;
      s_want[e] |= 8;
    }
    p.cmp_chunk0[n_cmp] = chunks;
    if (top < 0) atomicOr(p.err, GP_E_FREELIST);
    *p.free_top = top;
    p.hdr[HDR_N_CMP] = n_cmp;
    p.hdr[HDR_N_CITEM] = chunks * LH;
    p.counters[0] += grow; p.counters[1] += comp; p.counters[2] += fall; p.counters[3] += stall; p.counters[4] += cow;
    p.counters[9] += scored;
  }
  __syncthreads();
  for (int e = warp; e < n_bnd; e += nwarp) {             // fill in the targets, in table order
    if (!(s_want[e] & 8) || s_ksh[e] == 0) continue;
    const int r = s_req[e], Pr = s_P[e], base = s_base[e];
    const int* table = p.page_table + (size_t)r * p.cap;
    int* shadow = p.shadow + (size_t)r * p.cap;
    int running = 0;
    for (int j0 = 0; j0 < Pr - 1; j0 += 32) {
      const int j = j0 + lane;
      const bool sh = j < Pr - 1 && p.refcount[table[j]] > 1;
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

// ------------------------------------------------------------------------------------------------------
// working sets + speculative eviction list; three independent jobs per unit, one CTA each; the last CTA decides
// ------------------------------------------------------------------------------------------------------
struct SelGeom {
  static constexpr size_t BUF_BYTES = SEL_CAP * sizeof(double);
  static constexpr size_t H_BYTES = NBINS_PAD * 4 + NBINS_PAD * 8;
  static constexpr size_t MISC_BYTES = 8 * 8 + 8 * 4 + 8 * 8 + 16 * 4 + 16 * 4 + (8 * 16 + 32) * 8;
};

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

__global__ void __launch_bounds__(SEL_T)
gp_bsel_kernel(const __grid_constant__ GpDev p, const int* __restrict__ req_ids, int n_req, int* __restrict__ actions,
               float* __restrict__ out) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((256u - (smem_u32(smem_raw) & 255u)) & 255u);
  double* sbuf = reinterpret_cast<double*>(smem);                              // [SEL_CAP] a^S, a^L or s
  unsigned* hcnt = reinterpret_cast<unsigned*>(smem + SelGeom::BUF_BYTES);
  unsigned long long* hsum = reinterpret_cast<unsigned long long*>(hcnt + NBINS_PAD);
  unsigned long long* wsum = hsum + NBINS_PAD;                                 // [8]
  unsigned* wc = reinterpret_cast<unsigned*>(wsum + 8);                        // [8]
  long long* s_res = reinterpret_cast<long long*>(wc + 8);                     // [8]
  int* ev = reinterpret_cast<int*>(s_res + 8);                                 // [16]
  int* s_i = ev + 16;                                                          // [16]
  double* red = reinterpret_cast<double*>(s_i + 16);                           // [8][16]
  double* sM = red + 8 * 16;                                                   // [16]
  double* sZ = sM + 16;                                                        // [16]
  unsigned* loc = reinterpret_cast<unsigned*>(sZ + 16);                        // [cap*b/32 + 1]
  // the decision scratch aliases the score staging area: it is used after the last item only

  const int tid = threadIdx.x;
  const int LH = p.L * p.Hkv;
  const int n_bnd = p.hdr[HDR_N_BND];
  const long long items = (long long)n_bnd * LH * 3;
  const int G = p.G, G2 = 2 * p.G;

  // ---- attention outputs of requests that were split over several work items: merge the partials -----------
  {
    const int n_mc = p.hdr[HDR_N_MC], n_rc = p.hdr[HDR_N_RC], D = p.d;
    const int PSTRIDE = G * (D + 2);
    for (long long mi = blockIdx.x; mi < (long long)n_mc * LH; mi += gridDim.x) {
      const int4 mc = p.mc_list[mi / LH];
      const int lh = (int)(mi % LH), l = lh / p.Hkv, h = lh % p.Hkv;
      const int bi = mc.x, nch = mc.z;
      const float* first = p.partials + ((size_t)lh * n_rc + mc.y) * PSTRIDE;
      float* orow = out + (((size_t)l * n_req + bi) * p.Hq + h * G) * D;
      for (int idx = tid; idx < G * D; idx += SEL_T) {
        const int g = idx / D, dc = idx % D;
        const float* pg = first + g * (D + 2);
        float M = -INFINITY;
        for (int c = 0; c < nch; ++c) M = fmaxf(M, __ldcg(pg + (size_t)c * PSTRIDE + D));
        float acc = 0.f, ls = 0.f;
#pragma unroll 4
        for (int c = 0; c < nch; ++c) {
          const float* pc = pg + (size_t)c * PSTRIDE;
          const float w = exp2f(__ldcg(pc + D) - M);
          acc += w * __ldcg(pc + dc);
          ls += w * __ldcg(pc + D + 1);
        }
        orow[idx] = acc / ls;
      }
    }
  }

  for (long long item = blockIdx.x; item < items; item += gridDim.x) {
    const long long u = item / 3;
    const int task = (int)(item % 3);               // 0: K^S, 1: K^L, 2: eviction list
    const int bidx = (int)(u / LH), lh = (int)(u % LH);
    const int l = lh / p.Hkv, h = lh % p.Hkv;
    const int bi = p.bnd_list[bidx];
    const int r = req_ids[bi];
    const int Pr = p.P[r];
    const int nC = (Pr - 1) * GP_PAGE;
    int* Kout = p.Kx + (((size_t)r * p.L + l) * p.Hkv + h) * 2;
    int* evout = p.evict + (size_t)u * GP_PAGE;
    __syncthreads();
    if (nC == 0) {
      if (tid == 0 && task < 2) Kout[task] = 0;
      continue;
    }
    const long long t_s0 = GP_T_NOW();
    (void)t_s0;
    const long long off = p.bnd_off[bi];
    const double* z = p.zbuf + ((size_t)lh * p.max_batch_tokens + off) * G2;      // [nC][2][G]
    double* a = nC <= SEL_CAP ? sbuf : p.scores + ((size_t)task * LH + lh) * p.max_batch_tokens + off;
    // ---- per-head softmax over C, then the group mean (Sec. 3.2) --------------------------------------------
    // The attention kernel left, per 16-token page and column, the page's (max, sum of exponentials); they
    // merge into the normalisers of the whole candidate set without another pass over the logits.
    {
      const int ncols = task == 2 ? G2 : G;
      const int col0 = task == 1 ? G : 0;
      const int mycol = col0 + tid % ncols;                  // SEL_T is a multiple of ncols
      const int ntile = nC / GP_PAGE;
      const double* zs = p.zstat + ((size_t)lh * (p.max_batch_tokens / GP_PAGE) + off / GP_PAGE) * G2 * 2;
      double m = -INFINITY;
      for (int t = tid / ncols; t < ntile; t += SEL_T / ncols) m = fmax(m, __ldcg(zs + ((size_t)t * G2 + mycol) * 2));
      column_reduce<true>(m, ncols, red, sM);
      const double mc = sM[tid % ncols];
      double acc = 0.0;
      for (int t = tid / ncols; t < ntile; t += SEL_T / ncols) {
        const double2 ms = __ldcg(reinterpret_cast<const double2*>(zs + ((size_t)t * G2 + mycol) * 2));
        acc += ms.y * exp(ms.x - mc);
      }
      column_reduce<false>(acc, ncols, red, sZ);
      for (int i0 = tid; i0 < nC; i0 += 4 * SEL_T) {         // four tokens per thread in flight
        double zv[4][16];
#pragma unroll
        for (int u4 = 0; u4 < 4; ++u4) {
          const int i = i0 + u4 * SEL_T;
          if (i < nC) {
            const double* zr = z + (size_t)i * G2 + col0;
            for (int g = 0; g < ncols; ++g) zv[u4][g] = __ldcg(zr + g);
          }
        }
#pragma unroll
        for (int u4 = 0; u4 < 4; ++u4) {
          const int i = i0 + u4 * SEL_T;
          if (i < nC) {
            double s0 = 0.0, s1 = 0.0;
            for (int g = 0; g < G; ++g) s0 += exp(zv[u4][g] - sM[g]) / sZ[g];
            if (task == 2) {
              for (int g = 0; g < G; ++g) s1 += exp(zv[u4][G + g] - sM[G + g]) / sZ[G + g];
              a[i] = fmax(s0 / (double)G, s1 / (double)G);   // Eq. 9
            } else {
              a[i] = s0 / (double)G;
            }
          }
        }
      }
      __syncthreads();
    }
    const long long t_s1 = GP_T_NOW();
    (void)t_s1;
    if (task < 2) {
      // ---- Eq. 7 -------------------------------------------------------------------------------------------
      const int K = top_p_count<SEL_T>(p, a, nC, p.p_fix, hcnt, hsum, wc, wsum, s_res);
      if (tid == 0) {
        Kout[task] = K;
        GP_T_ADD(16, 1); GP_T_ADD(17, t_s1 - t_s0); GP_T_ADD(18, GP_T_NOW() - t_s1); GP_T_ADD(25, nC);
      }
      continue;
    }
    // ---- Eq. 10, block-local quota: the k' best slots of every page of C (score desc, slot asc) -------------
    for (int i = tid; i < (nC + 31) / 32; i += SEL_T) loc[i] = 0;
    if (tid == 0) s_i[0] = 0;
    __syncthreads();
    const int nblk = Pr - 1;
    const int K_t = nC - GP_PAGE;
    const int kq = min(p.k_loc, K_t / nblk);
    if (kq > 0) {
      for (int i = tid; i < nC; i += SEL_T) {
        const double s = a[i];
        const int b0 = i & ~15;
        int rank = 0;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const double sj = a[b0 + j];
          rank += (sj > s) || (sj == s && (b0 + j) < i);
        }
        if (rank < kq) atomicOr(&loc[i >> 5], 1u << (i & 31));
      }
    }
    __syncthreads();
    const long long t_s3 = GP_T_NOW();
    (void)t_s3;
    // ---- global cut: the b lowest of the rest are evicted (score asc, slot desc) --------------------------------
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
        const unsigned cstar = hcnt[HIDX(bin_star)];
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
    const long long t_s4 = GP_T_NOW();
    (void)t_s4;
    for (int i = tid; i < nC; i += SEL_T) {
      if (!((loc[i >> 5] >> (i & 31)) & 1u)) {
        const unsigned long long key = (unsigned long long)__double_as_longlong(a[i]);
        if (key < thr) { const int at = atomicAdd(&s_i[0], 1); if (at < GP_PAGE) ev[at] = i; }
      }
    }
    __syncthreads();
    if (tid == 0) {
      GP_T_ADD(31, 1); GP_T_ADD(19, t_s3 - t_s1); GP_T_ADD(20, t_s4 - t_s3); GP_T_ADD(22, t_s1 - t_s0);
      int cntv = s_i[0];
      for (int i = nC - 1; i >= 0 && need_eq > 0; --i) {     // rare: older (lower) slots win ties
        if (!((loc[i >> 5] >> (i & 31)) & 1u)) {
          const unsigned long long key = (unsigned long long)__double_as_longlong(a[i]);
          if (key == tie_key) { if (cntv < GP_PAGE) ev[cntv] = i; ++cntv; --need_eq; }
        }
      }
      if (cntv != GP_PAGE) atomicOr(p.err, GP_E_BOUNDS);
      for (int x = 1; x < GP_PAGE; ++x) {                    // sort the 16 slots ascending
        const int key = ev[x];
        int b2 = x - 1;
        while (b2 >= 0 && ev[b2] > key) { ev[b2 + 1] = ev[b2]; --b2; }
        ev[b2 + 1] = key;
      }
      for (int x = 0; x < GP_PAGE; ++x) evout[x] = ev[x];
      GP_T_ADD(21, GP_T_NOW() - t_s4);
    }
  }

  // ---- the last CTA takes the decisions ----------------------------------------------------------------------
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int prev = atomicAdd(&p.hdr[HDR_DONE_SEL], 1);
    s_i[2] = (prev == (int)gridDim.x - 1);
    if (prev == (int)gridDim.x - 1) p.hdr[HDR_DONE_SEL] = 0;
  }
  __syncthreads();
  if (s_i[2]) {
    __threadfence();
    const long long t_d0 = GP_T_NOW();
    (void)t_d0;
    decide_and_allocate(p, req_ids, n_req, actions, reinterpret_cast<int*>(sbuf));
    if (tid == 0) { GP_T_ADD(23, GP_T_NOW() - t_d0); GP_T_ADD(24, 1); }
  }
}

// ------------------------------------------------------------------------------------------------------
// compaction
// ------------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(CT)
gp_compact_kernel(const __grid_constant__ GpDev p, const int* __restrict__ req_ids, int n_req) {
  constexpr int CH = D / 8;
  constexpr int ROW_BYTES = D * 2;
  constexpr int PIECES = MOVE_TOK * 2 * CH / CT;        // 16-byte pieces per thread per chunk
  __shared__ int s_pref[GP_MAX_REQ + 1];
  __shared__ int ev[GP_PAGE];
  __shared__ int s_i[8];

  const int tid = threadIdx.x, lane = tid & 31;
  const int LH = p.L * p.Hkv;
  const int n_cmp = p.hdr[HDR_N_CMP];
  const int n_items = p.hdr[HDR_N_CITEM];
  const int stamp = p.hdr[HDR_STEP];
  for (int i = tid; i <= n_cmp; i += CT) s_pref[i] = p.cmp_chunk0[i];
  if (tid == 0) s_i[3] = 0;
  __syncthreads();

  for (;;) {
    __syncthreads();
    if (tid == 0) s_i[0] = n_items > 0 ? atomicAdd(&p.hdr[HDR_WORK_CMP], 1) : 0x7fffffff;
    __syncthreads();
    const int item = s_i[0];
    if (item >= n_items) break;
    // item -> (compressing request, layer/head, chunk); chunks of a unit are consecutive and ascending
    int lo = 0, hi = n_cmp;
    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (LH * s_pref[mid] <= item) lo = mid; else hi = mid; }
    const int ci = lo;
    const int nchunk = s_pref[ci + 1] - s_pref[ci];
    const int rem = item - LH * s_pref[ci];
    const int lh = rem / nchunk, j = rem % nchunk;
    const int l = lh / p.Hkv, h = lh % p.Hkv;
    const int bi = p.cmp_list[ci];
    const int r = req_ids[bi];
    const int Pr = p.P[r];
    const int n_src = Pr * GP_PAGE;
    const int* table = p.page_table + (size_t)r * p.cap;
    const int* shadow = p.shadow + (size_t)r * p.cap;
    if (tid < GP_PAGE) ev[tid] = p.evict[((size_t)p.cmp_bnd[ci] * LH + lh) * GP_PAGE + tid];
    __syncthreads();
    const int c0 = j * MOVE_TOK;

    uint4 val[PIECES];
    int dst_code[PIECES];
    int tokv = 0, tok_dst = -1;
#pragma unroll
    for (int k2 = 0; k2 < PIECES; ++k2) {
      const int piece = tid + k2 * CT;
      const int tl = piece / (2 * CH), pc = piece % (2 * CH);
      const int i = c0 + tl;
      dst_code[k2] = -1;
      val[k2] = make_uint4(0, 0, 0, 0);
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
          dst_code[k2] = ((i - sh) << 5) | ((cp ^ (i & 7)) << 1) | isv;   // slot, logical chunk, K or V
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
    // Touch every loaded value so that the loads have completed before the flag below is published: the
    // next chunk's CTA may overwrite the tail of this chunk's sources as soon as it sees the flag.
    unsigned touched = (unsigned)tokv;
#pragma unroll
    for (int k2 = 0; k2 < PIECES; ++k2) touched ^= val[k2].x ^ val[k2].y ^ val[k2].z ^ val[k2].w;
    if (touched == 0x9e3779b9u && c0 < 0) s_i[4] = 1;      // never true; keeps the dependency alive
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      *reinterpret_cast<volatile int*>(p.cflags + item) = stamp;      // "my sources are read"
      if (j > 0) {                                          // the previous chunk's tail is my first destination
        volatile int* prev = reinterpret_cast<volatile int*>(p.cflags + item - 1);
        unsigned it = 0;
        while (*prev != stamp && it < GP_SPIN_LIMIT) ++it;
        if (it >= GP_SPIN_LIMIT) atomicOr(p.err, GP_E_SPIN_CMP);
        __threadfence();
      }
    }
    __syncthreads();
#pragma unroll
    for (int k2 = 0; k2 < PIECES; ++k2) {
      if (dst_code[k2] >= 0) {
        const int ds = dst_code[k2] >> 5, c = (dst_code[k2] >> 1) & 15, isv = dst_code[k2] & 1;
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
  }
  __syncthreads();
  if (tid == 0 && s_i[3] > 0)
    atomicAdd(reinterpret_cast<unsigned long long*>(p.counters + 8), (unsigned long long)s_i[3]);

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

size_t gp_bsel_smem(const GpDev& p) {
  return SelGeom::BUF_BYTES + SelGeom::H_BYTES + SelGeom::MISC_BYTES + ((size_t)p.cap * GP_PAGE / 32 + 2) * 4 + 512;
}

void gp_launch_boundary(const GpDev& p, const int* req_ids, int n_req, int* actions, float* out, int grid_sel,
                        int grid_compact, cudaStream_t s, cudaEvent_t ev) {
  const size_t sel_sm = gp_bsel_smem(p);
  cudaFuncSetAttribute(gp_bsel_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sel_sm);
  gp_bsel_kernel<<<grid_sel, SEL_T, sel_sm, s>>>(p, req_ids, n_req, actions, out);
  if (ev) cudaEventRecord(ev, s);
  if (p.d == 128) gp_compact_kernel<128><<<grid_compact, CT, 0, s>>>(p, req_ids, n_req);
  else gp_compact_kernel<64><<<grid_compact, CT, 0, s>>>(p, req_ids, n_req);
}
