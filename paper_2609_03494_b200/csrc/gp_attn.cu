// Fused append + GQA paged decode attention + dual EMA summary update (Sec. 3.2 Eq. 6, Sec. 4.1), plus,
// for requests that reach their capacity boundary with this step, the logits of the two calibrated
// summaries against every candidate key (Eq. 12, App. D.1) while the key tile is in shared memory.
//
// Work decomposition.  The plan kernel cuts every stepped request into chunks of `chunk_pages` pages and
// writes one descriptor per chunk; a work item is (chunk, layer, KV head).  A persistent grid (two CTAs
// per SM) pulls items from a global counter.  Each CTA is warp-specialised:
//
//   warp 0      producer: claims items, publishes their descriptor in a ring of item slots, and streams
//               the K|V tiles of their pages (one contiguous `cp.async.bulk` per (layer, page, head))
//               into a ring of stages shared by the CTA.  It runs ahead across item boundaries, so the
//               ring never drains between items.
//   warps 1..4  consumers: take the tiles of an item round-robin.  The G query heads of the group are
//               rows 0..G-1 of an m16n8k16 bf16 MMA; S = Q K^T and O += P V run on the tensor cores with
//               fp32 accumulation.  Rows 8..15 of the A operand carry the bf16 rounding residual of
//               rows 0..7 (of the rotated query when RoPE is on, of P always), which costs nothing and
//               gives ~16 mantissa bits.  At the end of an item the four warps merge through shared
//               memory; requests split over several items merge through scratch, last arrival wins.
//   warp 5      summaries: Eq. 6 on the un-rotated query (read from one of two buffers, written to the
//               other, so that every item of a unit sees the old state), and for boundary units the
//               calibrated, rotated summaries q~ in fp64 for the consumers.
//
// All waits are bounded; a wait that gives up sets an error bit and an abort flag that drains the CTA.
#include "gp_dev.cuh"

namespace {

constexpr int NS = 8;                      // tile stages per CTA
constexpr int NI = 4;                      // item slots per CTA
constexpr int NCW = 4;                     // consumer warps
constexpr int NTHREADS = 32 * (NCW + 2);
constexpr int CONS_THREADS = 32 * NCW;

template <int D>
struct Geo {
  static constexpr int ROW_BYTES = D * 2;
  static constexpr int TILE_BYTES = 2 * GP_PAGE * ROW_BYTES;
  static constexpr int KSTEPS = D / 16;
  static constexpr int DTILES = D / 8;
  static constexpr int SLOT_DESC = 128;                                // 32 ints
  static constexpr int SLOT_BYTES = (SLOT_DESC + 8 * ROW_BYTES + 2 * ROW_BYTES + 127) / 128 * 128;
  static constexpr int QT_BYTES = 2 * 8 * D * 8;
  static constexpr int COMB_WARP = (16 + 8 * D) * 4;
  static constexpr int OFF_SLOTS = NS * TILE_BYTES;
  static constexpr int OFF_QT = OFF_SLOTS + NI * SLOT_BYTES;
  static constexpr int OFF_COMB = OFF_QT + QT_BYTES;
  static constexpr int OFF_BARS = OFF_COMB + NCW * COMB_WARP;
  static constexpr int N_BARS = 2 * NS + 2 * NI + 2;
  static constexpr int OFF_MISC = OFF_BARS + N_BARS * 8;
  static constexpr int SMEM_BYTES = OFF_MISC + 64 + 256;
};

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// bounded, abort-aware wait
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < GP_SPIN_LIMIT; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void cons_sync() { asm volatile("bar.sync 1, %0;" ::"n"(CONS_THREADS) : "memory"); }
// barrier over the consumer warps that also ORs a predicate
__device__ __forceinline__ bool cons_any(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, 1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)pred), "n"(CONS_THREADS)
      : "memory");
  return r != 0;
}

template <int D, bool ROPE>
__global__ void __launch_bounds__(NTHREADS, 2)
gp_attn_kernel(const __grid_constant__ GpDev p, int n_req, const __nv_bfloat16* __restrict__ q,
               const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, float* __restrict__ out) {
  using GEO = Geo<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((256u - (smem_u32(smem_raw) & 255u)) & 255u);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + GEO::OFF_BARS);
  uint64_t* full = bars;
  uint64_t* empty = bars + NS;
  uint64_t* slot_full = bars + 2 * NS;
  uint64_t* slot_empty = bars + 2 * NS + NI;
  uint64_t* qt_full = bars + 2 * NS + 2 * NI;
  uint64_t* qt_empty = qt_full + 1;
  volatile int* s_misc = reinterpret_cast<volatile int*>(smem + GEO::OFF_MISC);   // [0] abort, [1] last flag
  double* qt = reinterpret_cast<double*>(smem + GEO::OFF_QT);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.G;
  if (tid == 0) {
    for (int i = 0; i < NS; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < NI; ++i) { mbar_init(&slot_full[i], 1); mbar_init(&slot_empty[i], NCW + 1); }
    mbar_init(qt_full, 1);
    mbar_init(qt_empty, NCW);
    s_misc[0] = 0;
    fence_mbar_init();
  }
  __syncthreads();

  const int n_rc = p.hdr[HDR_N_RC];
  const int LH = p.L * p.Hkv;
  const long long total = (long long)n_rc * LH;
  const int q_bytes = G * GEO::ROW_BYTES;

  if (warp == 0) {
    // ================================= producer ===========================================
    uint32_t fillc = 0;
    for (uint32_t it = 0;; ++it) {
      long long item = 0;
      if (lane == 0) item = atomicAdd(&p.hdr[HDR_WORK_ATTN], 1);
      item = __shfl_sync(0xffffffffu, item, 0);
      const int sl = it % NI;
      if (!wait_bar(&slot_empty[sl], ((it / NI) & 1u) ^ 1u, s_misc)) break;
      uint8_t* slot = smem + GEO::OFF_SLOTS + sl * GEO::SLOT_BYTES;
      int* sd = reinterpret_cast<int*>(slot);
      if (item >= total) {
        if (lane == 0) { sd[3] = -1; }
        __syncwarp();
        if (lane == 0) mbar_arrive(&slot_full[sl]);
        break;
      }
      const int rc_i = (int)(item % n_rc);
      const int lh = (int)(item / n_rc);
      const int l = lh / p.Hkv, h = lh % p.Hkv;
      const int* desc = p.rcx + (size_t)rc_i * GP_DESC_INTS;
      const int w0 = desc[lane];                                  // header words 0..15, pages 0..15
      const int w1 = (lane < GP_DESC_INTS - 32) ? desc[32 + lane] : -1;   // pages 16..31
      const int bi = __shfl_sync(0xffffffffu, w0, 0);
      const int npg = __shfl_sync(0xffffffffu, w0, 3);
      const int chunk = __shfl_sync(0xffffffffu, w0, 4);
      const int nchunks = __shfl_sync(0xffffffffu, w0, 5);
      const int last_pg = (npg - 1 < 16) ? __shfl_sync(0xffffffffu, w0, 16 + ((npg - 1) & 15))
                                         : __shfl_sync(0xffffffffu, w1, (npg - 1 - 16) & 15);
      if (lane < 14) sd[lane] = w0;
      if (lane == 14) sd[14] = lh;
      if (lane == 15) sd[15] = (int)fillc;
      if (lane == 16) sd[16] = last_pg;
      __syncwarp();
      if (lane == 0) {
        const bool has_new = (chunk == nchunks - 1);
        fence_proxy_async();
        mbar_expect_tx(&slot_full[sl], q_bytes + (has_new ? 2 * GEO::ROW_BYTES : 0));
        bulk_g2s(slot + GEO::SLOT_DESC, q + (((size_t)l * n_req + bi) * p.Hq + h * G) * D, q_bytes, &slot_full[sl]);
        if (has_new) {
          const size_t kvo = (((size_t)l * n_req + bi) * p.Hkv + h) * D;
          bulk_g2s(slot + GEO::SLOT_DESC + 8 * GEO::ROW_BYTES, k + kvo, GEO::ROW_BYTES, &slot_full[sl]);
          bulk_g2s(slot + GEO::SLOT_DESC + 9 * GEO::ROW_BYTES, v + kvo, GEO::ROW_BYTES, &slot_full[sl]);
        }
      }
      bool ok = true;
      for (int j = 0; j < npg; ++j) {
        const int page = (j < 16) ? __shfl_sync(0xffffffffu, w0, 16 + j) : __shfl_sync(0xffffffffu, w1, j - 16);
        const uint32_t st = fillc % NS;
        if (!wait_bar(&empty[st], ((fillc / NS) & 1u) ^ 1u, s_misc)) { ok = false; break; }
        if (lane == 0) {
          fence_proxy_async();
          mbar_expect_tx(&full[st], GEO::TILE_BYTES);
          bulk_g2s(smem + st * GEO::TILE_BYTES, p.kv + gp_tile_off(p, l, page, h), GEO::TILE_BYTES, &full[st]);
        }
        ++fillc;
      }
      if (!ok) break;
    }
    if (s_misc[0]) {
      // aborted: let the copies already issued land before the CTA goes away
      if (lane == 0) atomicOr(p.err, GP_E_SPIN);
      for (uint32_t f = (fillc > NS ? fillc - NS : 0); f < fillc; ++f)
        for (uint32_t it = 0; it < (1u << 20); ++it)
          if (mbar_try_wait(&full[f % NS], (f / NS) & 1u)) break;
    }
  } else if (warp <= NCW) {
    // ================================= consumers ==========================================
    const int cw = warp - 1;
    const int ctid = tid - 32;
    const float sc = 1.4426950408889634f * rsqrtf((float)D);
    const int row = lane >> 2;
    const int qc = (lane & 3) * 2;
    uint32_t qt_uses = 0;
    float* comb = reinterpret_cast<float*>(smem + GEO::OFF_COMB);
    float* my_comb = comb + cw * (GEO::COMB_WARP / 4);
    for (uint32_t it = 0;; ++it) {
      const int sl = it % NI;
      if (!wait_bar(&slot_full[sl], (it / NI) & 1u, s_misc)) break;
      const uint8_t* slot = smem + GEO::OFF_SLOTS + sl * GEO::SLOT_BYTES;
      const int* sd = reinterpret_cast<const int*>(slot);
      const int npg = sd[3];
      if (npg < 0) break;
      const int bi = sd[0], r = sd[1], pg0 = sd[2], chunk = sd[4], nchunks = sd[5], n_old = sd[6];
      const int flags = sd[8], Pr = sd[9], lh = sd[14];
      const uint32_t stage_base = (uint32_t)sd[15];
      const int l = lh / p.Hkv, h = lh % p.Hkv;
      const int n_new = n_old + 1;
      const bool need_qt = (flags & 1) && (pg0 < Pr - 1);
      const int rc_i_slot = sd[13];

      // ---- query fragments (A operand), rotated when RoPE is on ----------------------------------
      uint32_t qa[GEO::KSTEPS][2];
      uint32_t ql[GEO::KSTEPS][2];
      {
        const bool valid = row < G;
        const uint8_t* qrow = slot + GEO::SLOT_DESC + (valid ? row : 0) * GEO::ROW_BYTES;
#pragma unroll
        for (int kk = 0; kk < GEO::KSTEPS; ++kk) {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int col = kk * 16 + half * 8 + qc;
            uint32_t hi = 0, lo = 0;
            if (valid) {
              if (!ROPE) {
                hi = *reinterpret_cast<const uint32_t*>(qrow + col * 2);
              } else {
                const int j = col % (D / 2);
                const uint32_t w1 = *reinterpret_cast<const uint32_t*>(qrow + j * 2);
                const uint32_t w2 = *reinterpret_cast<const uint32_t*>(qrow + (j + D / 2) * 2);
                const double* cs = p.rope_cs + ((size_t)bi * (D / 2) + j) * 2;
                const float c0 = (float)cs[0], s0 = (float)cs[1], c1 = (float)cs[2], s1 = (float)cs[3];
                float r0, r1;
                if (col < D / 2) {
                  r0 = bf16_lo_f(w1) * c0 - bf16_lo_f(w2) * s0;
                  r1 = bf16_hi_f(w1) * c1 - bf16_hi_f(w2) * s1;
                } else {
                  r0 = bf16_lo_f(w2) * c0 + bf16_lo_f(w1) * s0;
                  r1 = bf16_hi_f(w2) * c1 + bf16_hi_f(w1) * s1;
                }
                hi = pack_bf16(r0, r1);
                lo = pack_bf16(r0 - bf16_lo_f(hi), r1 - bf16_hi_f(hi));
              }
            }
            qa[kk][half] = hi;
            ql[kk][half] = lo;
          }
        }
      }
      if (need_qt) {
        if (!wait_bar(qt_full, qt_uses & 1u, s_misc)) break;
      }

      const bool last_chunk = (chunk == nchunks - 1);
      float o[GEO::DTILES][4];
#pragma unroll
      for (int i = 0; i < GEO::DTILES; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
      float m_run = -INFINITY, l_run = 0.f;
      bool ok = true;

      for (int pgl = cw; pgl < npg; pgl += NCW) {
        const uint32_t fidx = stage_base + (uint32_t)pgl;
        const uint32_t st = fidx % NS;
        if (!wait_bar(&full[st], (fidx / NS) & 1u, s_misc)) ok = false;   // keep the control flow uniform
        uint8_t* tile = smem + st * GEO::TILE_BYTES;
        const int tok0 = (pg0 + pgl) * GP_PAGE;
        const bool has_new = last_chunk && (pgl == npg - 1);
        if (has_new) {
          // append: slot n_old of this page receives k_t, v_t; patch the staged copy too
          const int s = n_old - tok0;
          const int page = sd[16];
          constexpr int CH = D / 8;
          if (lane < 2 * CH) {
            const int isv = lane / CH, c = lane % CH;
            const uint4 val = *reinterpret_cast<const uint4*>(slot + GEO::SLOT_DESC + (8 + isv) * GEO::ROW_BYTES + c * 16);
            const int off = isv * GP_PAGE * GEO::ROW_BYTES + s * GEO::ROW_BYTES + ((c ^ (s & 7)) << 4);
            *reinterpret_cast<uint4*>(tile + off) = val;
            uint8_t* g = reinterpret_cast<uint8_t*>(p.kv + gp_tile_off(p, l, page, h)) + off;
            *reinterpret_cast<uint4*>(g) = val;
            fence_proxy_async();
          }
          if (lane == 0) p.tok[gp_tok_off(p, l, page, h) + s] = sd[7];
          __syncwarp();
        }
        const uint32_t kt = smem_u32(tile);
        const uint32_t vt = kt + GP_PAGE * GEO::ROW_BYTES;

        // S = Q K^T for the 16 tokens of the page
        float s_acc[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i) s_acc[i][0] = s_acc[i][1] = s_acc[i][2] = s_acc[i][3] = 0.f;
        {
          const int token = (lane & 7) + ((lane >> 4) << 3);
          const int csel = (lane >> 3) & 1;
          const uint32_t rowaddr = kt + token * GEO::ROW_BYTES;
#pragma unroll
          for (int kk = 0; kk < GEO::KSTEPS; ++kk) {
            uint32_t b00, b01, b10, b11;
            ldsm_x4(rowaddr + ((((2 * kk + csel) ^ (token & 7))) << 4), b00, b01, b10, b11);
            mma_bf16(s_acc[0], qa[kk][0], ql[kk][0], qa[kk][1], ql[kk][1], b00, b01);
            mma_bf16(s_acc[1], qa[kk][0], ql[kk][0], qa[kk][1], ql[kk][1], b10, b11);
          }
        }
        // online softmax in the log2 domain
        float sv[2][2];
        const int n_valid = has_new ? (n_new - tok0) : GP_PAGE;
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            float x = s_acc[nt][j];
            if (ROPE) x += s_acc[nt][j + 2];
            x *= sc;
            if (nt * 8 + qc + j >= n_valid) x = -INFINITY;
            sv[nt][j] = x;
            mx = fmaxf(mx, x);
          }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);
        const float corr = exp2f(m_run - m_new);
        if (__any_sync(0xffffffffu, corr != 1.f)) {
          l_run *= corr;
#pragma unroll
          for (int i = 0; i < GEO::DTILES; ++i) {
            o[i][0] *= corr; o[i][1] *= corr; o[i][2] *= corr; o[i][3] *= corr;
          }
        }
        m_run = m_new;
        uint32_t pa[4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const float p0 = exp2f(sv[nt][0] - m_new), p1 = exp2f(sv[nt][1] - m_new);
          l_run += p0 + p1;
          const uint32_t hi = pack_bf16(p0, p1);
          pa[nt * 2] = hi;
          pa[nt * 2 + 1] = pack_bf16(p0 - bf16_lo_f(hi), p1 - bf16_hi_f(hi));
        }
        // O += P V
        {
          const int token = (lane & 7) + (((lane >> 3) & 1) << 3);
          const int csel = lane >> 4;
          const uint32_t rowaddr = vt + token * GEO::ROW_BYTES;
#pragma unroll
          for (int jd = 0; jd < GEO::DTILES; jd += 2) {
            uint32_t v0, v1, v2, v3;
            ldsm_x4_t(rowaddr + (((jd + csel) ^ (token & 7)) << 4), v0, v1, v2, v3);
            mma_bf16(o[jd], pa[0], pa[1], pa[2], pa[3], v0, v1);
            mma_bf16(o[jd + 1], pa[0], pa[1], pa[2], pa[3], v2, v3);
          }
        }
        // boundary unit: fp64 logits of the calibrated summaries against the 16 keys of a candidate page
        if (need_qt && (pg0 + pgl) < Pr - 1) {
          constexpr int CH = D / 8;
          const int t = lane & 15, x = lane >> 4;
          double acc[8];
#pragma unroll
          for (int g = 0; g < 8; ++g) acc[g] = 0.0;
          const uint8_t* krow = tile + t * GEO::ROW_BYTES;
#pragma unroll 2
          for (int c = 0; c < CH; ++c) {
            const uint4 kk = *reinterpret_cast<const uint4*>(krow + ((c ^ (t & 7)) << 4));
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
          const double sqrt_d = sqrt((double)D);
          const long long zoff = ((long long)(unsigned)sd[10]) | ((long long)sd[11] << 32);
          double* zrow = p.zbuf + (((size_t)lh * p.max_batch_tokens + zoff + tok0 + t) * 2 + x) * G;
#pragma unroll
          for (int g = 0; g < 8; ++g)
            if (g < G) zrow[g] = acc[g] / sqrt_d;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[st]);
      }
      // ---- merge the consumer warps ------------------------------------------------------------
      l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
      l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
      cons_sync();                      // everyone is done reading the previous item's merge buffer
      if (row < G) {
        if ((lane & 3) == 0) { my_comb[row] = m_run; my_comb[8 + row] = l_run; }
#pragma unroll
        for (int jd = 0; jd < GEO::DTILES; ++jd) {
          my_comb[16 + row * D + jd * 8 + qc] = o[jd][0] + o[jd][2];
          my_comb[16 + row * D + jd * 8 + qc + 1] = o[jd][1] + o[jd][3];
        }
      }
      cons_sync();
      const size_t out_row0 = (((size_t)l * n_req + bi) * p.Hq + h * G) * D;
      const int PSTRIDE = G * (D + 2);
      const int rc_i = rc_i_slot;
      float* part = p.partials + ((size_t)lh * n_rc + rc_i) * PSTRIDE;
      for (int idx = ctid; idx < G * D; idx += CONS_THREADS) {
        const int g = idx / D, dc = idx % D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NCW; ++w) M = fmaxf(M, comb[w * (GEO::COMB_WARP / 4) + g]);
        float acc = 0.f, ls = 0.f;
#pragma unroll
        for (int w = 0; w < NCW; ++w) {
          const float* base = comb + w * (GEO::COMB_WARP / 4);
          const float wgt = exp2f(base[g] - M);
          acc += wgt * base[16 + g * D + dc];
          ls += wgt * base[8 + g];
        }
        if (nchunks == 1) {
          out[out_row0 + idx] = acc / ls;
        } else {
          part[g * (D + 2) + dc] = acc;
          if (dc == 0) { part[g * (D + 2) + D] = M; part[g * (D + 2) + D + 1] = ls; }
        }
      }
      if (nchunks > 1) {
        __threadfence();
        cons_sync();
        if (ctid == 0) {
          int* cnt = p.unit_cnt + (size_t)bi * LH + lh;
          const int prev = atomicAdd(cnt, 1);
          s_misc[1] = (prev == nchunks - 1);
          if (prev == nchunks - 1) *cnt = 0;
        }
        cons_sync();
        if (s_misc[1]) {
          __threadfence();
          const float* first = p.partials + ((size_t)lh * n_rc + (rc_i - chunk)) * PSTRIDE;
          for (int idx = ctid; idx < G * D; idx += CONS_THREADS) {
            const int g = idx / D, dc = idx % D;
            float M = -INFINITY;
            for (int c = 0; c < nchunks; ++c) M = fmaxf(M, __ldcg(first + (size_t)c * PSTRIDE + g * (D + 2) + D));
            float acc = 0.f, ls = 0.f;
            for (int c = 0; c < nchunks; ++c) {
              const float* pc = first + (size_t)c * PSTRIDE + g * (D + 2);
              const float wgt = exp2f(__ldcg(pc + D) - M);
              acc += wgt * __ldcg(pc + dc);
              ls += wgt * __ldcg(pc + D + 1);
            }
            out[out_row0 + idx] = acc / ls;
          }
        }
      }
      if (need_qt) {
        ++qt_uses;
        __syncwarp();
        if (lane == 0) mbar_arrive(qt_empty);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&slot_empty[sl]);
      if (cons_any(!ok || s_misc[0] != 0)) break;        // same verdict in all four warps
    }
  } else {
    // ================================= summaries ==========================================
    uint32_t qt_uses = 0;
    constexpr int PER = D / 32;
    for (uint32_t it = 0;; ++it) {
      const int sl = it % NI;
      if (!wait_bar(&slot_full[sl], (it / NI) & 1u, s_misc)) break;
      const uint8_t* slot = smem + GEO::OFF_SLOTS + sl * GEO::SLOT_BYTES;
      const int* sd = reinterpret_cast<const int*>(slot);
      const int npg = sd[3];
      if (npg < 0) break;
      const int bi = sd[0], r = sd[1], pg0 = sd[2], chunk = sd[4];
      const int flags = sd[8], Pr = sd[9], par = sd[12], started = (flags >> 1) & 1;
      const int lh = sd[14];
      const int l = lh / p.Hkv, h = lh % p.Hkv;
      const bool need_qt = (flags & 1) && (pg0 < Pr - 1);
      if (chunk == 0 || need_qt) {
        if (need_qt) {
          if (!wait_bar(qt_empty, (qt_uses & 1u) ^ 1u, s_misc)) break;
        }
        for (int g = 0; g < G; ++g) {
          const int head = h * G + g;
          const __nv_bfloat16* qrow = reinterpret_cast<const __nv_bfloat16*>(slot + GEO::SLOT_DESC + g * GEO::ROW_BYTES);
          double qv[PER];
          double sq = 0.0;
#pragma unroll
          for (int e = 0; e < PER; ++e) {
            qv[e] = (double)__bfloat162float(qrow[lane + 32 * e]);
            sq += qv[e] * qv[e];
          }
#pragma unroll
          for (int x = 0; x < 2; ++x) {
            const double beta = x ? p.beta_l : p.beta_s;
            const double* oldp = p.summ + gp_summ_off(p, l, r, par, x, head);
            double* newp = p.summ + gp_summ_off(p, l, r, par ^ 1, x, head);
            double nv[PER];
            double ss = 0.0;
#pragma unroll
            for (int e = 0; e < PER; ++e) {
              nv[e] = started ? beta * oldp[lane + 32 * e] + (1.0 - beta) * qv[e] : qv[e];     // Eq. 6
              if (chunk == 0) newp[lane + 32 * e] = nv[e];
              ss += nv[e] * nv[e];
            }
            if (need_qt) {
              double sq2 = sq;
#pragma unroll
              for (int o2 = 16; o2 > 0; o2 >>= 1) {
                sq2 += __shfl_xor_sync(0xffffffffu, sq2, o2);
                ss += __shfl_xor_sync(0xffffffffu, ss, o2);
              }
              // Eq. 12
              const double gamma = ss > 0.0 ? sqrt(sq2 / (double)D) / sqrt(ss / (double)D) : 1.0;
              double* dst = qt + (x * 8 + g) * D;
              if (p.rope_theta != 0.0) {
                const double* cs = p.rope_cs + (size_t)bi * (D / 2) * 2;
#pragma unroll
                for (int e = 0; e < PER / 2; ++e) {
                  const int j = lane + 32 * e;
                  const double co = cs[2 * j], si = cs[2 * j + 1];
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
        if (need_qt) {
          ++qt_uses;
          __syncwarp();
          if (lane == 0) mbar_arrive(qt_full);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&slot_empty[sl]);
    }
  }
  __syncthreads();
}

}  // namespace

size_t gp_attention_smem(int d) { return d == 128 ? Geo<128>::SMEM_BYTES : Geo<64>::SMEM_BYTES; }
int gp_attention_ctas_per_sm(int d) { (void)d; return 2; }

void gp_launch_attention(const GpDev& p, const int* req_ids, int n_req, const void* q, const void* k, const void* v,
                         float* out, int grid, cudaStream_t s) {
  (void)req_ids;
  const __nv_bfloat16* qq = static_cast<const __nv_bfloat16*>(q);
  const __nv_bfloat16* kk = static_cast<const __nv_bfloat16*>(k);
  const __nv_bfloat16* vv = static_cast<const __nv_bfloat16*>(v);
  const bool rope = p.rope_theta != 0.0;
#define GP_LAUNCH(DD, RR)                                                                              \
  do {                                                                                                 \
    auto kern = gp_attn_kernel<DD, RR>;                                                                \
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<DD>::SMEM_BYTES);      \
    kern<<<grid, NTHREADS, Geo<DD>::SMEM_BYTES, s>>>(p, n_req, qq, kk, vv, out);                      \
  } while (0)
  if (p.d == 128) {
    if (rope) GP_LAUNCH(128, true); else GP_LAUNCH(128, false);
  } else {
    if (rope) GP_LAUNCH(64, true); else GP_LAUNCH(64, false);
  }
#undef GP_LAUNCH
}
