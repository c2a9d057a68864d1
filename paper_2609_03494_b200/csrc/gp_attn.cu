// Fused append + GQA paged decode attention + dual EMA summary update (Sec. 3.2 Eq. 6, Sec. 4.1).
//
// Work decomposition.  The plan kernel cuts every stepped request into chunks of `chunk_pages`
// pages; one work item is (chunk, layer, KV head).  A persistent grid (a multiple of the SM
// count) pulls items from a global counter.  Inside a CTA the four warps take the pages of the
// item round-robin, each through its own ring of bulk-copy stages: one `cp.async.bulk` brings the
// contiguous K|V tile of a (layer, page, head) into shared memory and signals an mbarrier.
//
// Arithmetic.  The G query heads of the group are the rows of an m16n8k16 bf16 MMA (rows G..7
// are zero); S = Q K^T and O += P V run on the tensor cores with fp32 accumulation.  Rows 8..15
// of the A operand carry the bf16 rounding residual of rows 0..7 (of the rotated query when RoPE
// is on, and of the probabilities P always), so the tile's unused half buys ~16 mantissa bits.
//
// The item that holds the request's last page also appends the new token (writes k_t, v_t and
// the token index to the pool and patches the staged tile); the item of chunk 0 updates the two
// summaries.  Split requests leave partial (max, sum, O) in scratch; the last CTA to arrive for a
// (request, layer, head) merges them.
#include "gp_dev.cuh"

namespace {

template <int D>
struct AttnGeom {
  static constexpr int ROW_BYTES = D * 2;
  static constexpr int TILE_BYTES = 2 * GP_PAGE * ROW_BYTES;
  static constexpr int KSTEPS = D / 16;
  static constexpr int DTILES = D / 8;
  static constexpr int STAGE_BYTES = GP_ATTN_WARPS * GP_ATTN_STAGES * TILE_BYTES;
  static constexpr int SMEM_BYTES = STAGE_BYTES + GP_ATTN_WARPS * GP_ATTN_STAGES * 8 + 64 * 4 + 16 * 4 + 256;
};

template <int D, bool ROPE>
__global__ void __launch_bounds__(GP_ATTN_WARPS * 32, (D == 128 ? 2 : 4))
gp_attn_kernel(const __grid_constant__ GpDev p, const int* __restrict__ req_ids, int n_req,
               const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
               const __nv_bfloat16* __restrict__ v, float* __restrict__ out) {
  using GEO = AttnGeom<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((256u - (smem_u32(smem_raw) & 255u)) & 255u);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + GEO::STAGE_BYTES);
  int* s_pages = reinterpret_cast<int*>(bars + GP_ATTN_WARPS * GP_ATTN_STAGES);
  int* s_misc = s_pages + 64;   // [0] item, [1] abort, [2] last-arriver flag

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.G;
  if (tid == 0) {
    for (int i = 0; i < GP_ATTN_WARPS * GP_ATTN_STAGES; ++i) mbar_init(&bars[i], 1);
    s_misc[1] = 0;
    fence_mbar_init();
  }
  __syncthreads();

  uint8_t* my_stage = smem + warp * GP_ATTN_STAGES * GEO::TILE_BYTES;
  uint64_t* my_bar = bars + warp * GP_ATTN_STAGES;
  uint32_t fill = 0, cons = 0;   // lifetime counts of copies issued / tiles consumed by this warp
  const float sc = 1.4426950408889634f * rsqrtf((float)D);
  const int n_rc = p.hdr[HDR_N_RC];
  const int LH = p.L * p.Hkv;
  const long long total = (long long)n_rc * LH;
  const int row = lane >> 2;          // query head of the group held by this lane's fragments
  const int qc = (lane & 3) * 2;      // column pair inside an 8-wide fragment

  for (;;) {
    __syncthreads();
    if (tid == 0) s_misc[0] = atomicAdd(&p.hdr[HDR_WORK_ATTN], 1);
    __syncthreads();
    const long long item = s_misc[0];
    if (item >= total || s_misc[1]) break;
    const int rc_i = (int)(item % n_rc);
    const int lh = (int)(item / n_rc);
    const int l = lh / p.Hkv, h = lh % p.Hkv;
    const int4 e = p.rc[rc_i];
    const int bi = e.x, pg0 = e.y, npg = e.z, chunk = e.w & 0xffff, nchunks = e.w >> 16;
    const int r = req_ids[bi];
    const int n_old = p.b_nold[bi];
    const int n_new = n_old + 1;
    if (tid < npg) s_pages[tid] = p.page_table[(size_t)r * p.cap + pg0 + tid];
    __syncthreads();

    // ---- query fragments (A operand), rotated when RoPE is on --------------------------------
    uint32_t qa[GEO::KSTEPS][2];
    uint32_t ql[GEO::KSTEPS][2];
    {
      const bool valid = row < G;
      const __nv_bfloat16* qrow = q + (((size_t)l * n_req + bi) * p.Hq + h * G + (valid ? row : 0)) * D;
#pragma unroll
      for (int kk = 0; kk < GEO::KSTEPS; ++kk) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int col = kk * 16 + half * 8 + qc;
          uint32_t hi = 0, lo = 0;
          if (valid) {
            if (!ROPE) {
              hi = *reinterpret_cast<const uint32_t*>(qrow + col);
            } else {
              const int j = col % (D / 2);
              const uint32_t w1 = *reinterpret_cast<const uint32_t*>(qrow + j);
              const uint32_t w2 = *reinterpret_cast<const uint32_t*>(qrow + j + D / 2);
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

    // ---- summaries: the item of chunk 0 applies Eq. 6 to the un-rotated query -------------------
    if (chunk == 0) {
      const int started = p.started[r];
      for (int idx = tid; idx < G * D; idx += GP_ATTN_WARPS * 32) {
        const int g = idx / D, dd = idx % D;
        const double qv = (double)__bfloat162float(q[(((size_t)l * n_req + bi) * p.Hq + h * G + g) * D + dd]);
        double* ps = p.summ + gp_summ_off(p, l, r, 0, h * G + g) + dd;
        double* pl = p.summ + gp_summ_off(p, l, r, 1, h * G + g) + dd;
        if (!started) {
          *ps = qv;
          *pl = qv;
        } else {
          *ps = p.beta_s * (*ps) + (1.0 - p.beta_s) * qv;
          *pl = p.beta_l * (*pl) + (1.0 - p.beta_l) * qv;
        }
      }
    }

    // ---- stream the pages of this warp ---------------------------------------------------------
    const int my_cnt = (npg > warp) ? (npg - warp + GP_ATTN_WARPS - 1) / GP_ATTN_WARPS : 0;
    const bool last_chunk = (chunk == nchunks - 1);
    float o[GEO::DTILES][4];
#pragma unroll
    for (int i = 0; i < GEO::DTILES; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;

    int issued = 0;
    auto issue = [&](int jj) {
      const int page = s_pages[warp + jj * GP_ATTN_WARPS];
      const uint32_t st = fill % GP_ATTN_STAGES;
      if (lane == 0) {
        fence_proxy_async();
        mbar_expect_tx(&my_bar[st], GEO::TILE_BYTES);
        bulk_g2s(my_stage + st * GEO::TILE_BYTES, p.kv + gp_tile_off(p, l, page, h), GEO::TILE_BYTES, &my_bar[st]);
      }
      ++fill;
    };
    for (; issued < my_cnt && issued < GP_ATTN_STAGES; ++issued) issue(issued);

    for (int jj = 0; jj < my_cnt; ++jj) {
      const uint32_t st = cons % GP_ATTN_STAGES;
      const uint32_t parity = (cons / GP_ATTN_STAGES) & 1u;
      if (!mbar_wait(&my_bar[st], parity)) {
        if (lane == 0) { atomicOr(p.err, GP_E_SPIN); s_misc[1] = 1; }
      }
      ++cons;
      uint8_t* tile = my_stage + st * GEO::TILE_BYTES;
      const int pgl = warp + jj * GP_ATTN_WARPS;          // page index inside the item
      const int tok0 = (pg0 + pgl) * GP_PAGE;             // first slot of this page
      const bool has_new = last_chunk && (pgl == npg - 1);
      if (has_new) {
        // append: slot n_old of this page receives k_t, v_t; patch the staged copy too
        const int s = n_old - tok0;
        const int page = s_pages[pgl];
        constexpr int CH = D / 8;   // 16-byte chunks per row
        if (lane < 2 * CH) {
          const int isv = lane / CH, c = lane % CH;
          const __nv_bfloat16* src = (isv ? v : k) + (((size_t)l * n_req + bi) * p.Hkv + h) * D + c * 8;
          const uint4 val = *reinterpret_cast<const uint4*>(src);
          const int off = isv * GP_PAGE * GEO::ROW_BYTES + s * GEO::ROW_BYTES + ((c ^ (s & 7)) << 4);
          *reinterpret_cast<uint4*>(tile + off) = val;
          uint8_t* g = reinterpret_cast<uint8_t*>(p.kv + gp_tile_off(p, l, page, h)) + off;
          *reinterpret_cast<uint4*>(g) = val;
          fence_proxy_async();
        }
        if (lane == 0) p.tok[gp_tok_off(p, l, page, h) + s] = (int)p.pos[r];
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
      __syncwarp();
      if (issued < my_cnt) { issue(issued); ++issued; }
    }

    // ---- merge the warps of the CTA -------------------------------------------------------------
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    {
      float* pm = reinterpret_cast<float*>(my_stage);
      float* pl = pm + 8;
      float* po = pm + 16;
      if (row < G) {
        if ((lane & 3) == 0) { pm[row] = m_run; pl[row] = l_run; }
#pragma unroll
        for (int jd = 0; jd < GEO::DTILES; ++jd) {
          po[row * D + jd * 8 + qc] = o[jd][0] + o[jd][2];
          po[row * D + jd * 8 + qc + 1] = o[jd][1] + o[jd][3];
        }
      }
    }
    fence_proxy_async();   // these generic writes precede the next item's bulk copies into the stages
    __syncthreads();
    const size_t out_row0 = (((size_t)l * n_req + bi) * p.Hq + h * G) * D;
    const int PSTRIDE = G * (D + 2);
    float* part = p.partials + ((size_t)lh * n_rc + rc_i) * PSTRIDE;
    for (int idx = tid; idx < G * D; idx += GP_ATTN_WARPS * 32) {
      const int g = idx / D, dc = idx % D;
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < GP_ATTN_WARPS; ++w)
        M = fmaxf(M, reinterpret_cast<float*>(smem + w * GP_ATTN_STAGES * GEO::TILE_BYTES)[g]);
      float acc = 0.f, ls = 0.f;
#pragma unroll
      for (int w = 0; w < GP_ATTN_WARPS; ++w) {
        const float* base = reinterpret_cast<float*>(smem + w * GP_ATTN_STAGES * GEO::TILE_BYTES);
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
      __syncthreads();
      if (tid == 0) {
        int* cnt = p.unit_cnt + (size_t)bi * LH + lh;
        const int prev = atomicAdd(cnt, 1);
        s_misc[2] = (prev == nchunks - 1);
        if (prev == nchunks - 1) *cnt = 0;
      }
      __syncthreads();
      if (s_misc[2]) {
        __threadfence();
        const float* first = p.partials + ((size_t)lh * n_rc + (rc_i - chunk)) * PSTRIDE;
        for (int idx = tid; idx < G * D; idx += GP_ATTN_WARPS * 32) {
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
  }
}

}  // namespace

size_t gp_attention_smem(int d) { return d == 128 ? AttnGeom<128>::SMEM_BYTES : AttnGeom<64>::SMEM_BYTES; }
int gp_attention_ctas_per_sm(int d) { return d == 128 ? 2 : 4; }

void gp_launch_attention(const GpDev& p, const int* req_ids, int n_req, const void* q, const void* k, const void* v,
                         float* out, int grid, cudaStream_t s) {
  const __nv_bfloat16* qq = static_cast<const __nv_bfloat16*>(q);
  const __nv_bfloat16* kk = static_cast<const __nv_bfloat16*>(k);
  const __nv_bfloat16* vv = static_cast<const __nv_bfloat16*>(v);
  const bool rope = p.rope_theta != 0.0;
  const int threads = GP_ATTN_WARPS * 32;
#define GP_LAUNCH(DD, RR)                                                                                   \
  do {                                                                                                      \
    auto kern = gp_attn_kernel<DD, RR>;                                                                     \
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnGeom<DD>::SMEM_BYTES);      \
    kern<<<grid, threads, AttnGeom<DD>::SMEM_BYTES, s>>>(p, req_ids, n_req, qq, kk, vv, out);              \
  } while (0)
  if (p.d == 128) {
    if (rope) GP_LAUNCH(128, true); else GP_LAUNCH(128, false);
  } else {
    if (rope) GP_LAUNCH(64, true); else GP_LAUNCH(64, false);
  }
#undef GP_LAUNCH
}
