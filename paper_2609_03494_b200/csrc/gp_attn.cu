// Fused append + GQA paged decode attention (Sec. 4.1), plus, for requests that reach their capacity boundary
// with this step, the logits of the two calibrated summaries against every candidate key (Eq. 12, App. D.1)
// while the key tile is in shared memory.  (The summaries themselves, Eq. 6, and the calibrated q~ are updated
// by the plan kernel's summary CTAs before this kernel starts.)
//
// Work decomposition.  The plan kernel cuts every stepped request into chunks of `chunk_pages` pages and
// writes one descriptor per chunk, sorted by descending cost; a work item is (chunk, layer, KV head).  A
// persistent grid (two CTAs per SM) deals the items out round by round, alternating the CTA order so that
// every CTA gets about the same total.  Each CTA is warp-specialised:
//
//   warp 0      producer: takes its items (a static deal of the cost-sorted list) and publishes each in a ring
//               of item slots: descriptor, query rows (and the new key/value row) by bulk copy, page ids.  For
//               boundary items it also brings q~ into the CTA's single q~ buffer.
//   warps 4..7  consumers: take the tiles of an item round-robin (tile j belongs to warp (j - item number) mod 4,
//               so the odd tiles of successive items fall on different warps).  Each warp
//               fetches its own K|V tiles (one contiguous 8 KB per (layer, page, head)) with 16-byte
//               asynchronous copies into a private ring of stages, running ahead across item boundaries, so
//               the ring never drains between items.  The G query heads of the group are rows 0..G-1 of an
//               m16n8k16 bf16 MMA; S = Q K^T and O += P V run on the tensor cores with fp32 accumulation.
//               Rows 8..15 of the A operand carry the bf16 rounding residual of rows 0..7 (of the rotated
//               query when RoPE is on, of P always), which costs nothing and gives ~16 mantissa bits.  For
//               boundary units the summary logits of a candidate page are an fp64 tensor-core contraction
//               (m8n8k4 DMMA: 8 tokens x (2 views x G heads) x d).
//   warp 2      merger: combines the four consumers' partial (max, sum, O) of an item and writes the output
//               or, for requests split over several items, the partial (the next kernel merges those).
//               Consumers hand over through a double buffer and go straight on to the next item.
//   warps 1, 3  idle.
//
// The two warp groups re-split the register file (setmaxnreg): the service warps keep 56 registers per
// thread, the consumers, which hold the output accumulators, get 200.
// All waits are bounded; a wait that gives up sets an error bit (with a code for which wait it was) and an
// abort flag that drains the CTA.  No wait of an item depends on a later item being published.
#include "gp_dev.cuh"

namespace {

constexpr int NI_MAX = 8;                  // item slots per CTA (4 when the group is 8 heads wide)
constexpr int NSW = 2;                     // tile stages per consumer warp (at most 3: see the wait in the tile loop)
constexpr int NCW = 4;                     // consumer warps
constexpr int NTHREADS = 256;              // warp group 0: producer, idle, merger, idle; warp group 1: consumers
constexpr int REGS_SERVICE = 56;           // registers per thread after the split (setmaxnreg)
constexpr int REGS_CONSUMER = 200;
constexpr int QT_PAD = 8;                  // doubles of padding per q~ row: rows alternate bank halves

template <int D>
struct Geo {
  static constexpr int ROW_BYTES = D * 2;
  static constexpr int TILE_BYTES = 2 * GP_PAGE * ROW_BYTES;
  static constexpr int KSTEPS = D / 16;
  static constexpr int DTILES = D / 8;
  static constexpr int SLOT_DESC = 384;                                // 96 ints: descriptor (32), then up to 64 page ids
  static constexpr int SLOT_PAGES = 32;                                // first page id (int index)
  static constexpr int SLOT_BYTES = (SLOT_DESC + 8 * ROW_BYTES + 2 * ROW_BYTES + 127) / 128 * 128;
};

struct Lay {            // shared-memory layout, depends on the group size
  int ni, ncomb, off_slots, off_qt, off_comb, comb_warp, off_bars, off_misc, total;
};
template <int D>
__host__ __device__ inline Lay make_lay(int G) {
  using GEO = Geo<D>;
  Lay L;
  const bool wide = (D == 128 && G == 8);
  L.ni = wide ? 4 : NI_MAX;
  L.ncomb = wide ? 1 : 2;
  L.off_slots = NCW * NSW * GEO::TILE_BYTES;
  L.off_qt = L.off_slots + L.ni * GEO::SLOT_BYTES;
  const int nrows = 2 * G < 8 ? 8 : 2 * G;
  L.off_comb = L.off_qt + nrows * (D + QT_PAD) * 8;
  L.comb_warp = (16 + G * D) * 4;
  L.off_bars = L.off_comb + L.ncomb * NCW * L.comb_warp;
  L.off_misc = L.off_bars + (2 * NCW * NSW + 2 * NI_MAX + 2 + 4) * 8;
  L.total = L.off_misc + 128 + 256;          // abort flag and code, then the queue of q~ copies
  return L;
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// bounded, abort-aware wait
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int where, uint32_t limit) {
  for (uint32_t it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u && *abort_flag) return false;
  }
  if (*abort_flag == 0) abort_flag[1] = where;      // which wait gave up first (reported with the error bit)
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void dmma(double& d0, double& d1, double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(d0), "+d"(d1)
               : "d"(a), "d"(b));
}

template <int D, bool ROPE>
__global__ void __launch_bounds__(NTHREADS, 2)
gp_attn_kernel(const __grid_constant__ GpDev p, int n_req, const __nv_bfloat16* __restrict__ q,
               const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, float* __restrict__ out, int lh0,
               int lh_n, int adv_lh) {
  // lh0, lh_n: the (layer, KV head) units this launch covers, [lh0, lh0 + lh_n): all of them, or one layer's
  // adv_lh: the unit whose append also moves the request's counters on by one token (-1: none; the layer-by-layer
  // step does that at its end)
  using GEO = Geo<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((256u - (smem_u32(smem_raw) & 255u)) & 255u);
  const int G = p.G;
  const Lay L = make_lay<D>(G);
  const uint32_t NI = (uint32_t)L.ni, NCOMB = (uint32_t)L.ncomb;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L.off_bars);
  uint64_t* slot_full = bars + 2 * NCW * NSW;  // [NI]
  uint64_t* slot_empty = slot_full + NI_MAX;   // [NI]
  uint64_t* qt_full = slot_empty + NI_MAX;
  uint64_t* qt_empty = qt_full + 1;
  uint64_t* comb_full = qt_empty + 1;          // [2]
  uint64_t* comb_empty = comb_full + 2;        // [2]
  volatile int* s_misc = reinterpret_cast<volatile int*>(smem + L.off_misc);   // [0] abort
  double* qt = reinterpret_cast<double*>(smem + L.off_qt);                     // [2G][D + QT_PAD]
  float* comb = reinterpret_cast<float*>(smem + L.off_comb);                   // [2][NCW][16 + G*D]
  const int comb_w = L.comb_warp / 4;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t lim = p.spin_limit;
  if (tid == 0) {
    for (int i = 0; i < NI_MAX; ++i) { mbar_init(&slot_full[i], 2); mbar_init(&slot_empty[i], NCW + 1); }
    mbar_init(qt_full, 1);
    mbar_init(qt_empty, NCW);
    for (int i = 0; i < 2; ++i) { mbar_init(&comb_full[i], NCW); mbar_init(&comb_empty[i], 1); }
    s_misc[0] = 0;
    s_misc[1] = 0;
    fence_mbar_init();
  }
  gp_pdl_wait();                  // everything above touched only this CTA's shared memory
  gp_pdl_launch_dependents();
  __syncthreads();

  const int n_rc = p.hdr[HDR_N_RC];
  const int LH = p.L * p.Hkv;
  const long long total = (long long)n_rc * lh_n;
  const int q_bytes = G * GEO::ROW_BYTES;

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_SERVICE));
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_CONSUMER));
  }
  if (warp == 0) {
    // ================================= producer ===========================================
    // Software pipeline over items, one stage per tick, so that no global round trip of one item delays
    // another: A = item known, descriptor header load issued; B = header here: the slot is claimed, the
    // descriptor written, the query rows (and the new key/value row) copied in, the page ids requested;
    // C = page ids here: written to the slot, which completes its `full` barrier (two arrivals: B and C, plus
    // the bytes of B's copies).  The ring of slots paces the producer: it runs NI items ahead at most.
    const long long grid = gridDim.x;
    // static schedule: items are sorted by descending cost; round k goes to the CTAs in alternating order
    auto item_of_tick = [&](long long kk) -> long long {
      const long long item = kk * grid + ((kk & 1) ? grid - 1 - (long long)blockIdx.x : (long long)blockIdx.x);
      return item < total ? item : total;
    };
    long long itA = item_of_tick(0), itB = total, itC = total;
    int hB = 0, hC = 0;                        // descriptor header, word `lane` (lanes 0..15)
    int pC = -1, pC2 = -1;                     // page ids of tiles `lane` and `lane + 32` of the item
    int slC = 0;                               // slot of the item in stage C
    uint32_t n_pub = 0, n_comp = 0;          // items published (stage B), items completed (stage C)
    bool sentinel_out = false;
    // The q~ buffer is single: the copy for a boundary item is issued once the consumers are done with the
    // previous boundary item.  The producer never blocks on that (it would hold back the slots of other
    // items, possibly of the very item the consumers have to finish first): copies wait in a queue (never
    // more entries than item slots) and are issued from the polls below, oldest first.
    volatile int* qt_queue = s_misc + 16;          // [NI_MAX][2]: batch slot, layer/head
    uint32_t qt_head = 0, qt_tail = 0;              // qt_head = copies issued so far
    auto poll_qt = [&]() {
      if (qt_head != qt_tail && mbar_test_wait(qt_empty, (qt_head & 1u) ^ 1u)) {
        if (lane == 0) {
          const int qbi = qt_queue[(qt_head % NI_MAX) * 2], qlh = qt_queue[(qt_head % NI_MAX) * 2 + 1];
          fence_proxy_async();
          mbar_expect_tx(qt_full, 2 * G * D * 8);
          const double* src = p.qtil + ((size_t)qbi * LH + qlh) * 2 * G * D;
          for (int row2 = 0; row2 < 2 * G; ++row2)
            bulk_g2s(qt + (size_t)row2 * (D + QT_PAD), src + (size_t)row2 * D, D * 8, qt_full);
        }
        ++qt_head;
      }
    };
    auto wait_polling = [&](uint64_t* bar, uint32_t parity) -> bool {     // bounded, abort-aware, keeps q~ moving
      for (uint32_t w = 0; w < lim; ++w) {
        if (mbar_try_wait(bar, parity)) return true;
        poll_qt();
        if ((w & 63u) == 63u && s_misc[0]) return false;
      }
      if (s_misc[0] == 0) s_misc[1] = 1;
      s_misc[0] = 1;
      return false;
    };
    for (uint32_t tick = 0;; ++tick) {
      // ---- issue the loads of the young stages --------------------------------------------------
      int hNew = 0;
      if (itA < total && lane < GP_DESC_INTS) hNew = p.rcx[(size_t)(itA / lh_n) * GP_DESC_INTS + lane];
      int pNew = -1, pNew2 = -1;
      int slNew = 0;
      // ---- page ids of stage C have arrived: into the slot, which is then complete ----------------------
      if (itC < total) {
        int* sd = reinterpret_cast<int*>(smem + L.off_slots + slC * GEO::SLOT_BYTES);
        sd[GEO::SLOT_PAGES + lane] = pC;
        sd[GEO::SLOT_PAGES + 32 + lane] = pC2;
        __syncwarp();
        // (test support: the first CTA's second item can be withheld, so that the consumers' bounded wait runs out)
        const bool withheld = (p.withhold & GP_WITHHOLD_ITEM) && blockIdx.x == 0 && n_comp == 1;
        ++n_comp;
        if (lane == 0 && !withheld) mbar_arrive(&slot_full[slC]);
      }
      poll_qt();
      // ---- header of stage B has arrived: load its page ids and fill its slot -----------------------
      if (tick >= 1 && !sentinel_out) {
        const int sl = n_pub % NI;
        slNew = sl;
        if (!wait_polling(&slot_empty[sl], ((n_pub / NI) & 1u) ^ 1u)) break;
        uint8_t* slot = smem + L.off_slots + sl * GEO::SLOT_BYTES;
        int* sd = reinterpret_cast<int*>(slot);
        if (itB >= total) {
          if (lane == 0) sd[3] = -1;
          __syncwarp();
          if (lane == 0) { mbar_arrive(&slot_full[sl]); mbar_arrive(&slot_full[sl]); }
          sentinel_out = true;
        } else {
          const int lh = lh0 + (int)(itB % lh_n);
          const int l = lh / p.Hkv, h = lh % p.Hkv;
          const int bi = __shfl_sync(0xffffffffu, hB, 0);
          const int r = __shfl_sync(0xffffffffu, hB, 1), pg0 = __shfl_sync(0xffffffffu, hB, 2);
          const int npg = __shfl_sync(0xffffffffu, hB, 3);
          const int chunk = __shfl_sync(0xffffffffu, hB, 4);
          const int nchunks = __shfl_sync(0xffffffffu, hB, 5);
          if (lane < npg) pNew = p.page_table[(size_t)r * p.cap + pg0 + lane];
          if (lane + 32 < npg) pNew2 = p.page_table[(size_t)r * p.cap + pg0 + 32 + lane];
          if (lane < 14) sd[lane] = hB;
          if (lane == 14) sd[14] = lh;
          if (lane == 15) sd[15] = hB;            // index among the step's boundary requests
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
          // boundary unit with candidate pages in this chunk: its calibrated summaries q~ (written by the
          // plan kernel's summary CTAs) go into the single q~ buffer once the previous such item is done
          const int flags = __shfl_sync(0xffffffffu, hB, 8), Pr = __shfl_sync(0xffffffffu, hB, 9);
          if ((flags & 1) && pg0 < Pr - 1) {
            if (lane == 0) { qt_queue[(qt_tail % NI_MAX) * 2] = bi; qt_queue[(qt_tail % NI_MAX) * 2 + 1] = lh; }
            __syncwarp();
            ++qt_tail;
            poll_qt();
          }
        }
        ++n_pub;
      }
      if (sentinel_out && itC >= total) break;
      // ---- rotate -----------------------------------------------------------------------------------------
      itC = itB; hC = hB; pC = pNew; pC2 = pNew2; slC = slNew;
      itB = itA; hB = hNew;
      itA = item_of_tick((long long)tick + 1);
    }
    (void)hC;
    while (qt_head != qt_tail && !s_misc[0]) {           // copies still queued when the last slot is out
      if (!wait_polling(qt_empty, (qt_head & 1u) ^ 1u)) break;
      poll_qt();
    }
  } else if (warp >= 4) {
    // ================================= consumers ==========================================
    const int cw = warp - 4;
    const float sc = 1.4426950408889634f * rsqrtf((float)D);
    const int row = lane >> 2;
    const int qc = (lane & 3) * 2;
    uint32_t qt_uses = 0, my_tiles = 0;
    // Each consumer warp fetches its own tiles (tile j of an item belongs to warp j mod 4) into its private
    // ring of NSW stages: as soon as it is done with a stage it issues the copy of its next tile but NSW - 1,
    // which may belong to a later item (the fetch position runs ahead of the compute position, across item
    // boundaries, but never further than the ring of item slots allows).  No other warp touches the ring, so
    // program order plus a proxy fence orders the reads of a stage before the copy that overwrites it.
    const uint64_t kv_policy = l2_policy_evict_first();    // the K/V stream is read once per step: first out of the L2
    uint32_t my_fetch = 0, f_it = 0;
    int f_pgl = 0, f_npg = 0, f_lh = 0;
    bool f_have = false, f_done = false;
    auto top_up = [&](uint32_t it_now) -> bool {           // false: a wait gave up
      while (!f_done && my_fetch - my_tiles < (uint32_t)NSW) {
        const int* fsd = reinterpret_cast<const int*>(smem + L.off_slots + (f_it % NI) * GEO::SLOT_BYTES);
        if (!f_have) {
          if (f_it + 1 >= it_now + NI) break;              // that slot may still hold an item this warp has not finished
          // an item ahead of the one being computed is fetched from only if its slot is already there:
          // nothing the current item needs may wait for a later item to be published
          if (f_it > it_now) {
            if (!mbar_test_wait(&slot_full[f_it % NI], (f_it / NI) & 1u)) break;
          } else if (!wait_bar(&slot_full[f_it % NI], (f_it / NI) & 1u, s_misc, 3, lim)) {
            return false;
          }
          f_npg = fsd[3];
          if (f_npg < 0) { f_done = true; break; }
          f_lh = fsd[14];
          f_pgl = (cw + f_it) % NCW;                      // the first tile goes to another warp from item to item
          f_have = true;
        }
        if (f_pgl >= f_npg) { ++f_it; f_have = false; continue; }
        const int page = fsd[GEO::SLOT_PAGES + f_pgl];
        const uint32_t fst = cw * NSW + (my_fetch % NSW);
        {
          // 16-byte asynchronous copies through the load/store path, 512 contiguous bytes per warp instruction:
          // the bulk-copy engine takes several hundred cycles to accept an 8 KB copy, which paced the kernel
          const uint8_t* src = reinterpret_cast<const uint8_t*>(p.kv + gp_tile_off(p, f_lh / p.Hkv, page, f_lh % p.Hkv)) + lane * 16;
          const uint32_t dst = smem_u32(smem + fst * GEO::TILE_BYTES) + lane * 16;
#pragma unroll
          for (int c = 0; c < GEO::TILE_BYTES / 512; ++c) cp_async16_hint(dst + c * 512, src + c * 512, kv_policy);
          cp_async_commit();
        }
        ++my_fetch;
        f_pgl += NCW;
      }
      return true;
    };
    for (uint32_t it = 0;; ++it) {
      const int sl = it % NI;
      if (!top_up(it)) break;
      if (!wait_bar(&slot_full[sl], (it / NI) & 1u, s_misc, 4, lim)) break;
      const uint8_t* slot = smem + L.off_slots + sl * GEO::SLOT_BYTES;
      const int* sd = reinterpret_cast<const int*>(slot);
      const int npg = sd[3];
      if (npg < 0) break;
      const int bi = sd[0], pg0 = sd[2], chunk = sd[4], nchunks = sd[5], n_old = sd[6];
      const int flags = sd[8], Pr = sd[9], lh = sd[14];
      const int l = lh / p.Hkv, h = lh % p.Hkv;
      const int n_new = n_old + 1;
      const bool need_qt = (flags & 1) && (pg0 < Pr - 1);

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
        if (!wait_bar(qt_full, qt_uses & 1u, s_misc, 5, lim)) break;
      }

      const bool last_chunk = (chunk == nchunks - 1);
      float o[GEO::DTILES][4];
#pragma unroll
      for (int i = 0; i < GEO::DTILES; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
      float m_run = -INFINITY, l_run = 0.f;
      bool ok = true;

      for (int pgl = (cw + it) % NCW; pgl < npg; pgl += NCW) {
        const uint32_t st = cw * NSW + (my_tiles % NSW);
        {
          // one copy group per tile, in fetch order: all but the groups younger than this tile's must be done
          const uint32_t younger = my_fetch - my_tiles - 1;
          if (younger == 0) cp_async_wait<0>(); else if (younger == 1) cp_async_wait<1>(); else cp_async_wait<2>();
          __syncwarp();
        }
        ++my_tiles;
        uint8_t* tile = smem + st * GEO::TILE_BYTES;
        const int tok0 = (pg0 + pgl) * GP_PAGE;
        const bool has_new = last_chunk && (pgl == npg - 1);
        if (has_new) {
          // append: slot n_old of this page receives k_t, v_t; patch the staged copy too
          const int s = n_old - tok0;
          const int page = sd[GEO::SLOT_PAGES + npg - 1];
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
          if (lane == 1 && lh == adv_lh) {
            // the request is one token further; the summary CTAs of this step have written the buffer not in use
            // (the plan kernel had completed before this kernel passed its wait)
            const int r = sd[1];
            p.n[r] = n_new; p.pos[r] = (long long)sd[7] + 1; p.started[r] = 1; p.sum_par[r] = sd[12] ^ 1;
          }
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
        // Boundary unit: fp64 logits of the calibrated summaries against the 16 keys of a candidate page,
        // Z[token][n] = sum_d K[token][d] q~[n][d], n = view * G + head.  One m8n8k4 DMMA covers 8 tokens,
        // 8 columns and 4 values of d; inside a 16-byte chunk of a key row lane t of a quad takes the
        // bf16 pair at byte 4t, whose low and high element feed two successive k-steps (q~ is read with
        // the same mapping, so the contraction is over the same d on both sides).
        if (need_qt && (pg0 + pgl) < Pr - 1) {
          constexpr int CH = D / 8;
          const int grp = lane >> 2, t4 = lane & 3;
          const int n_tiles = (2 * G + 7) / 8;
          const double sqrt_d = sqrt((double)D);
          const long long zoff = ((long long)(unsigned)sd[10]) | ((long long)sd[11] << 32);
          for (int nt = 0; nt < n_tiles; ++nt) {
            const int n = nt * 8 + grp;                           // B column held by this lane's group
            const bool ncol = n < 2 * G;
            const double* qrow = qt + (size_t)(ncol ? n : 0) * (D + QT_PAD) + 2 * t4;
            double z00 = 0.0, z01 = 0.0, z10 = 0.0, z11 = 0.0;    // [m-tile][column pair], even chunks
            double y00 = 0.0, y01 = 0.0, y10 = 0.0, y11 = 0.0;    // odd chunks: four independent DMMA chains
            const uint8_t* krow0 = tile + grp * GEO::ROW_BYTES + 4 * t4;
            const uint8_t* krow1 = tile + (8 + grp) * GEO::ROW_BYTES + 4 * t4;
#pragma unroll 4
            for (int c = 0; c < CH; c += 2) {
              const uint32_t ka = *reinterpret_cast<const uint32_t*>(krow0 + ((c ^ grp) << 4));   // grp == token & 7
              const uint32_t kb = *reinterpret_cast<const uint32_t*>(krow1 + ((c ^ grp) << 4));
              const uint32_t kc = *reinterpret_cast<const uint32_t*>(krow0 + (((c + 1) ^ grp) << 4));
              const uint32_t kd = *reinterpret_cast<const uint32_t*>(krow1 + (((c + 1) ^ grp) << 4));
              const double2 qq = *reinterpret_cast<const double2*>(qrow + c * 8);
              const double2 qr = *reinterpret_cast<const double2*>(qrow + c * 8 + 8);
              const double b0 = ncol ? qq.x : 0.0, b1 = ncol ? qq.y : 0.0;
              const double b2 = ncol ? qr.x : 0.0, b3 = ncol ? qr.y : 0.0;
              dmma(z00, z01, (double)bf16_lo_f(ka), b0);
              dmma(z10, z11, (double)bf16_lo_f(kb), b0);
              dmma(y00, y01, (double)bf16_lo_f(kc), b2);
              dmma(y10, y11, (double)bf16_lo_f(kd), b2);
              dmma(z00, z01, (double)bf16_hi_f(ka), b1);
              dmma(z10, z11, (double)bf16_hi_f(kb), b1);
              dmma(y00, y01, (double)bf16_hi_f(kc), b3);
              dmma(y10, y11, (double)bf16_hi_f(kd), b3);
            }
            z00 += y00; z01 += y01; z10 += y10; z11 += y11;
            // D fragment: row = grp (token), columns 2*t4, 2*t4 + 1
            const int col = nt * 8 + 2 * t4;
            z00 /= sqrt_d; z01 /= sqrt_d; z10 /= sqrt_d; z11 /= sqrt_d;
            // the page's softmax partials per column: max and sum of exponentials over its 16 tokens; the
            // exponentials themselves are what is stored per token
            double m0 = fmax(z00, z10), m1 = fmax(z01, z11);
#pragma unroll
            for (int o2 = 4; o2 < 32; o2 <<= 1) {
              m0 = fmax(m0, __shfl_xor_sync(0xffffffffu, m0, o2));
              m1 = fmax(m1, __shfl_xor_sync(0xffffffffu, m1, o2));
            }
            z00 = exp(z00 - m0); z10 = exp(z10 - m0); z01 = exp(z01 - m1); z11 = exp(z11 - m1);
            double e0 = z00 + z10, e1 = z01 + z11;
#pragma unroll
            for (int o2 = 4; o2 < 32; o2 <<= 1) {
              e0 += __shfl_xor_sync(0xffffffffu, e0, o2);
              e1 += __shfl_xor_sync(0xffffffffu, e1, o2);
            }
            if (col < 2 * G) {
              // view = col / G (short or long summary); a view's values of one unit are contiguous [token][G]
              const size_t tokrow = (size_t)(zoff + tok0 + grp);
              if (G >= 2) {
                double* z0 = p.zbuf + (((size_t)lh * 2 + col / G) * p.z_stride + tokrow) * G + col % G;
                *reinterpret_cast<double2*>(z0) = make_double2(z00, z01);
                *reinterpret_cast<double2*>(z0 + (size_t)8 * G) = make_double2(z10, z11);
              } else {
                double* zS = p.zbuf + ((size_t)lh * 2 * p.z_stride + tokrow);
                double* zL = zS + p.z_stride;
                zS[0] = z00; zS[8] = z10; zL[0] = z01; zL[8] = z11;
              }
              if (grp == 0) {
                double* st2 = p.zstat + (((size_t)lh * (p.max_boundary_tokens / GP_PAGE) + (zoff + tok0) / GP_PAGE) * (2 * G) + col) * 2;
                *reinterpret_cast<double2*>(st2) = make_double2(m0, e0);
                *reinterpret_cast<double2*>(st2 + 2) = make_double2(m1, e1);
              }
            }
          }
        }
        __syncwarp();
        if (!top_up(it)) { ok = false; break; }            // the stage is free: fetch the next tile into it
      }
      if (!ok) break;

      // ---- a request at its boundary: this warp's share of the unit's summary logits (and the appended row, and the
      // request's counters) is written; the boundary work that may run beside this kernel counts the reports
      if ((flags & 1) && p.report_units) {
        __threadfence();
        __syncwarp();
        if (lane == 0 && !(p.withhold & GP_WITHHOLD_READY)) atomicAdd(p.unit_ready + (size_t)sd[15] * LH + lh, 1);
      }
      // ---- hand the partial result to the merger warp ---------------------------------------------
      l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
      l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
      const int cb = it % NCOMB;
      if (!wait_bar(&comb_empty[cb], ((it / NCOMB) & 1u) ^ 1u, s_misc, 6, lim)) break;
      float* my_comb = comb + (cb * NCW + cw) * comb_w;
      if (row < G) {
        if ((lane & 3) == 0) { my_comb[row] = m_run; my_comb[8 + row] = l_run; }
#pragma unroll
        for (int jd = 0; jd < GEO::DTILES; ++jd) {
          *reinterpret_cast<float2*>(&my_comb[16 + row * D + jd * 8 + qc]) =
              make_float2(o[jd][0] + o[jd][2], o[jd][1] + o[jd][3]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&comb_full[cb]);
      if (need_qt) {
        ++qt_uses;
        if (lane == 0) mbar_arrive(qt_empty);
      }
      if (lane == 0) mbar_arrive(&slot_empty[sl]);
    }
    cp_async_wait<0>();                  // after an abort copies may still be in flight: let them land
  } else if (warp == 2) {
    // ================================= merger =============================================
    for (uint32_t it = 0;; ++it) {
      const int sl = it % NI;
      if (!wait_bar(&slot_full[sl], (it / NI) & 1u, s_misc, 7, lim)) break;
      const uint8_t* slot = smem + L.off_slots + sl * GEO::SLOT_BYTES;
      const int* sd = reinterpret_cast<const int*>(slot);
      const int npg = sd[3];
      if (npg < 0) break;
      const int bi = sd[0], nchunks = sd[5], rc_i = sd[13], lh = sd[14];
      const int l = lh / p.Hkv, h = lh % p.Hkv;
      const int cb = it % NCOMB;
      if (!wait_bar(&comb_full[cb], (it / NCOMB) & 1u, s_misc, 8, lim)) break;
      const float* cbuf = comb + (size_t)cb * NCW * comb_w;
      const size_t out_row0 = (((size_t)l * n_req + bi) * p.Hq + h * G) * D;
      const int PSTRIDE = G * (D + 2);
      float* part = p.partials + ((size_t)lh * n_rc + rc_i) * PSTRIDE;
      for (int g = 0; g < G; ++g) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NCW; ++w) M = fmaxf(M, cbuf[w * comb_w + g]);
        float wgt[NCW];
        float ls = 0.f;
#pragma unroll
        for (int w = 0; w < NCW; ++w) {
          wgt[w] = exp2f(cbuf[w * comb_w + g] - M);
          ls += wgt[w] * cbuf[w * comb_w + 8 + g];
        }
        const float inv = 1.f / ls;
        for (int dc = lane; dc < D; dc += 32) {
          float acc = 0.f;
#pragma unroll
          for (int w = 0; w < NCW; ++w) acc += wgt[w] * cbuf[w * comb_w + 16 + g * D + dc];
          if (nchunks == 1) out[out_row0 + g * D + dc] = acc * inv;
          else part[g * (D + 2) + dc] = acc;
        }
        if (nchunks > 1 && lane == 0) { part[g * (D + 2) + D] = M; part[g * (D + 2) + D + 1] = ls; }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&comb_empty[cb]);
      __syncwarp();
      if (lane == 0) mbar_arrive(&slot_empty[sl]);
    }
  }
  __syncthreads();
  // a wait of this CTA gave up (whichever warp it was, and however late): say so, with the code of the wait
  if (tid == 0 && s_misc[0]) atomicOr(p.err, GP_E_SPIN | (1 << (7 + s_misc[1])));
}

}  // namespace

size_t gp_attention_smem(int d, int G) { return d == 128 ? make_lay<128>(G).total : make_lay<64>(G).total; }
int gp_attention_ctas_per_sm(int d) { (void)d; return 2; }

void gp_attention_setup(const GpDev& p) {           // once per pool: opt into the kernel's shared memory
  const int sm = (int)gp_attention_smem(p.d, p.G);
  if (p.d == 128) {
    cudaFuncSetAttribute(gp_attn_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
    cudaFuncSetAttribute(gp_attn_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
  } else {
    cudaFuncSetAttribute(gp_attn_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
    cudaFuncSetAttribute(gp_attn_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, sm);
  }
}

void gp_launch_attention(const GpDev& p, const int* req_ids, int n_req, const void* q, const void* k, const void* v,
                         float* out, int grid, cudaStream_t s, bool pdl, int lh0, int lh_n, int adv_lh) {
  (void)req_ids;
  const __nv_bfloat16* qq = static_cast<const __nv_bfloat16*>(q);
  const __nv_bfloat16* kk = static_cast<const __nv_bfloat16*>(k);
  const __nv_bfloat16* vv = static_cast<const __nv_bfloat16*>(v);
  const bool rope = p.rope_theta != 0.0;
  const int sm = (int)gp_attention_smem(p.d, p.G);
#define GP_LAUNCH(DD, RR)                                                                 \
  do {                                                                                    \
    auto kern = gp_attn_kernel<DD, RR>;                                                   \
    gp_launch(kern, grid, NTHREADS, (size_t)sm, s, pdl, p, n_req, qq, kk, vv, out, lh0, lh_n, adv_lh); \
  } while (0)
  if (p.d == 128) {
    if (rope) GP_LAUNCH(128, true); else GP_LAUNCH(128, false);
  } else {
    if (rope) GP_LAUNCH(64, true); else GP_LAUNCH(64, false);
  }
#undef GP_LAUNCH
}
