// Device-side view of a GrowPage pool and the small PTX wrappers the kernels share.
//
// HBM layout (all regions carved from the caller's blob, 256-byte aligned):
//   kv        bf16  [L][n_pages][H_kv][2 (K|V)][b][d]   one (layer, page, KV head) tile is a
//                   contiguous 2*b*d*2 bytes: a warp stages K and V of a page with 512-byte rows of
//                   16-byte asynchronous copies.
//                   Inside a row of d elements the 16-byte chunks are XOR-swizzled with the
//                   slot index: logical chunk c of slot s lives at chunk c ^ (s & 7).  A tile
//                   copied verbatim to shared memory is then bank-conflict free for ldmatrix.
//   tok       int32 [L][n_pages][H_kv][b]               original token index of every slot
//   summaries fp64  [L][M][2][2][H_q][d]                Eq. 11 layout (short then long), double-buffered
//   page_table / shadow int32 [M][cap]                  shadow holds copy-on-write targets
//   scores    fp64  [jobs][L*H_kv][max_boundary_tokens] scores of candidate sets too large for shared memory
//   partials  fp32  split-KV partial outputs
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#define GP_PAGE 16             // tokens per physical page: the unit of the K/V tiles, the page tables and the free list.
                               // The method's page (gp_config.page_size, b = 16 ... 256 tokens: the unit in which capacity
                               // grows, blocks are formed and slots are freed) is `sub` of these, always taken together.
#define GP_MAX_BLK 256         // largest page_size
#define GP_SPIN_LIMIT (1u << 21)
#define GP_MAX_REQ 1024        // upper limit of max_requests (shared-memory arrays are sized by it)
#define GP_MOVE_TOK 64         // source slots per compaction chunk
#define GP_COST_BINS 288       // cost classes of attention work items (pages, x4 at a boundary)
#define GP_DESC_INTS 16        // ints per attention work descriptor
#define GP_ATTN_CONSUMERS 4    // consumer warps of an attention thread block: each reports once per item it worked on

// plan header slots (int32)
enum {
  HDR_N_RC = 0,      // (request, chunk) work items of this step
  HDR_N_BND,         // requests at a capacity boundary
  HDR_N_CMP,         // requests that compress
  HDR_DECIDED,       // boundary work in one kernel: stamped by the CTA that took the step's decisions
  HDR_DONE_CMP,      // CTAs of the compaction kernel that have finished
  HDR_STEP,          // step serial number
  HDR_N_ACTIVE,      // requests actually stepped
  HDR_DONE_SEL,      // CTAs of the selection kernel that have finished
  HDR_WORK_CMP,      // ticket counter of the compaction kernel
  HDR_N_CITEM,       // compaction work items (chunks x layers x heads)
  HDR_N_MC,          // requests whose attention was split over several work items
  HDR_N_COW,         // copy-on-write targets allotted this step
  HDR_COUNT = 16
};

// hand-overs a test can withhold (gp_test_withhold): the bounded wait for it then runs out
enum {
  GP_WITHHOLD_ITEM = 1,     // attention kernel, first CTA: its second work item is never published to the consumers
  GP_WITHHOLD_CHUNK = 2,    // compaction: the first chunk of a unit never says that its sources are read
  GP_WITHHOLD_DECIDED = 4,  // boundary kernel: the deciding CTA never tells the others
  GP_WITHHOLD_READY = 8,    // attention kernel: the consumer warps never report a boundary unit's logits complete
  GP_TEST_COMPACT_BY_UNIT = 16,   // (not a withheld hand-over) the compaction claims whole units whatever their number
};

// error bits
enum {
  GP_E_SPIN = 1,        // a bounded wait gave up
  GP_E_FREELIST = 2,    // free-list accounting went negative or overflowed
  GP_E_BOUNDS = 4,      // an index failed a bounds check and the access was skipped
  GP_E_SPIN_CMP = 8,    // the compaction kernel's bounded wait on the previous chunk gave up
  GP_E_SPIN_SEL = 16,   // a selection job's bounded wait for its unit's summary logits gave up
};

struct GpDev {
  // geometry
  int L, Hq, Hkv, G, d, M, cap, k_loc, chunk_pages, max_rc;     // cap, n_pages: in physical pages
  int sub, blk;                          // physical pages per page of the method (page_size / 16), and its tokens (page_size)
  long long n_pages, max_batch_tokens;
  long long max_boundary_tokens;         // bound on the summed candidate tokens of one step's boundary requests
  unsigned spin_limit;                   // iterations after which a bounded wait gives up (GP_SPIN_LIMIT; tests shorten it)
  int withhold;                          // test support, GP_WITHHOLD_*: a hand-over inside a kernel that is made not to happen
  int async;                             // 1: the boundary chain of a step runs beside the next step (see gp_decode_step)
  double beta_s, beta_l, top_p, tau, rope_theta;
  int bchunk_pages;                      // pages per work item of a request at its capacity boundary
  int metric;                            // GP_METRIC_*: working-set size (Eq. 7) or attention entropy
  double* Hx;                            // [M][L][H_kv][2] entropies of the two views at a request's last boundary (entropy metric)
  int policy;                            // GP_POLICY_* (0 demand, 1 inverse, 2 random, 3 shrink)
  unsigned long long policy_seed;
  double p_compress;
  double shrink_below;                   // Eq. 13: Shrink under this
  int min_pages_after_shrink;            // a Shrink must leave at least this many physical pages (the minimum capacity,
                                         // and two pages of the method)
  unsigned long long p_fix;              // top_p in 2^62 fixed point
  // pool
  __nv_bfloat16* kv;
  int* tok;
  int* refcount;
  int* free_stack;
  int* free_top;                         // number of free pages (stack height)
  int* page_table;
  int* shadow;
  // per request
  // Pages, occupied slots, "has decoded", summary buffer in use and position of every request.  A decode step's
  // plan only reads them; the attention kernel advances a stepped request by one token where it appends the
  // token (after the plan has completed), the decision step then sets pages and slots of the requests at a
  // boundary.  In the asynchronous mode a request that sits a step out is touched by that step's kernels not at
  // all, so the boundary chain that runs beside them owns its words.
  int* P; int* n; int* started; int* live; int* n_pristine; long long* pos;
  int* bstep;                            // [M] number of the decode step at which the request last reached its boundary
  int* last_act;                         // [M] decision taken at that boundary (GP_ACT_*)
  double* summ;
  int* Kx;                               // [M][L][H_kv][2]
  double* delta;                         // [M]
  // per step
  int* hdr;
  int* rcx;                              // [max_rc][GP_DESC_INTS] attention work descriptors:
                                         //   0 batch index, 1 request, 2 first page, 3 pages, 4 chunk, 5 chunks,
                                         //   6 n before the append, 7 position, 8 flags (1 boundary, 2 started),
                                         //   9 P, 10-11 offset into the logit scratch, 12 summary buffer in use,
                                         //   13 index of its partial-output slot
  int4* mc_list;                         // [M] split requests: {batch index, first partial, chunks, 0}
  int4* bnd_info;                        // [M][2] requests at a boundary: {slot in the batch, request, P, position of the step's token}, {score offset lo, hi, 0, 0}
  int* shard_sums;                       // [M][2] per boundary request: sum of K^S, sum of K^L over this pool's units (to be
                                         // summed over the pools that hold the other KV heads), then over all units
  int report_units;                      // the attention kernel reports boundary units complete (the boundary kernel that
                                         // runs behind it starts its jobs on those reports)
  int units_total;                       // (layer, KV head) units of the model: L H_kv times the number of KV-head shards
  int* unit_ready;                       // [M][L H_kv] per boundary unit: consumer warps of the attention kernel done with it
  int* bnd_acc;                          // [M][4] per boundary request: sum of K^S, sum of K^L, shared pages of C, 0
  int* free_peek;                        // [M+1] free_top at plan time, then the top entries of the free list, top first
  int4* cmp_info;                        // [M+1] compressing requests: {request, P, index in bnd_info, first compaction chunk}
  double* zbuf;                          // [L*H_kv][2][z_stride][G] boundary units, per view (short, long): exp(summary logit - its page's max)
  long long z_stride;                    // max_boundary_tokens rounded up to a multiple of the page size
  double* qtil;                          // [M][L*H_kv][2][G][d] calibrated, rotated summaries q~ of boundary requests, by batch slot
  double* zstat;                         // [L*H_kv][max_boundary_tokens / b][2][G][2] per-page softmax partials (max, sum)
  int* sum_par;                          // [M] which of the two summary buffers is current
  int* evict;                            // [M][L*H_kv][page_size] slots a compression evicts, ascending
  int* evict2;                           // [M][L*H_kv][2 page_size] slots a Shrink evicts, ascending (Shrink policy only)
  int* cflags;                           // compaction chunk flags, stamped with the step number
  double* rope_cs;                       // [M][d/2][2] cos, sin at the step's position
  float* partials;
  double* scores;
  long long* counters;                   // [16]
  int* err;
};

__device__ __forceinline__ size_t gp_tile_off(const GpDev& p, int l, long long page, int h) {
  // element offset of the K tile of (layer, page, head); the V tile follows b*d elements later
  return ((((size_t)l * (size_t)p.n_pages + (size_t)page) * p.Hkv + h) * 2) * (size_t)(GP_PAGE * p.d);
}
__device__ __forceinline__ size_t gp_tok_off(const GpDev& p, int l, long long page, int h) {
  return (((size_t)l * (size_t)p.n_pages + (size_t)page) * p.Hkv + h) * GP_PAGE;
}
// summaries: [L][M][2 buffers][2 views][H_q][d]
__device__ __forceinline__ size_t gp_summ_off(const GpDev& p, int l, int r, int buf, int x, int head) {
  return ((((((size_t)l * p.M + r) * 2 + buf) * 2 + x) * p.Hq) + head) * (size_t)p.d;
}

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
// One bounded hardware wait (the thread may be suspended for up to about a microsecond); the spins built
// on it are bounded by an iteration limit on top.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(1000u)
      : "memory");
  return ok != 0;
}
// non-blocking probe of a phase
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: returns false when the limit ran out (the caller records GP_E_SPIN and goes on).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  for (uint32_t it = 0; it < GP_SPIN_LIMIT; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
  }
  return false;
}
// 1-D bulk copy global -> shared of this CTA (this CTA only), completion counted on an mbarrier.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst_smem)),
      "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
// 16-byte asynchronous copy global -> shared (L2 only), tracked per thread in commit groups
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src_gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src_gmem) : "memory");
}
// the same with an L2 eviction-priority hint (createpolicy): streamed data marked evict-first leaves the L2 before
// the small, reused state and the code of the step's other kernels
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void cp_async16_hint(uint32_t dst_smem, const void* src_gmem, uint64_t policy) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src_gmem), "l"(policy)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo_f(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi_f(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ---- host-visible launchers (one per translation unit) -------------------------------------------
void gp_launch_attention(const GpDev& p, const int* req_ids, int n_req, const void* q, const void* k, const void* v,
                         float* out, int grid, cudaStream_t s, bool pdl, int lh0, int lh_n, int adv_lh);
size_t gp_attention_smem(int d, int G);
int gp_attention_ctas_per_sm(int d);
// ---- programmatic dependent launch -------------------------------------------------------------------
// Every kernel of the decode step waits at its top for the kernel before it in the stream (completion and
// memory flush), then lets the kernel after it be scheduled: the next grid's CTAs become resident while this
// one drains, which hides the launch latency between the step's kernels.  All of the step's grids are a
// single resident wave, so early-scheduled dependents only ever take resources nobody else is waiting for.
// Without the launch attribute both instructions do nothing.
#ifdef __CUDACC__
__device__ __forceinline__ void gp_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void gp_pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t gp_launch(void (*kern)(KArgs...), int grid, int block, size_t smem, cudaStream_t s, bool pdl,
                             Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3((unsigned)block);
  cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
#endif

void gp_attention_setup(const GpDev& p);
void gp_launch_chain(const GpDev& p, const GpDev& pa, int n_req_merge, float* out_merge, int serial, int has_chain, int grid,
                     cudaStream_t s, bool pdl, const int* req_ids = nullptr, int* actions = nullptr, int* actions_copy = nullptr);
// merge of the split requests' partial outputs for the units [lh0, lh0 + lh_n) (per-layer entry point)
void gp_launch_select_only(const GpDev& p, const int* req_ids, int n_req, int* actions, float* out, int grid_sel, cudaStream_t s,
                           bool pdl, int serial);
void gp_launch_decide_compact(const GpDev& p, const int* req_ids, int n_req, int* actions, int grid_compact, cudaStream_t s,
                              int serial);
void gp_launch_merge(const GpDev& p, int n_req, float* out, int lh0, int lh_n, int grid, cudaStream_t s, bool pdl);
void gp_boundary_setup(const GpDev& p, int num_sms, int* grid_sel, int* grid_compact);
size_t gp_bsel_smem_for_cap(long long cap);
#define GP_MAX_DYN_SMEM (227 * 1024)   // opt-in shared memory per CTA on sm_100
// boundary chain: probabilities + working sets + selection + decision, then compaction.
// `ev`, when not null, is recorded between the two kernels.  `pdl`: launch with programmatic stream serialization.
void gp_launch_boundary(const GpDev& p, const int* req_ids, int n_req, int* actions, float* out, int grid_sel,
                        int grid_compact, cudaStream_t s, cudaEvent_t ev, bool pdl, int serial);
