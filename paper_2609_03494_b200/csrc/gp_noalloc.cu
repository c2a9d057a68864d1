// gp_attention_noalloc: GQA decode attention over plain (un-paged) K/V that needs no memory beyond what the
// caller passes in.  The split-KV partial results, which the pool's attention kernel keeps in the pool blob,
// live here in a fixed array inside the library image.
//
// Who needs this: callers that are not allowed to allocate device memory when they call us.  Examples are a
// serving process that commits all of the GPU's memory to its KV pool at start-up (a later cudaMalloc would
// fail, and even a successful one synchronises the device in the middle of a decode loop), and hosts that run
// this library as a plug-in under a rule that library code never calls the allocator.  Such a caller can hand
// us inputs and outputs it already owns, but has nowhere to get scratch from.
//
// The price: every GPU whose context loads this library carries the array (8.5 MB) until the process exits,
// the problem size is capped (GP_NOALLOC_MAX_ROWS query-head rows), and all calls share the one array, so two
// calls that overlap on the GPU (different streams) corrupt each other's partial results.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "../../include/growpage.h"

namespace {

constexpr int NA_SPLITS = GP_NOALLOC_SPLITS;
constexpr int NA_MAX_ROWS = GP_NOALLOC_MAX_ROWS;
constexpr int NA_MAX_D = 128;
constexpr int NA_STRIDE = NA_MAX_D + 2;        // accumulator row, then running max and sum
constexpr int NA_THREADS = 128;
constexpr int NA_MAX_DEVICES = 64;

// Scratch of the entry point.  In host code this name is only a handle for the runtime's symbol calls; the
// device address is fetched once per device with cudaGetSymbolAddress (below) and passed to the kernels.
static __device__ __align__(256) float gp_noalloc_scratch[(size_t)NA_MAX_ROWS * NA_SPLITS * NA_STRIDE];

static float* g_scratch_addr[NA_MAX_DEVICES];  // device address of the array, per device, once known

// One CTA per (split, request, KV head): the split's share of the tokens, all G query heads of the group.
__global__ void __launch_bounds__(NA_THREADS)
na_partial_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                  const __nv_bfloat16* __restrict__ v, const int* __restrict__ lens, int Hq, int Hkv, int d,
                  int max_len, float* __restrict__ scratch) {
  __shared__ float s_q[8 * NA_MAX_D];
  __shared__ float s_part[NA_THREADS / 32][8][NA_MAX_D + 2];
  const int split = blockIdx.x, unit = blockIdx.y;
  const int req = unit / Hkv, h = unit % Hkv, G = Hq / Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int per = d / 32;
  for (int i = tid; i < G * d; i += NA_THREADS)
    s_q[(i / d) * NA_MAX_D + i % d] = __bfloat162float(q[((size_t)req * Hq + h * G + i / d) * d + i % d]);
  __syncthreads();
  const int len = min(lens[req], max_len);
  const int chunk = (len + NA_SPLITS - 1) / NA_SPLITS;
  const int t0 = split * chunk, t1 = min(len, t0 + chunk);
  const float scale = 1.4426950408889634f * rsqrtf((float)d);
  float m[8], l[8], acc[8][4];
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    m[g] = -INFINITY; l[g] = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[g][e] = 0.f;
  }
  const __nv_bfloat16* kbase = k + ((size_t)req * Hkv + h) * (size_t)max_len * d;
  const __nv_bfloat16* vbase = v + ((size_t)req * Hkv + h) * (size_t)max_len * d;
  for (int t = t0 + warp; t < t1; t += NA_THREADS / 32) {
    float kv[4], vv[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      kv[e] = e < per ? __bfloat162float(kbase[(size_t)t * d + lane + 32 * e]) : 0.f;
      vv[e] = e < per ? __bfloat162float(vbase[(size_t)t * d + lane + 32 * e]) : 0.f;
    }
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      if (g < G) {
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) s += (e < per ? s_q[g * NA_MAX_D + lane + 32 * e] : 0.f) * kv[e];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        s *= scale;
        const float mn = fmaxf(m[g], s);
        const float corr = exp2f(m[g] - mn), p = exp2f(s - mn);
        l[g] = l[g] * corr + p;
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[g][e] = acc[g][e] * corr + p * vv[e];
        m[g] = mn;
      }
    }
  }
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    if (g < G) {
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (e < per) s_part[warp][g][lane + 32 * e] = acc[g][e];
      if (lane == 0) { s_part[warp][g][NA_MAX_D] = m[g]; s_part[warp][g][NA_MAX_D + 1] = l[g]; }
    }
  }
  __syncthreads();
  // merge the warps; every slot of this (row, split) is rewritten on every call, so nothing stale survives
  for (int i = tid; i < G * d; i += NA_THREADS) {
    const int g = i / d, c = i % d;
    float M = -INFINITY;
    for (int w = 0; w < NA_THREADS / 32; ++w) M = fmaxf(M, s_part[w][g][NA_MAX_D]);
    float a = 0.f, ls = 0.f;
    for (int w = 0; w < NA_THREADS / 32; ++w) {
      const float wt = (M == -INFINITY) ? 0.f : exp2f(s_part[w][g][NA_MAX_D] - M);
      a += wt * s_part[w][g][c];
      ls += wt * s_part[w][g][NA_MAX_D + 1];
    }
    float* dst = scratch + (((size_t)req * Hq + h * G + g) * NA_SPLITS + split) * NA_STRIDE;
    dst[c] = a;
    if (c == 0) { dst[NA_MAX_D] = M; dst[NA_MAX_D + 1] = ls; }
  }
}

// One CTA per query-head row: merge the splits.
__global__ void na_merge_kernel(const float* __restrict__ scratch, int d, float* __restrict__ out) {
  const int row = blockIdx.x;
  const float* base = scratch + (size_t)row * NA_SPLITS * NA_STRIDE;
  float M = -INFINITY;
  for (int s = 0; s < NA_SPLITS; ++s) M = fmaxf(M, base[s * NA_STRIDE + NA_MAX_D]);
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float a = 0.f, ls = 0.f;
    for (int s = 0; s < NA_SPLITS; ++s) {
      const float ms = base[s * NA_STRIDE + NA_MAX_D];
      const float wt = (ms == -INFINITY) ? 0.f : exp2f(ms - M);
      a += wt * base[s * NA_STRIDE + c];
      ls += wt * base[s * NA_STRIDE + NA_MAX_D + 1];
    }
    out[(size_t)row * d + c] = ls > 0.f ? a / ls : 0.f;       // a request without tokens: a row of zeros
  }
}

}  // namespace

extern "C" int gp_attention_noalloc(const void* q, const void* k, const void* v, const int32_t* lens, int32_t n_req,
                                    int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t max_len,
                                    void* out, void* stream) {
  if (!q || !k || !v || !lens || !out) return GP_ERR_INVALID;
  if (n_req < 1 || n_q_heads < 1 || n_kv_heads < 1 || max_len < 1) return GP_ERR_INVALID;
  if (n_q_heads % n_kv_heads) return GP_ERR_INVALID;
  const int G = n_q_heads / n_kv_heads;
  if (G > 8 || (head_dim != 64 && head_dim != 128)) return GP_ERR_INVALID;
  if ((long long)n_req * n_q_heads > NA_MAX_ROWS) return GP_ERR_TOO_LARGE;   // the fixed array has no room
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES) return GP_ERR_CUDA;
  if (!g_scratch_addr[dev]) {
    // First call on this device: ask the runtime where the array lives here.  No allocation happens; the
    // array came with the library image.
    float* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), gp_noalloc_scratch) != cudaSuccess || !ptr) return GP_ERR_CUDA;
    g_scratch_addr[dev] = ptr;
  }
  float* scratch = g_scratch_addr[dev];
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const dim3 grid(NA_SPLITS, (unsigned)(n_req * n_kv_heads));
  na_partial_kernel<<<grid, NA_THREADS, 0, s>>>(static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k),
                                               static_cast<const __nv_bfloat16*>(v), lens, n_q_heads, n_kv_heads,
                                               head_dim, max_len, scratch);
  na_merge_kernel<<<(unsigned)(n_req * n_q_heads), head_dim, 0, s>>>(scratch, head_dim, static_cast<float*>(out));
  return cudaGetLastError() == cudaSuccess ? GP_OK : GP_ERR_CUDA;
}
