// The step after compression: one new query token per sequence attends over the compact cache
// (paper Sec. 3.1: generation continues on the compressed K, V).  The rows of a (layer,
// sequence, KV head) are few (B, a few hundred) and contiguous, so one CTA per such unit reads
// its K rows once for all G query heads of the group, keeps the G x n logits in shared memory,
// normalises them, and reads its V rows once.  All layers of a model go in one launch.
#include "common.cuh"

namespace mixkv {
namespace {

constexpr int kDecThreads = 256;
constexpr int kDecMaxG = 16;

// grid: n_layers * batch * H.  Dynamic shared memory: G * 128 floats (queries) + G * max_rows
// floats (logits, then weights).
__global__ void __launch_bounds__(kDecThreads, 2)
k_decode_attention(const __nv_bfloat16* __restrict__ Kc, const __nv_bfloat16* __restrict__ Vc,
                   const int* __restrict__ row_offsets, const long long rows_cap,
                   const __nv_bfloat16* __restrict__ q, const int BH, const int H, const int G,
                   const float scale_log2e, const int max_rows, float* __restrict__ out) {
  extern __shared__ float dsm[];
  float* sq = dsm;                       // [G][128]
  float* sp = dsm + G * kHeadDim;        // [G][max_rows]
  __shared__ float sinv[kDecMaxG];
  __shared__ float part[2][kDecMaxG][kHeadDim];
  const int unit = blockIdx.x, layer = unit / BH, bh = unit % BH, b = bh / H, h = bh % H;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int* ro = row_offsets + (size_t)layer * (BH + 1);
  const int r0 = ro[bh], n = min(ro[bh + 1] - r0, max_rows);
  const __nv_bfloat16* Kb = Kc + ((size_t)layer * rows_cap + r0) * kHeadDim;
  const __nv_bfloat16* Vb = Vc + ((size_t)layer * rows_cap + r0) * kHeadDim;
  const size_t qoff = (((size_t)layer * (BH / H) + b) * H + h) * (size_t)G * kHeadDim;
  for (int e = tid; e < G * kHeadDim; e += kDecThreads) sq[e] = __bfloat162float(q[qoff + e]);
  __syncthreads();

  // ---- logits (log2 units): one row per thread and sweep (its 256 bytes stay in L1 between
  // the sixteen 16-byte loads), all G query heads from shared memory; no cross-lane traffic
  for (int r = tid; r < n; r += kDecThreads) {
    float d[kDecMaxG];
#pragma unroll
    for (int g = 0; g < kDecMaxG; ++g) d[g] = 0.f;
    const uint4* krow = reinterpret_cast<const uint4*>(Kb + (size_t)r * kHeadDim);
#pragma unroll 4
    for (int c8 = 0; c8 < kHeadDim / 8; ++c8) {
      const uint4 kv = krow[c8];
      const float2 k0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kv.x));
      const float2 k1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kv.y));
      const float2 k2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kv.z));
      const float2 k3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kv.w));
#pragma unroll
      for (int g = 0; g < kDecMaxG; ++g) {
        if (g < G) {
          const float4 qa = *reinterpret_cast<const float4*>(sq + g * kHeadDim + 8 * c8);
          const float4 qb = *reinterpret_cast<const float4*>(sq + g * kHeadDim + 8 * c8 + 4);
          d[g] = fmaf(k0.x, qa.x, fmaf(k0.y, qa.y, fmaf(k1.x, qa.z, fmaf(k1.y, qa.w, d[g]))));
          d[g] = fmaf(k2.x, qb.x, fmaf(k2.y, qb.y, fmaf(k3.x, qb.z, fmaf(k3.y, qb.w, d[g]))));
        }
      }
    }
#pragma unroll
    for (int g = 0; g < kDecMaxG; ++g)
      if (g < G) sp[g * max_rows + r] = d[g] * scale_log2e;
  }
  __syncthreads();

  // ---- softmax weights per query head: warp w takes heads w, w + 8, ...
  for (int g = warp; g < G; g += kDecThreads / 32) {
    float* row = sp + g * max_rows;
    float mx = -INFINITY;
    for (int r = lane; r < n; r += 32) mx = fmaxf(mx, row[r]);
    mx = warp_max(mx);
    float sum = 0.f;
    for (int r = lane; r < n; r += 32) {
      const float e = exp2f(row[r] - mx);
      row[r] = e;
      sum += e;
    }
    sum = warp_sum(sum);
    if (lane == 0) sinv[g] = sum > 0.f ? 1.0f / sum : 0.f;
  }
  __syncthreads();

  // ---- weighted sum of the value rows: thread t takes column t % 128 of the rows of parity t / 128
  const int c = tid & (kHeadDim - 1), half = tid >> 7;
  float acc[kDecMaxG];
#pragma unroll
  for (int g = 0; g < kDecMaxG; ++g) acc[g] = 0.f;
#pragma unroll 4
  for (int r = half; r < n; r += 2) {
    const float v = __bfloat162float(Vb[(size_t)r * kHeadDim + c]);
#pragma unroll
    for (int g = 0; g < kDecMaxG; ++g)
      if (g < G) acc[g] = fmaf(sp[g * max_rows + r], v, acc[g]);
  }
#pragma unroll
  for (int g = 0; g < kDecMaxG; ++g)
    if (g < G) part[half][g][c] = acc[g];
  __syncthreads();
  for (int e = tid; e < G * kHeadDim; e += kDecThreads) {
    const int g = e / kHeadDim, cc = e % kHeadDim;
    out[qoff + e] = (part[0][g][cc] + part[1][g][cc]) * sinv[g];
  }
}

}  // namespace
}  // namespace mixkv

using namespace mixkv;

extern "C" int mixkv_decode_attention(const void* K_cache, const void* V_cache,
                                      const int32_t* out_row_offsets, int64_t rows_cap,
                                      const void* q, int32_t n_layers, int32_t batch,
                                      int32_t kv_heads, int32_t gqa_ratio, int32_t head_dim,
                                      float softmax_scale, int32_t max_rows, float* out,
                                      void* stream) {
  if (!K_cache || !V_cache || !out_row_offsets || !q || !out) return MIXKV_ERR_INVALID_ARG;
  if (n_layers < 1 || batch < 1 || kv_heads < 1 || gqa_ratio < 1 || rows_cap < 0 || max_rows < 1 ||
      !(softmax_scale >= 0.f))
    return MIXKV_ERR_INVALID_ARG;
  if (head_dim != kHeadDim || gqa_ratio > kDecMaxG) return MIXKV_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(K_cache) & 15u) || (reinterpret_cast<uintptr_t>(V_cache) & 15u) ||
      (reinterpret_cast<uintptr_t>(q) & 15u))
    return MIXKV_ERR_INVALID_ARG;
  const size_t smem = ((size_t)gqa_ratio * kHeadDim + (size_t)gqa_ratio * max_rows) * 4;
  if (smem > 160 * 1024) return MIXKV_ERR_UNSUPPORTED;
  {
    const int rc = device_check(nullptr);
    if (rc != MIXKV_OK) return rc;
  }
  if (smem > 48 * 1024) {
    static bool done[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MIXKV_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !done[dev]) {
      if (cudaFuncSetAttribute(k_decode_attention, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               160 * 1024) != cudaSuccess)
        return MIXKV_ERR_CUDA;
      if (dev >= 0 && dev < 64) done[dev] = true;
    }
  }
  const long long units = (long long)n_layers * batch * kv_heads;
  if (units > 0x7fffffffLL) return MIXKV_ERR_UNSUPPORTED;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)kHeadDim);
  k_decode_attention<<<(unsigned)units, kDecThreads, smem, (cudaStream_t)stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(K_cache), reinterpret_cast<const __nv_bfloat16*>(V_cache),
      out_row_offsets, rows_cap, reinterpret_cast<const __nv_bfloat16*>(q), batch * kv_heads, kv_heads,
      gqa_ratio, scale * kLog2e, max_rows, out);
  return cudaGetLastError() == cudaSuccess ? MIXKV_OK : MIXKV_ERR_CUDA;
}
