// The step after compression: one new query token per sequence attends over the compact cache
// (paper Sec. 3.1, Eq. 1: generation continues on the compressed K, V).  All layers of a model go
// in one launch.  The rows of a (layer, sequence, KV head) unit are split over the CTAs of a
// thread-block cluster (1, 2, 4 or 8: the fewest CTAs that fill the GPU once); a CTA walks its rows in blocks of 128 with a running softmax (reference, sum,
// weighted value sum per query head of the group).  Per block: the V rows start towards shared
// memory as one bulk copy, two threads per K row load its 256 bytes straight into registers (all
// loads in flight at once) and leave the G logits, the softmax weights are formed while the V
// copy lands, sixteen threads per V row add the weighted rows.  The cluster's partial results
// are merged through distributed shared memory by its first CTA.  Every row is read once.
#include <cooperative_groups.h>

#include "tc_common.cuh"

namespace cg = cooperative_groups;

namespace mixkv {
namespace {

constexpr int kDecThreads = 256;
constexpr int kDecMaxG = 16;
constexpr int kDecBlock = 128;   // rows per block: two threads per logit row

// Floats of dynamic shared memory in front of the V block: sq [G][128] queries, sp [G][128]
// logits then weights, part [8][G][128] per-warp value sums, xo [G][128] running weighted value
// sum, xm / xz / sscale [16] each.
__host__ __device__ constexpr size_t dec_floats(int G) {
  return (size_t)G * (kHeadDim + kDecBlock + 8 * kHeadDim + kHeadDim) + 3 * kDecMaxG;
}

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

// grid: n_layers * batch * H * S, clusters of S.
__global__ void __launch_bounds__(kDecThreads, 2)
k_decode_attention(const __nv_bfloat16* __restrict__ Kc, const __nv_bfloat16* __restrict__ Vc,
                   const int* __restrict__ row_offsets, const long long rows_cap,
                   const __nv_bfloat16* __restrict__ q, const int BH, const int H, const int G,
                   const float scale_log2e, const int max_rows, float* __restrict__ out) {
  extern __shared__ __align__(16) float dsm[];
  float* sq = dsm;                              // [G][128]
  float* sp = sq + G * kHeadDim;                // [G][128]
  float* part = sp + G * kDecBlock;             // [8][G][128]
  float* xo = part + 8 * G * kHeadDim;          // [G][128]
  float* xm = xo + G * kHeadDim;                // [16]
  float* xz = xm + kDecMaxG;                    // [16]
  float* sscale = xz + kDecMaxG;                // [16] rescale of the running sums for this block
  unsigned char* sV = reinterpret_cast<unsigned char*>(dsm + dec_floats(G));   // [128][256 B]
  __shared__ __align__(8) uint64_t vbar;
  __shared__ int vabort;
  cg::cluster_group cluster = cg::this_cluster();
  const int S = (int)cluster.num_blocks(), crank = (int)cluster.block_rank();
  const int unit = blockIdx.x / S, layer = unit / BH, bh = unit % BH, b = bh / H, h = bh % H;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  pdl_launch_dependents();
  if (tid == 0) {
    mbar_init(&vbar, 1);
    vabort = 0;
    mbar_init_fence();
  }
  pdl_wait();
  const int* ro = row_offsets + (size_t)layer * (BH + 1);
  const int r0 = ro[bh], n_unit = min(ro[bh + 1] - r0, max_rows);
  const int chunk = (n_unit + S - 1) / S;
  const int c0 = min(crank * chunk, n_unit), n = min(chunk, n_unit - c0);   // this CTA's rows
  const __nv_bfloat16* Kb = Kc + ((size_t)layer * rows_cap + r0 + c0) * kHeadDim;
  const __nv_bfloat16* Vb = Vc + ((size_t)layer * rows_cap + r0 + c0) * kHeadDim;
  const size_t qoff = (((size_t)layer * (BH / H) + b) * H + h) * (size_t)G * kHeadDim;
  for (int e = tid; e < G * kHeadDim; e += kDecThreads) {
    sq[e] = __bfloat162float(q[qoff + e]);
    xo[e] = 0.f;
  }
  if (tid < kDecMaxG) xm[tid] = -INFINITY, xz[tid] = 0.f;
  __syncthreads();

  int nblk = 0;
  for (int blk0 = 0; blk0 < n; blk0 += kDecBlock, ++nblk) {
    const int nb = min(kDecBlock, n - blk0);
    // ---- the block's V rows start towards shared memory (the previous block's readers are done)
    if (tid == 0) {
      mbar_expect_tx(&vbar, (uint32_t)nb * 256u);
      bulk_load(sV, Vb + (size_t)blk0 * kHeadDim, (uint32_t)nb * 256u, &vbar);
    }
    // ---- logits (log2 units): two threads per row, 64 dimensions each, all eight loads in flight
    {
      const int row = tid >> 1, hf = tid & 1;
      float d[kDecMaxG];
#pragma unroll
      for (int g = 0; g < kDecMaxG; ++g) d[g] = 0.f;
      if (row < nb) {
        const uint4* krow = reinterpret_cast<const uint4*>(Kb + (size_t)(blk0 + row) * kHeadDim + hf * 64);
        uint4 kv[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) kv[c] = krow[c];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const float2 k0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kv[c].x));
          const float2 k1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kv[c].y));
          const float2 k2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kv[c].z));
          const float2 k3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kv[c].w));
#pragma unroll
          for (int g = 0; g < kDecMaxG; ++g) {
            if (g < G) {
              const float* qg = sq + g * kHeadDim + hf * 64 + 8 * c;
              const float4 qa = *reinterpret_cast<const float4*>(qg);
              const float4 qb = *reinterpret_cast<const float4*>(qg + 4);
              d[g] = fmaf(k0.x, qa.x, fmaf(k0.y, qa.y, fmaf(k1.x, qa.z, fmaf(k1.y, qa.w, d[g]))));
              d[g] = fmaf(k2.x, qb.x, fmaf(k2.y, qb.y, fmaf(k3.x, qb.z, fmaf(k3.y, qb.w, d[g]))));
            }
          }
        }
      }
#pragma unroll
      for (int g = 0; g < kDecMaxG; ++g) {
        if (g < G) {
          const float o = __shfl_xor_sync(0xffffffffu, d[g], 1);
          const float t = hf ? o + d[g] : d[g] + o;   // first half + second half in both threads
          if (hf == 0 && row < nb) sp[g * kDecBlock + row] = t * scale_log2e;
        }
      }
    }
    __syncthreads();
    // ---- running softmax per query head: warp w takes heads w, w + 8, ...
    for (int g = warp; g < G; g += kDecThreads / 32) {
      float* row = sp + g * kDecBlock;
      float mx = -INFINITY;
      for (int r = lane; r < nb; r += 32) mx = fmaxf(mx, row[r]);
      mx = warp_max(mx);
      const float m_old = xm[g], m_new = fmaxf(m_old, mx);
      float sum = 0.f;
      for (int r = lane; r < nb; r += 32) {
        const float e = exp2f(row[r] - m_new);
        row[r] = e;
        sum += e;
      }
      sum = warp_sum(sum);
      if (lane == 0) {
        const float sc = m_old == -INFINITY ? 0.f : exp2f(m_old - m_new);
        sscale[g] = sc;
        xz[g] = xz[g] * sc + sum;
        xm[g] = m_new;
      }
    }
    const bool vok = mbar_wait(&vbar, nblk & 1, &vabort);
    __syncthreads();
    // ---- weighted sum of the value rows from shared memory: sixteen threads per row (16 bytes
    // each), sixteen rows per sweep, four query heads at a time
    const int c8 = tid & 15, rg = tid >> 4;
    for (int g0 = 0; g0 < G; g0 += 4) {
      float acc[4][8];
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[k][e] = 0.f;
      if (vok) {
#pragma unroll 2
        for (int r = rg; r < nb; r += 16) {
          const uint4 vv = *reinterpret_cast<const uint4*>(sV + (size_t)r * 256 + 16 * c8);
          float v[8];
          const float2 v0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vv.x));
          const float2 v1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vv.y));
          const float2 v2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vv.z));
          const float2 v3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vv.w));
          v[0] = v0.x, v[1] = v0.y, v[2] = v1.x, v[3] = v1.y, v[4] = v2.x, v[5] = v2.y, v[6] = v3.x, v[7] = v3.y;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            if (g0 + k < G) {
              const float wgt = sp[(g0 + k) * kDecBlock + r];
#pragma unroll
              for (int e = 0; e < 8; ++e) acc[k][e] = fmaf(wgt, v[e], acc[k][e]);
            }
          }
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float t = acc[k][e] + __shfl_xor_sync(0xffffffffu, acc[k][e], 16);
          if (lane < 16 && g0 + k < G) part[(warp * G + g0 + k) * kHeadDim + 8 * c8 + e] = t;
        }
      }
    }
    __syncthreads();
    for (int e = tid; e < G * kHeadDim; e += kDecThreads) {
      const int g = e / kHeadDim;
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) t += part[w * G * kHeadDim + e];
      xo[e] = xo[e] * sscale[g] + t;
    }
    __syncthreads();
  }

  // ---- merge the cluster's partial results in its first CTA
  cluster.sync();
  if (crank == 0) {
    for (int e = tid; e < G * kHeadDim; e += kDecThreads) {
      const int g = e / kHeadDim;
      float M = -INFINITY;
      for (int r = 0; r < S; ++r) M = fmaxf(M, *cluster.map_shared_rank(&xm[g], r));
      float num = 0.f, den = 0.f;
      if (M != -INFINITY) {
        for (int r = 0; r < S; ++r) {
          const float mr = *cluster.map_shared_rank(&xm[g], r);
          const float sc = mr == -INFINITY ? 0.f : exp2f(mr - M);
          num = fmaf(*cluster.map_shared_rank(&xo[e], r), sc, num);
          den = fmaf(*cluster.map_shared_rank(&xz[g], r), sc, den);
        }
      }
      out[qoff + e] = den > 0.f ? num / den : 0.f;
    }
  }
  cluster.sync();   // the peers' shared memory stays alive until the first CTA has read it
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
  const size_t smem = dec_floats(gqa_ratio) * 4 + (size_t)kDecBlock * 256;
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
                               128 * 1024) != cudaSuccess)
        return MIXKV_ERR_CUDA;
      if (dev >= 0 && dev < 64) done[dev] = true;
    }
  }
  const long long units = (long long)n_layers * batch * kv_heads;
  if (units * 8 > 0x7fffffffLL) return MIXKV_ERR_UNSUPPORTED;
  // rows of a unit over a cluster: the fewest CTAs that fill the GPU once (more CTAs than that
  // were measured slower: the cost of a call is the serial latency of a CTA, and launching more
  // of them adds to it), and no CTA with more than 1024 rows
  int S = 1;
  while (S < 8 && units * S < device_sm_count()) S *= 2;
  while (S < 8 && (max_rows + S - 1) / S > 8 * kDecBlock) S *= 2;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)kHeadDim);
  const cudaError_t e = launch_pdl(
      k_decode_attention, dim3((unsigned)(units * S)), dim3(kDecThreads), smem, (cudaStream_t)stream, S,
      reinterpret_cast<const __nv_bfloat16*>(K_cache), reinterpret_cast<const __nv_bfloat16*>(V_cache),
      out_row_offsets, (long long)rows_cap, reinterpret_cast<const __nv_bfloat16*>(q), batch * kv_heads,
      kv_heads, gqa_ratio, scale * kLog2e, max_rows, out);
  return e == cudaSuccess ? MIXKV_OK : MIXKV_ERR_CUDA;
}
