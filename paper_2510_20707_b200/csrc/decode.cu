// The step after compression: one new query token per sequence attends over the compact cache
// (paper Sec. 3.1, Eq. 1: generation continues on the compressed K, V).  All layers of a model go
// in one launch.  The rows of a (layer, sequence, KV head) unit are split over the CTAs of a
// thread-block cluster (1, 2, 4 or 8: the fewest CTAs that fill the GPU once); a CTA walks its
// rows in blocks of 128 with a running softmax (reference, sum, weighted value sum per query head
// of the group).  The loads run ahead of the arithmetic: the V rows of two blocks are on their
// way to shared memory (bulk copies into a two-stage ring) and the K rows of the next block are
// on their way to registers (two threads per row, all eight 16-byte loads of a thread in flight)
// while a block is worked on: logits from the registers, softmax weights, then sixteen threads
// per V row add the weighted rows of all query heads in one sweep (packed fp32 pairs).  The
// cluster's partial results are merged through distributed shared memory, every CTA taking a
// slice of the outputs.  Every row is read once.
#include <cooperative_groups.h>

#include "tc_common.cuh"

namespace cg = cooperative_groups;

namespace mixkv {
namespace {

constexpr int kDecThreads = 256;
constexpr int kDecMaxG = 16;
constexpr int kDecBlock = 128;   // rows per block: two threads per logit row
constexpr int kDecSweep = 8;     // query heads whose value sums a thread holds at once

// Floats of dynamic shared memory in front of the V ring: sq [G][128] queries, sp [G][128]
// logits then weights, part [8][G][128] per-warp value sums, xo [G][128] running weighted value
// sum, xm / xz / sscale [16] each, then the merge's copy of every rank's xm and xz [2][8][16].
__host__ __device__ constexpr size_t dec_floats(int G) {
  return (size_t)G * (kHeadDim + kDecBlock + 8 * kHeadDim + kHeadDim) + 3 * kDecMaxG +
         2 * 8 * kDecMaxG;
}

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

// Packed fp32 pairs: one instruction for two lanes of arithmetic.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float a, float b) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
// The two bf16 of a 32-bit word as an fp32 pair (low half first).
__device__ __forceinline__ f32x2 bf16x2_to_f32x2(uint32_t w) {
  return pack2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
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
  float* allm = sscale + kDecMaxG;              // [8][16] merge: every rank's xm
  float* allz = allm + 8 * kDecMaxG;            // [8][16] merge: every rank's xz
  unsigned char* sV = reinterpret_cast<unsigned char*>(dsm + dec_floats(G));   // [2][128][256 B]
  __shared__ __align__(8) uint64_t vbar[2];
  __shared__ int vabort;
  cg::cluster_group cluster = cg::this_cluster();
  const int S = (int)cluster.num_blocks(), crank = (int)cluster.block_rank();
  const int unit = blockIdx.x / S, layer = unit / BH, bh = unit % BH, b = bh / H, h = bh % H;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  pdl_launch_dependents();
  if (tid == 0) {
    mbar_init(&vbar[0], 1);
    mbar_init(&vbar[1], 1);
    vabort = 0;
    mbar_init_fence();
  }
  pdl_wait();
  const int* ro = row_offsets + (size_t)layer * (BH + 1);
  const int r0 = ro[bh], n_unit = min(ro[bh + 1] - r0, max_rows);
  const int chunk = (n_unit + S - 1) / S;
  const int c0 = min(crank * chunk, n_unit), n = min(chunk, n_unit - c0);   // this CTA's rows
  const int nblk = (n + kDecBlock - 1) / kDecBlock;
  const __nv_bfloat16* Kb = Kc + ((size_t)layer * rows_cap + r0 + c0) * kHeadDim;
  const __nv_bfloat16* Vb = Vc + ((size_t)layer * rows_cap + r0 + c0) * kHeadDim;
  const size_t qoff = (((size_t)layer * (BH / H) + b) * H + h) * (size_t)G * kHeadDim;
  __syncthreads();   // the barriers are initialised
  // ---- the V rows of the first two blocks start towards the ring
  if (tid == 0) {
    for (int k = 0; k < 2 && k < nblk; ++k) {
      const uint32_t bytes = (uint32_t)min(kDecBlock, n - k * kDecBlock) * 256u;
      mbar_expect_tx(&vbar[k], bytes);
      bulk_load(sV + (size_t)k * kDecBlock * 256, Vb + (size_t)k * kDecBlock * kHeadDim, bytes, &vbar[k]);
    }
  }
  // ---- the K rows of the first block start towards registers: row tid / 2, dimensions
  // 64 * (tid & 1) .. + 63
  const int row = tid >> 1, hf = tid & 1;
  uint4 kv[8];
  auto load_k = [&](const int blk) {
    const int rr = blk * kDecBlock + row;
    if (rr < n) {
      const uint4* krow = reinterpret_cast<const uint4*>(Kb + (size_t)rr * kHeadDim + hf * 64);
#pragma unroll
      for (int c = 0; c < 8; ++c) kv[c] = __ldg(krow + c);
    }
  };
  if (nblk > 0) load_k(0);
  for (int e = tid; e < G * kHeadDim; e += kDecThreads) {
    sq[e] = __bfloat162float(q[qoff + e]);
    xo[e] = 0.f;
  }
  if (tid < kDecMaxG) xm[tid] = -INFINITY, xz[tid] = 0.f;
  __syncthreads();

  for (int blk = 0; blk < nblk; ++blk) {
    const int nb = min(kDecBlock, n - blk * kDecBlock);
    const int st = blk & 1;
    // ---- logits (log2 units) from the K registers
    {
      f32x2 d[kDecMaxG];
#pragma unroll
      for (int g = 0; g < kDecMaxG; ++g) d[g] = pack2(0.f, 0.f);
      if (row < nb) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const f32x2 k0 = bf16x2_to_f32x2(kv[c].x), k1 = bf16x2_to_f32x2(kv[c].y);
          const f32x2 k2 = bf16x2_to_f32x2(kv[c].z), k3 = bf16x2_to_f32x2(kv[c].w);
#pragma unroll
          for (int g = 0; g < kDecMaxG; ++g) {
            if (g < G) {
              const ulonglong2* qg =
                  reinterpret_cast<const ulonglong2*>(sq + g * kHeadDim + hf * 64 + 8 * c);
              const ulonglong2 qa = qg[0], qb = qg[1];
              d[g] = fma2(k0, qa.x, fma2(k1, qa.y, d[g]));
              d[g] = fma2(k2, qb.x, fma2(k3, qb.y, d[g]));
            }
          }
        }
      }
      // the next block's K rows start towards the registers just read
      if (blk + 1 < nblk) load_k(blk + 1);
#pragma unroll
      for (int g = 0; g < kDecMaxG; ++g) {
        if (g < G) {
          float d0, d1;
          unpack2(d[g], d0, d1);
          const float mine = d0 + d1;
          const float o = __shfl_xor_sync(0xffffffffu, mine, 1);
          const float t = hf ? o + mine : mine + o;   // first half + second half in both threads
          if (hf == 0 && row < nb) sp[g * kDecBlock + row] = t * scale_log2e;
        }
      }
    }
    __syncthreads();
    // ---- running softmax per query head: warp w takes heads w, w + 8, ...
    for (int g = warp; g < G; g += kDecThreads / 32) {
      float* prow = sp + g * kDecBlock;
      float mx = -INFINITY;
      for (int r = lane; r < nb; r += 32) mx = fmaxf(mx, prow[r]);
      mx = warp_max(mx);
      const float m_old = xm[g], m_new = fmaxf(m_old, mx);
      float sum = 0.f;
      for (int r = lane; r < nb; r += 32) {
        const float e = exp2f(prow[r] - m_new);
        prow[r] = e;
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
    const bool vok = mbar_wait(&vbar[st], (blk >> 1) & 1, &vabort);
    __syncthreads();
    // ---- weighted sum of the value rows from shared memory: sixteen threads per row (16 bytes
    // each), sixteen rows per sweep over the block, up to eight query heads at a time
    const unsigned char* vblk = sV + (size_t)st * kDecBlock * 256;
    const int c8 = tid & 15, rg = tid >> 4;
    for (int g0 = 0; g0 < G; g0 += kDecSweep) {
      f32x2 acc[kDecSweep][4];
#pragma unroll
      for (int k = 0; k < kDecSweep; ++k)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[k][e] = pack2(0.f, 0.f);
      if (vok) {
#pragma unroll 2
        for (int r = rg; r < nb; r += 16) {
          const uint4 vv = *reinterpret_cast<const uint4*>(vblk + (size_t)r * 256 + 16 * c8);
          const f32x2 v0 = bf16x2_to_f32x2(vv.x), v1 = bf16x2_to_f32x2(vv.y);
          const f32x2 v2 = bf16x2_to_f32x2(vv.z), v3 = bf16x2_to_f32x2(vv.w);
#pragma unroll
          for (int k = 0; k < kDecSweep; ++k) {
            if (g0 + k < G) {
              const float wgt = sp[(g0 + k) * kDecBlock + r];
              const f32x2 w2 = pack2(wgt, wgt);
              acc[k][0] = fma2(w2, v0, acc[k][0]);
              acc[k][1] = fma2(w2, v1, acc[k][1]);
              acc[k][2] = fma2(w2, v2, acc[k][2]);
              acc[k][3] = fma2(w2, v3, acc[k][3]);
            }
          }
        }
      }
#pragma unroll
      for (int k = 0; k < kDecSweep; ++k) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float a0, a1;
          unpack2(acc[k][e], a0, a1);
          a0 += __shfl_xor_sync(0xffffffffu, a0, 16);
          a1 += __shfl_xor_sync(0xffffffffu, a1, 16);
          if (lane < 16 && g0 + k < G)
            *reinterpret_cast<float2*>(part + (warp * G + g0 + k) * kHeadDim + 8 * c8 + 2 * e) =
                make_float2(a0, a1);
        }
      }
    }
    __syncthreads();   // the block's V stage is free, `part` is complete
    if (tid == 0 && blk + 2 < nblk) {
      const uint32_t bytes = (uint32_t)min(kDecBlock, n - (blk + 2) * kDecBlock) * 256u;
      mbar_expect_tx(&vbar[st], bytes);
      bulk_load(sV + (size_t)st * kDecBlock * 256, Vb + (size_t)(blk + 2) * kDecBlock * kHeadDim, bytes,
                &vbar[st]);
    }
    for (int e = tid; e < G * kHeadDim; e += kDecThreads) {
      const int g = e / kHeadDim;
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) t += part[w * G * kHeadDim + e];
      xo[e] = xo[e] * sscale[g] + t;
    }
    __syncthreads();
  }

  // ---- merge the cluster's partial results: every CTA copies all ranks' (reference, sum) pairs,
  // then takes a slice of the G * 128 outputs
  cluster.sync();
  for (int e = tid; e < S * G; e += kDecThreads) {
    const int r = e / G, g = e % G;
    allm[r * kDecMaxG + g] = *cluster.map_shared_rank(&xm[g], r);
    allz[r * kDecMaxG + g] = *cluster.map_shared_rank(&xz[g], r);
  }
  __syncthreads();
  const int per = (G * kHeadDim + S - 1) / S;
  for (int e = crank * per + tid; e < min((crank + 1) * per, G * kHeadDim); e += kDecThreads) {
    const int g = e / kHeadDim;
    float M = -INFINITY;
    for (int r = 0; r < S; ++r) M = fmaxf(M, allm[r * kDecMaxG + g]);
    float num = 0.f, den = 0.f;
    if (M != -INFINITY) {
      for (int r = 0; r < S; ++r) {
        const float mr = allm[r * kDecMaxG + g];
        const float sc = mr == -INFINITY ? 0.f : exp2f(mr - M);
        num = fmaf(*cluster.map_shared_rank(&xo[e], r), sc, num);
        den = fmaf(allz[r * kDecMaxG + g], sc, den);
      }
    }
    out[qoff + e] = den > 0.f ? num / den : 0.f;
  }
  cluster.sync();   // a CTA's shared memory stays alive until its peers have read it
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
  const size_t smem = dec_floats(gqa_ratio) * 4 + 2 * (size_t)kDecBlock * 256;
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
