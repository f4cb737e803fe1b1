// The step after compression: one new query token per sequence attends over the compact cache
// (paper Sec. 3.1, Eq. 1: generation continues on the compressed K, V).  All layers of a model go
// in one launch.  With one query token and G query heads per KV head the two contractions have
// 7 .. 16 rows on one side: too few for the 64- or 128-row tcgen05 tiles (nine tenths of such a
// tile would be padding), too many multiply-adds for the fp32 pipe at HBM speed (2 * 2 * G * 128
// per 512-byte row pair), so they run as warp-level mma.sync m16n8k16 (bf16 x bf16 -> fp32) with
// every operand loaded from global memory straight into its fragment, no shared-memory staging:
//
//   * a warp takes 16 cache rows per step.  logits: D[head, row] = q[head, :] . K[row, :],
//     A = q (held in registers for the whole kernel), B = K rows.  The contraction index may be
//     permuted freely as long as A and B agree, so a lane takes 64 CONTIGUOUS bytes of its row
//     (four 16-byte loads) and deals them out over the eight k-steps.
//   * softmax weights with a running (reference, sum) per head in log2 units; the weights leave
//     as TWO bf16 (value and remainder), so the value sum is fp32-grade.
//   * values: D[head, dim] += P[head, row] . V[row, dim].  B wants two rows of one dim per
//     register: a lane loads 32 contiguous bytes of four rows and byte-permutes pairs of rows
//     together; which output column a lane's dim lands in is again a free permutation.
//
// The rows of a (layer, sequence, KV head) unit are dealt out in steps of 16 over the warps of a
// thread-block cluster (1, 2, 4 or 8 CTAs of four warps; as many as fit the GPU in one wave), and
// a warp keeps two register sets so that the loads of its next step fly while it works.  Warps merge through shared memory, the CTAs of a cluster through distributed
// shared memory, every CTA taking a slice of the outputs.  Every row is read once.
#include <cooperative_groups.h>

#include "tc_common.cuh"

namespace cg = cooperative_groups;

namespace mixkv {
namespace {

constexpr int kDecWarps = 4;
constexpr int kDecThreads = kDecWarps * 32;
constexpr int kDecMaxG = 16;
constexpr int kDecStep = 16;     // cache rows per warp step

// Floats of dynamic shared memory for GP = 8 or 16 head slots: wacc [warps][GP][132] per-warp
// value sums, xo [GP][128] the CTA's, wm / wz [warps][16], xm / xz [16], allm / allz [8][16]
// every rank's (reference, sum) during the cluster merge.
constexpr int kDecHeadPitch = kHeadDim + 4;   // floats between the heads of a warp's value sums
__host__ __device__ constexpr size_t dec_floats(int GP) {
  return (size_t)kDecWarps * GP * kDecHeadPitch + (size_t)GP * kHeadDim + 2 * kDecWarps * kDecMaxG +
         2 * kDecMaxG + 2 * 8 * kDecMaxG;
}
// Slot of dimension `dim` inside a head of a warp's value sums: one pad word per 32 dimensions
// and a head pitch of 132 put the 32 lanes of a fragment store (8 heads x 4 dimensions 32 apart)
// into 32 different banks.
__device__ __forceinline__ int dec_slot(int dim) { return dim + (dim >> 5); }

// D (16 x 8, fp32) += A (16 x 16, bf16, row) * B (16 x 8, bf16, col).  Lane l = 4 g + t holds
//   A: a0 (row g, k 2t..2t+1)  a1 (row g+8, same k)  a2 (row g, k 2t+8..2t+9)  a3 (row g+8, ..)
//   B: b0 (k 2t..2t+1, col g)  b1 (k 2t+8..2t+9, col g)
//   D: d0 d1 (row g, cols 2t, 2t+1)  d2 d3 (row g+8, same cols)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], const uint32_t b0,
                                         const uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
      "{%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// bf16 pair (x in the low half) of two floats, and what rounding left over.
__device__ __forceinline__ uint32_t pack_bf16(const float x, const float y) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(x, y);
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ void split_bf16(const float x, const float y, uint32_t& hi, uint32_t& lo) {
  hi = pack_bf16(x, y);
  lo = pack_bf16(x - __uint_as_float(hi << 16), y - __uint_as_float(hi & 0xffff0000u));
}
__device__ __forceinline__ uint32_t word_of(const uint4& v, const int i) {
  return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
}
__device__ __forceinline__ float quad_max(float v) {
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
  return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ float quad_sum(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  return v + __shfl_xor_sync(0xffffffffu, v, 2);
}

// grid: n_layers * batch * H * S, clusters of S.  WIDE: more than eight query heads per KV head
// (head slots 8..15 of the tiles carry data).
template <bool WIDE>
__global__ void __launch_bounds__(kDecThreads, 2)
k_decode_attention(const __nv_bfloat16* __restrict__ Kc, const __nv_bfloat16* __restrict__ Vc,
                   const int* __restrict__ row_offsets, const long long rows_cap,
                   const __nv_bfloat16* __restrict__ q, const int BH, const int H, const int G,
                   const float scale_log2e, const int max_rows, float* __restrict__ out) {
  constexpr int GP = WIDE ? 16 : 8;
  extern __shared__ __align__(16) float dsm[];
  float* wacc = dsm;                                   // [warps][GP][kDecHeadPitch]
  float* xo = wacc + kDecWarps * GP * kDecHeadPitch;   // [GP][128]
  float* wm = xo + GP * kHeadDim;                      // [warps][16]
  float* wz = wm + kDecWarps * kDecMaxG;               // [warps][16]
  float* xm = wz + kDecWarps * kDecMaxG;               // [16]
  float* xz = xm + kDecMaxG;                           // [16]
  float* allm = xz + kDecMaxG;                         // [8][16]
  float* allz = allm + 8 * kDecMaxG;                   // [8][16]
  cg::cluster_group cluster = cg::this_cluster();
  const int S = (int)cluster.num_blocks(), crank = (int)cluster.block_rank();
  const int unit = blockIdx.x / S, layer = unit / BH, bh = unit % BH, b = bh / H, h = bh % H;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  pdl_launch_dependents();
  pdl_wait();
  const int* ro = row_offsets + (size_t)layer * (BH + 1);
  const int r0 = ro[bh], n = min(ro[bh + 1] - r0, max_rows);
  const __nv_bfloat16* Kb = Kc + ((size_t)layer * rows_cap + r0) * kHeadDim;
  const __nv_bfloat16* Vb = Vc + ((size_t)layer * rows_cap + r0) * kHeadDim;
  const size_t qoff = (((size_t)layer * (BH / H) + b) * H + h) * (size_t)G * kHeadDim;

  // ---- query fragments: k-step kt of lane (g, t) covers dimensions 32 t + 4 kt .. + 3 of heads
  // g and g + 8, the first two as a0 / a1, the last two as a2 / a3
  uint32_t qa[8][4];
  {
    const uint4* q0 = reinterpret_cast<const uint4*>(q + qoff + (size_t)g * kHeadDim + 32 * t);
    const uint4* q1 = reinterpret_cast<const uint4*>(q + qoff + (size_t)(g + 8) * kHeadDim + 32 * t);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint4 u0 = make_uint4(0, 0, 0, 0), u1 = u0;
      if (g < G) u0 = __ldg(q0 + i);
      if (WIDE && g + 8 < G) u1 = __ldg(q1 + i);
      qa[2 * i][0] = u0.x, qa[2 * i][2] = u0.y, qa[2 * i + 1][0] = u0.z, qa[2 * i + 1][2] = u0.w;
      qa[2 * i][1] = u1.x, qa[2 * i][3] = u1.y, qa[2 * i + 1][1] = u1.z, qa[2 * i + 1][3] = u1.w;
    }
  }
  // value sums: tile dt, registers 0 1 = head g, dimensions 16 (2t) + dt and 16 (2t + 1) + dt;
  // registers 2 3 = head g + 8
  float acc[16][4];
#pragma unroll
  for (int dt = 0; dt < 16; ++dt)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[dt][c] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, z0 = 0.f, z1 = 0.f;

  const int nsteps = (n + kDecStep - 1) / kDecStep;
  // All loads of a step: K rows rb + 8 j + g (64 bytes from 64 t), V rows rb + 2t, 2t + 1,
  // 2t + 8, 2t + 9 (32 bytes from 32 g).  Rows past the end repeat the last row; their weights
  // are zero.
  auto load_step = [&](const int step, uint4 (&kq)[2][4], uint4 (&vq)[4][2]) {
    const int rb = step * kDecStep;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int row = min(rb + 8 * j + g, n - 1);
      const uint4* p = reinterpret_cast<const uint4*>(Kb + (size_t)row * kHeadDim + 32 * t);
#pragma unroll
      for (int i = 0; i < 4; ++i) kq[j][i] = __ldg(p + i);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int row = min(rb + 2 * t + (u & 1) + 8 * (u >> 1), n - 1);
      const uint4* p = reinterpret_cast<const uint4*>(Vb + (size_t)row * kHeadDim + 16 * g);
      vq[u][0] = __ldg(p);
      vq[u][1] = __ldg(p + 1);
    }
  };
  auto work_step = [&](const int step, const uint4 (&kq)[2][4], const uint4 (&vq)[4][2]) {
    const int rb = step * kDecStep;
    // ---- logits: s[j] registers 0 1 = head g, rows rb + 8 j + 2t, + 1; 2 3 = head g + 8
    float s[2][4];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
#pragma unroll
      for (int c = 0; c < 4; ++c) s[j][c] = 0.f;
#pragma unroll
      for (int kt = 0; kt < 8; ++kt)
        mma_bf16(s[j], qa[kt], word_of(kq[j][kt >> 1], 2 * (kt & 1)),
                 word_of(kq[j][kt >> 1], 2 * (kt & 1) + 1));
    }
    // ---- softmax weights under the running reference of each head (log2 units)
    float p[2][4];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int c = 0; c < 4; ++c)
        p[j][c] = rb + 8 * j + 2 * t + (c & 1) < n ? s[j][c] * scale_log2e : -INFINITY;
    {
      const float mx = quad_max(fmaxf(fmaxf(p[0][0], p[0][1]), fmaxf(p[1][0], p[1][1])));
      const float mn = fmaxf(m0, mx), f = exp2f(m0 - mn);   // mx is finite: the step has a row
      if (f != 1.f) {
        z0 *= f;
#pragma unroll
        for (int dt = 0; dt < 16; ++dt) acc[dt][0] *= f, acc[dt][1] *= f;
      }
      m0 = mn;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        p[j][0] = exp2f(p[j][0] - mn);
        p[j][1] = exp2f(p[j][1] - mn);
        z0 += p[j][0] + p[j][1];
      }
    }
    if (WIDE) {
      const float mx = quad_max(fmaxf(fmaxf(p[0][2], p[0][3]), fmaxf(p[1][2], p[1][3])));
      const float mn = fmaxf(m1, mx), f = exp2f(m1 - mn);
      if (f != 1.f) {
        z1 *= f;
#pragma unroll
        for (int dt = 0; dt < 16; ++dt) acc[dt][2] *= f, acc[dt][3] *= f;
      }
      m1 = mn;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        p[j][2] = exp2f(p[j][2] - mn);
        p[j][3] = exp2f(p[j][3] - mn);
        z1 += p[j][2] + p[j][3];
      }
    }
    // the weights as bf16 value + bf16 remainder: A fragments over the 16 rows of the step
    uint32_t ahi[4] = {0, 0, 0, 0}, alo[4] = {0, 0, 0, 0};
    split_bf16(p[0][0], p[0][1], ahi[0], alo[0]);
    split_bf16(p[1][0], p[1][1], ahi[2], alo[2]);
    if (WIDE) {
      split_bf16(p[0][2], p[0][3], ahi[1], alo[1]);
      split_bf16(p[1][2], p[1][3], ahi[3], alo[3]);
    }
    // ---- values: tile dt takes dimension 16 g + dt of this lane's four rows
#pragma unroll
    for (int dt = 0; dt < 16; ++dt) {
      const int w = dt >> 1;
      const uint32_t sel = (dt & 1) ? 0x7632u : 0x5410u;
      const uint32_t b0 = __byte_perm(word_of(vq[0][w >> 2], w & 3), word_of(vq[1][w >> 2], w & 3), sel);
      const uint32_t b1 = __byte_perm(word_of(vq[2][w >> 2], w & 3), word_of(vq[3][w >> 2], w & 3), sel);
      mma_bf16(acc[dt], ahi, b0, b1);
      mma_bf16(acc[dt], alo, b0, b1);
    }
  };
  // two register sets: the loads of a warp's next step are in flight while it works on this one
  {
    const int stride = S * kDecWarps;
    uint4 kA[2][4], vA[4][2], kB[2][4], vB[4][2];
    int step = crank * kDecWarps + warp;
    if (step < nsteps) load_step(step, kA, vA);
    while (step < nsteps) {
      if (step + stride < nsteps) load_step(step + stride, kB, vB);
      work_step(step, kA, vA);
      step += stride;
      if (step >= nsteps) break;
      if (step + stride < nsteps) load_step(step + stride, kA, vA);
      work_step(step, kB, vB);
      step += stride;
    }
  }

  // ---- the warps of the CTA merge through shared memory
  z0 = quad_sum(z0);
  z1 = quad_sum(z1);
#pragma unroll
  for (int dt = 0; dt < 16; ++dt) {
    float* w0 = wacc + ((size_t)warp * GP + g) * kDecHeadPitch;
    w0[dec_slot(16 * (2 * t) + dt)] = acc[dt][0];
    w0[dec_slot(16 * (2 * t + 1) + dt)] = acc[dt][1];
    if (WIDE) {
      w0[8 * kDecHeadPitch + dec_slot(16 * (2 * t) + dt)] = acc[dt][2];
      w0[8 * kDecHeadPitch + dec_slot(16 * (2 * t + 1) + dt)] = acc[dt][3];
    }
  }
  if (t == 0) {
    wm[warp * kDecMaxG + g] = m0, wz[warp * kDecMaxG + g] = z0;
    wm[warp * kDecMaxG + g + 8] = WIDE ? m1 : -INFINITY, wz[warp * kDecMaxG + g + 8] = WIDE ? z1 : 0.f;
  }
  __syncthreads();
  for (int e = tid; e < GP * kHeadDim; e += kDecThreads) {
    const int head = e / kHeadDim, dim = e % kHeadDim;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, wm[w * kDecMaxG + head]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
      const float mw = wm[w * kDecMaxG + head];
      const float sc = mw == -INFINITY ? 0.f : exp2f(mw - M);
      num = fmaf(wacc[((size_t)w * GP + head) * kDecHeadPitch + dec_slot(dim)], sc, num);
      den = fmaf(wz[w * kDecMaxG + head], sc, den);
    }
    xo[e] = num;
    if (dim == 0) xm[head] = M, xz[head] = den;
  }

  // ---- the CTAs of the cluster merge through distributed shared memory: every CTA copies all
  // ranks' (reference, sum) pairs, then takes a slice of the G * 128 outputs
  cluster.sync();
  for (int e = tid; e < S * G; e += kDecThreads) {
    const int r = e / G, head = e % G;
    allm[r * kDecMaxG + head] = *cluster.map_shared_rank(&xm[head], r);
    allz[r * kDecMaxG + head] = *cluster.map_shared_rank(&xz[head], r);
  }
  __syncthreads();
  const int per = (G * kHeadDim + S - 1) / S;
  for (int e = crank * per + tid; e < min((crank + 1) * per, G * kHeadDim); e += kDecThreads) {
    const int head = e / kHeadDim;
    float M = -INFINITY;
    for (int r = 0; r < S; ++r) M = fmaxf(M, allm[r * kDecMaxG + head]);
    float num = 0.f, den = 0.f;
    if (M != -INFINITY) {
      for (int r = 0; r < S; ++r) {
        const float mr = allm[r * kDecMaxG + head];
        const float sc = mr == -INFINITY ? 0.f : exp2f(mr - M);
        num = fmaf(*cluster.map_shared_rank(&xo[e], r), sc, num);
        den = fmaf(allz[r * kDecMaxG + head], sc, den);
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
  {
    const int rc = device_check(nullptr);
    if (rc != MIXKV_OK) return rc;
  }
  const long long units = (long long)n_layers * batch * kv_heads;
  if (units * 8 > 0x7fffffffLL) return MIXKV_ERR_UNSUPPORTED;
  // CTAs per unit: as many as still fit the GPU in one wave (two CTAs of four warps per SM: the
  // two register sets of a warp hold 16 KB of loads in flight) while every warp keeps at least
  // two steps to overlap
  const long long steps = ((long long)max_rows + kDecStep - 1) / kDecStep;
  int S = 1;
  while (S < 8 && units * (2 * S) <= 2LL * device_sm_count() && 2LL * (2 * S) * kDecWarps <= steps)
    S *= 2;
  const bool wide = gqa_ratio > 8;
  const size_t smem = dec_floats(wide ? 16 : 8) * 4;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)kHeadDim);
  const cudaError_t e = launch_pdl(
      wide ? k_decode_attention<true> : k_decode_attention<false>, dim3((unsigned)(units * S)),
      dim3(kDecThreads), smem, (cudaStream_t)stream, S,
      reinterpret_cast<const __nv_bfloat16*>(K_cache), reinterpret_cast<const __nv_bfloat16*>(V_cache),
      out_row_offsets, (long long)rows_cap, reinterpret_cast<const __nv_bfloat16*>(q), batch * kv_heads,
      kv_heads, gqa_ratio, scale * kLog2e, max_rows, out);
  return e == cudaSuccess ? MIXKV_OK : MIXKV_ERR_CUDA;
}
