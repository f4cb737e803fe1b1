// The two passes over K (and the one pass over V) of the MixKV scoring step, written with
// warp-level mma.sync bf16 tensor-core tiles.
//
//   pass 1: for a chunk of keys of one (sequence, head): window logits Q K^T with queries on
//           the M side, per-row running softmax (max, sum) in log2 units; key norms, sum of
//           unit keys; value norms with their (min, max, sum) over the candidate positions.
//   pass 2: logits again with keys on the M side, normalised with the finished row
//           statistics and summed over the window rows and the G query heads -> s_ex_raw;
//           the mean unit key rides along as three extra bf16 "query" rows (hi / lo / lo2
//           split) so that the same tile also yields K_i . kbar -> s_div.
//
// Paper: extrinsic importance and diversity of Sec. 3.2, redundancy of Eq. 3-4.
#include "common.cuh"

namespace mixkv {

namespace {

constexpr int kLd = kHeadDim + 8;  // padded smem row (bf16 elements): 272 bytes

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, bool pred) {
  unsigned s = (unsigned)__cvta_generic_to_shared(smem);
  int sz = pred ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldsm_x4(unsigned (&r)[4], const void* p) {
  unsigned a = (unsigned)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(a));
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], const unsigned (&a)[4], unsigned b0,
                                         unsigned b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Copies `rows` rows of 128 bf16 from global (row stride 128) into padded smem rows; rows at
// or beyond `valid` are zero-filled.
__device__ __forceinline__ void load_rows(__nv_bfloat16* dst, const __nv_bfloat16* src, int rows,
                                          int valid, int tid, int nthreads) {
  for (int c = tid; c < rows * 16; c += nthreads) {
    const int r = c >> 4, q = c & 15;
    const bool ok = r < valid;
    cp_async16(dst + r * kLd + q * 8, src + (size_t)(ok ? r : 0) * kHeadDim + q * 8, ok);
  }
}

// ------------------------------------------------------------------------------ pass 1
template <int MB>
__global__ void __launch_bounds__(256)
k_pass1_mma(const SeqTable st, const __nv_bfloat16* __restrict__ K,
            const __nv_bfloat16* __restrict__ V, const __nv_bfloat16* __restrict__ Q,
            const Workspace ws, const float scale_log2e, const int use_vnorm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int NQ = st.NQ, W = st.W;
  __nv_bfloat16* sQ = reinterpret_cast<__nv_bfloat16*>(smem_raw);
  __nv_bfloat16* sK = sQ + (size_t)NQ * kLd;          // [2][64][kLd]
  float* skinv = reinterpret_cast<float*>(sK + 2 * 64 * kLd);  // [2][64]
  float* sred = skinv + 128;                           // [4][128]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int chunk = blockIdx.x, h = blockIdx.y;
  const int b = find_seq(st.chunk_start, st.batch, chunk);
  const int L = st.cu[b + 1] - st.cu[b], P = L - W;
  const int k0 = (chunk - st.chunk_start[b]) * kChunk;
  const int kend = min(k0 + kChunk, L);
  const int nsub = (kend - k0 + 63) >> 6;
  const size_t row0 = (size_t)h * st.Ltot + st.cu[b];  // first K/V row of this (b, h)
  const __nv_bfloat16* Kh = K + row0 * kHeadDim;
  const __nv_bfloat16* Qg = Q + ((size_t)b * st.H + h) * (size_t)NQ * kHeadDim;

  load_rows(sQ, Qg, NQ, NQ, tid, 256);
  load_rows(sK, Kh + (size_t)k0 * kHeadDim, 64, kend - k0, tid, 256);
  cp_async_commit();

  // ---- value norms of this chunk (candidate positions only); independent of smem
  float vmin = INFINITY, vmax = -INFINITY, vsum = 0.f;
  if (use_vnorm) {
    const __nv_bfloat16* Vh = V + row0 * kHeadDim;
    const int vend = min(kend, P);
    const int hw = lane >> 4, hl = lane & 15;
    for (int i = k0 + warp * 2 + hw; i < k0 + kChunk; i += 16) {
      float ss = 0.f;
      if (i < vend) {
        const uint4 u = __ldg(reinterpret_cast<const uint4*>(Vh + (size_t)i * kHeadDim) + hl);
        const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(v2[e]);
          ss = fmaf(f.x, f.x, ss);
          ss = fmaf(f.y, f.y, ss);
        }
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      if (i < vend && hl == 0) {
        const float n = sqrtf(ss);
        ws.vnorm[(size_t)h * st.Ptot + (st.cu[b] - b * W) + i] = n;
        vmin = fminf(vmin, n);
        vmax = fmaxf(vmax, n);
        vsum += n;
      }
    }
  }

  // ---- query fragments (A operand), resident for the whole chunk
  cp_async_wait<0>();
  __syncthreads();
  unsigned aQ[MB][8][4];
  bool mb_on[MB];
#pragma unroll
  for (int mb = 0; mb < MB; ++mb) {
    const int r0 = (warp * MB + mb) * 16;
    mb_on[mb] = r0 < NQ;
    if (mb_on[mb]) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
        ldsm_x4(aQ[mb][ks], sQ + (size_t)(r0 + (lane & 15)) * kLd + ks * 16 + 8 * (lane >> 4));
    }
  }

  float m_run[MB][2], z_run[MB][2];
#pragma unroll
  for (int mb = 0; mb < MB; ++mb)
    m_run[mb][0] = m_run[mb][1] = -1e30f, z_run[mb][0] = z_run[mb][1] = 0.f;
  float ks0 = 0.f, ks1 = 0.f;  // partial sum of unit keys, dims 2*(tid%64), +1
  const bool need_mask = kend > P;

  for (int s = 0; s < nsub; ++s) {
    const int buf = s & 1;
    __nv_bfloat16* sKb = sK + (size_t)buf * 64 * kLd;
    if (s + 1 < nsub) {
      const int kk = k0 + (s + 1) * 64;
      load_rows(sK + (size_t)(buf ^ 1) * 64 * kLd, Kh + (size_t)kk * kHeadDim, 64, kend - kk, tid,
                256);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    // -- key norms: 4 threads per key
    {
      const int key = tid >> 2, part = tid & 3;
      const uint4* p4 = reinterpret_cast<const uint4*>(sKb + (size_t)key * kLd + part * 32);
      float ss = 0.f;
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        const uint4 u = p4[v];
        const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(v2[e]);
          ss = fmaf(f.x, f.x, ss);
          ss = fmaf(f.y, f.y, ss);
        }
      }
      ss += __shfl_xor_sync(0xffffffffu, ss, 1);
      ss += __shfl_xor_sync(0xffffffffu, ss, 2);
      if (part == 0) {
        const int i = k0 + s * 64 + key;
        const float inv = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
        skinv[buf * 64 + key] = inv;
        if (i < kend) ws.kinv[row0 + i] = inv;
      }
    }
    __syncthreads();
    // -- sum of unit keys
    {
      const int pr = tid & 63, grp = tid >> 6;
#pragma unroll 4
      for (int kk = 0; kk < 16; ++kk) {
        const int key = grp * 16 + kk;
        const float2 f = __bfloat1622float2(
            *reinterpret_cast<const __nv_bfloat162*>(sKb + (size_t)key * kLd + 2 * pr));
        const float inv = skinv[buf * 64 + key];
        ks0 = fmaf(f.x, inv, ks0);
        ks1 = fmaf(f.y, inv, ks1);
      }
    }
    // -- logits and running softmax statistics
    if (mb_on[0]) {
#pragma unroll 1
      for (int ntp = 0; ntp < 4; ++ntp) {
        float acc[MB][2][4];
#pragma unroll
        for (int mb = 0; mb < MB; ++mb)
#pragma unroll
          for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[mb][nt][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          unsigned bk[4];
          ldsm_x4(bk, sKb + (size_t)(ntp * 16 + (lane & 7) + 8 * (lane >> 4)) * kLd + ks * 16 +
                          8 * ((lane >> 3) & 1));
#pragma unroll
          for (int mb = 0; mb < MB; ++mb) {
            if (mb_on[mb]) {
              mma_bf16(acc[mb][0], aQ[mb][ks], bk[0], bk[1]);
              mma_bf16(acc[mb][1], aQ[mb][ks], bk[2], bk[3]);
            }
          }
        }
        const int ibase = k0 + s * 64 + ntp * 16 + 2 * (lane & 3);
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
          if (!mb_on[mb]) continue;
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            const int row = (warp * MB + mb) * 16 + (lane >> 2) + 8 * hf;
            const int lim = need_mask ? min(P + (row % W), L - 1) : 0x7fffffff;  // last visible key
            float v[4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const int i = ibase + nt * 8 + e;
                const float x = acc[mb][nt][hf * 2 + e] * scale_log2e;
                v[nt * 2 + e] = (i <= lim) ? x : -INFINITY;
              }
            const float mx = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3]));
            const float mn = fmaxf(m_run[mb][hf], mx);
            float z = z_run[mb][hf] * ex2(m_run[mb][hf] - mn);
#pragma unroll
            for (int e = 0; e < 4; ++e) z += ex2(v[e] - mn);
            m_run[mb][hf] = mn;
            z_run[mb][hf] = z;
          }
        }
      }
    }
    __syncthreads();
  }

  // ---- write the chunk's partial results
  const size_t pc = (size_t)h * st.chunks_total + chunk;
#pragma unroll
  for (int mb = 0; mb < MB; ++mb) {
    if (!mb_on[mb]) continue;
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      float m = m_run[mb][hf];
      m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
      m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
      float z = z_run[mb][hf] * ex2(m_run[mb][hf] - m);
      z += __shfl_xor_sync(0xffffffffu, z, 1);
      z += __shfl_xor_sync(0xffffffffu, z, 2);
      if ((lane & 3) == 0) {
        const int row = (warp * MB + mb) * 16 + (lane >> 2) + 8 * hf;
        ws.rowstat[pc * NQ + row] = make_float2(m, z);
      }
    }
  }
  {
    const int pr = tid & 63, grp = tid >> 6;
    sred[grp * 128 + 2 * pr] = ks0;
    sred[grp * 128 + 2 * pr + 1] = ks1;
  }
  __syncthreads();
  if (tid < 128)
    ws.ksum[pc * kHeadDim + tid] = (sred[tid] + sred[128 + tid]) + (sred[256 + tid] + sred[384 + tid]);
  __syncthreads();
  if (use_vnorm) {
    vmin = warp_min(vmin);
    vmax = warp_max(vmax);
    vsum = warp_sum(vsum);
    if (lane == 0) {
      sred[warp] = vmin;
      sred[8 + warp] = vmax;
      sred[16 + warp] = vsum;
    }
    __syncthreads();
    if (tid == 0) {
      float a = sred[0], bb = sred[8], c = sred[16];
      for (int w = 1; w < 8; ++w) {
        a = fminf(a, sred[w]);
        bb = fmaxf(bb, sred[8 + w]);
        c += sred[16 + w];
      }
      ws.vstat[pc] = make_float4(a, bb, c, 0.f);
    }
  }
}

// ------------------------------------------------------------------------------ pass 2
__global__ void __launch_bounds__(256)
k_pass2_mma(const SeqTable st, const __nv_bfloat16* __restrict__ K,
            const __nv_bfloat16* __restrict__ Q, const Workspace ws, float* __restrict__ s_div_out,
            const float scale_log2e) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int NQ = st.NQ, W = st.W;
  const int NB = NQ + kExtraRows;
  __nv_bfloat16* sQ = reinterpret_cast<__nv_bfloat16*>(smem_raw);  // [NB][kLd]
  __nv_bfloat16* sK = sQ + (size_t)NB * kLd;                       // [2][128][kLd]
  float* sbq = reinterpret_cast<float*>(sK + 2 * 128 * kLd);       // [NQ]
  float* sred = sbq + kMaxNQ;                                      // [32]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int chunk = blockIdx.x, h = blockIdx.y;
  const int b = find_seq(st.chunk_start, st.batch, chunk);
  const int L = st.cu[b + 1] - st.cu[b], P = L - W;
  const int k0 = (chunk - st.chunk_start[b]) * kChunk;
  const int kend = min(k0 + kChunk, P);  // candidate positions only
  const size_t pc = (size_t)h * st.chunks_total + chunk;
  if (kend <= k0) {
    if (tid == 0) ws.dstat[pc] = make_float4(INFINITY, -INFINITY, 0.f, 0.f);
    return;
  }
  const int nsub = (kend - k0 + 127) >> 7;
  const size_t row0 = (size_t)h * st.Ltot + st.cu[b];
  const size_t poff = (size_t)h * st.Ptot + (st.cu[b] - b * W);
  const __nv_bfloat16* Kh = K + row0 * kHeadDim;
  const int bh = b * st.H + h;

  load_rows(sQ, Q + (size_t)bh * NQ * kHeadDim, NQ, NQ, tid, 256);
  load_rows(sQ + (size_t)NQ * kLd, ws.kbar_rows + (size_t)bh * 3 * kHeadDim, kExtraRows, 3, tid,
            256);
  load_rows(sK, Kh + (size_t)k0 * kHeadDim, 128, kend - k0, tid, 256);
  cp_async_commit();
  for (int q = tid; q < NQ; q += 256) sbq[q] = ws.bq[(size_t)bh * NQ + q];

  float dmin = INFINITY, dmax = -INFINITY, dsum = 0.f;
  for (int s = 0; s < nsub; ++s) {
    const int buf = s & 1;
    const __nv_bfloat16* sKb = sK + (size_t)buf * 128 * kLd;
    if (s + 1 < nsub) {
      const int kk = k0 + (s + 1) * 128;
      load_rows(sK + (size_t)(buf ^ 1) * 128 * kLd, Kh + (size_t)kk * kHeadDim, 128, kend - kk,
                tid, 256);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    unsigned aK[8][4];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)
      ldsm_x4(aK[ks], sKb + (size_t)(warp * 16 + (lane & 15)) * kLd + ks * 16 + 8 * (lane >> 4));
    float rs[2] = {0.f, 0.f}, dot[2] = {0.f, 0.f};
#pragma unroll 1
    for (int np = 0; np <= NQ / 16; ++np) {
      float acc[2][4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[nt][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        unsigned bq4[4];
        ldsm_x4(bq4, sQ + (size_t)(np * 16 + (lane & 7) + 8 * (lane >> 4)) * kLd + ks * 16 +
                         8 * ((lane >> 3) & 1));
        mma_bf16(acc[0], aK[ks], bq4[0], bq4[1]);
        mma_bf16(acc[1], aK[ks], bq4[2], bq4[3]);
      }
      if (np < NQ / 16) {
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const float2 nb = *reinterpret_cast<const float2*>(sbq + np * 16 + nt * 8 + 2 * (lane & 3));
          rs[0] += ex2(fmaf(acc[nt][0], scale_log2e, -nb.x)) + ex2(fmaf(acc[nt][1], scale_log2e, -nb.y));
          rs[1] += ex2(fmaf(acc[nt][2], scale_log2e, -nb.x)) + ex2(fmaf(acc[nt][3], scale_log2e, -nb.y));
        }
      } else {  // the mean-key rows: columns 0..2 hold hi, lo, lo2; the rest are zero
        dot[0] = (acc[0][0] + acc[0][1]) + (acc[1][0] + acc[1][1]);
        dot[1] = (acc[0][2] + acc[0][3]) + (acc[1][2] + acc[1][3]);
      }
    }
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      rs[hf] += __shfl_xor_sync(0xffffffffu, rs[hf], 1);
      rs[hf] += __shfl_xor_sync(0xffffffffu, rs[hf], 2);
      dot[hf] += __shfl_xor_sync(0xffffffffu, dot[hf], 1);
      dot[hf] += __shfl_xor_sync(0xffffffffu, dot[hf], 2);
      const int i = k0 + s * 128 + warp * 16 + (lane >> 2) + 8 * hf;
      if ((lane & 3) == 0 && i < kend) {
        ws.s_ex_raw[poff + i] = rs[hf];
        const float sd = -dot[hf] * ws.kinv[row0 + i];
        s_div_out[poff + i] = sd;
        dmin = fminf(dmin, sd);
        dmax = fmaxf(dmax, sd);
        dsum += sd;
      }
    }
    __syncthreads();
  }
  dmin = warp_min(dmin);
  dmax = warp_max(dmax);
  dsum = warp_sum(dsum);
  if (lane == 0) {
    sred[warp] = dmin;
    sred[8 + warp] = dmax;
    sred[16 + warp] = dsum;
  }
  __syncthreads();
  if (tid == 0) {
    float a = sred[0], bb = sred[8], c = sred[16];
    for (int w = 1; w < 8; ++w) {
      a = fminf(a, sred[w]);
      bb = fmaxf(bb, sred[8 + w]);
      c += sred[16 + w];
    }
    ws.dstat[pc] = make_float4(a, bb, c, 0.f);
  }
}

size_t pass1_smem(int NQ) {
  return (size_t)NQ * kLd * 2 + 2 * 64 * kLd * 2 + 128 * 4 + 512 * 4;
}
size_t pass2_smem(int NQ) {
  return (size_t)(NQ + kExtraRows) * kLd * 2 + 2 * 128 * kLd * 2 + kMaxNQ * 4 + 32 * 4;
}

}  // namespace

cudaError_t launch_pass1(const LaunchCtx& c, const void* K, const void* V, const void* Q) {
  const dim3 grid(c.st.chunks_total, c.st.H);
  const size_t smem = pass1_smem(c.st.NQ);
  auto k = c.st.NQ <= 128 ? k_pass1_mma<1> : k_pass1_mma<2>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  k<<<grid, 256, smem, c.stream>>>(c.st, (const __nv_bfloat16*)K, (const __nv_bfloat16*)V,
                                   (const __nv_bfloat16*)Q, c.ws, c.scale_log2e, c.p.use_vnorm);
  return cudaGetLastError();
}

cudaError_t launch_pass2(const LaunchCtx& c, const void* K, const void* Q, float* s_div_out) {
  const dim3 grid(c.st.chunks_total, c.st.H);
  const size_t smem = pass2_smem(c.st.NQ);
  cudaError_t e = cudaFuncSetAttribute(k_pass2_mma, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  k_pass2_mma<<<grid, 256, smem, c.stream>>>(c.st, (const __nv_bfloat16*)K,
                                             (const __nv_bfloat16*)Q, c.ws, s_div_out,
                                             c.scale_log2e);
  return cudaGetLastError();
}

}  // namespace mixkv
