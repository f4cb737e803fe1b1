// Redundancy analysis at fine resolution (block = 1, 2, 4, 8 or 16 rows per cell): the dense
// cosine-similarity matrix R = X^ X^T of Eq. 3 on the tensor cores.  With few rows per cell the
// Gram of block sums IS the L x L contraction, so it runs as tcgen05 tiles:
//
//   k_unit_rows   one streaming pass over X: every row is normalised in fp32 and written as two
//                 bf16 arrays, hi = bf16(x^) and lo = bf16(x^ - hi) (together 16 mantissa bits,
//                 which keeps a cell within 1e-6 of the fp32 dot product); per 256-row slice the
//                 sum of the unit rows and the number of non-zero rows (for the head mean).
//   k_gram_tc     persistent CTAs, one row of 128 x 128 tiles at a time (rows I and nT-1-I
//                 paired so that every work item has the same length); only tiles J >= I are
//                 computed, the mirrored cells are written from the same registers.  Per tile
//                 24 tcgen05.mma steps accumulate hi.hi + hi.lo + lo.hi in tensor memory; the
//                 epilogue reduces the block x block sub-squares (columns in the thread, rows by
//                 warp shuffles), drops the i == j pairs and divides by the pair count.
#include <cuda.h>

#include "tc_common.cuh"

namespace mixkv {
namespace {

constexpr int kURows = 256;      // rows per slice of k_unit_rows
constexpr int kUThreads = 256;

// grid (ceil(L / 256), H).  A warp takes four rows at a time; lane l holds elements 4l .. 4l+3.
__global__ void __launch_bounds__(kUThreads)
k_unit_rows(const __nv_bfloat16* __restrict__ X, const int L, __nv_bfloat16* __restrict__ hi,
            __nv_bfloat16* __restrict__ lo, float* __restrict__ u, int* __restrict__ nz) {
  __shared__ float part[kUThreads / 32][kHeadDim];
  __shared__ int cnt[kUThreads / 32];
  const int sl = blockIdx.x, h = blockIdx.y, S = gridDim.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r0 = sl * kURows, r1 = min(L, r0 + kURows);
  const size_t hbase = (size_t)h * L * kHeadDim;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  int nonzero = 0;
  constexpr int kW = kUThreads / 32, kInFlight = 4;
  for (int r = r0 + warp; r < r1; r += kInFlight * kW) {
    uint2 v[kInFlight];
#pragma unroll
    for (int k = 0; k < kInFlight; ++k) {
      const int rk = r + k * kW;
      v[k] = rk < r1 ? *reinterpret_cast<const uint2*>(X + hbase + (size_t)rk * kHeadDim + 4 * lane)
                     : make_uint2(0u, 0u);
    }
    float f[kInFlight][4], n2[kInFlight];
#pragma unroll
    for (int k = 0; k < kInFlight; ++k) {
      const float2 p = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v[k].x));
      const float2 q = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v[k].y));
      f[k][0] = p.x, f[k][1] = p.y, f[k][2] = q.x, f[k][3] = q.y;
      n2[k] = (p.x * p.x + p.y * p.y) + (q.x * q.x + q.y * q.y);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
      for (int k = 0; k < kInFlight; ++k) n2[k] += __shfl_xor_sync(0xffffffffu, n2[k], o);
#pragma unroll
    for (int k = 0; k < kInFlight; ++k) {
      const int rk = r + k * kW;
      const float inv = n2[k] > 0.f ? rsqrtf(n2[k]) : 0.f;
      nonzero += n2[k] > 0.f;
      __nv_bfloat16 hh[4], ll[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float x = f[k][e] * inv;
        acc[e] += x;
        hh[e] = __float2bfloat16_rn(x);
        ll[e] = __float2bfloat16_rn(x - __bfloat162float(hh[e]));
      }
      if (rk < r1) {
        *reinterpret_cast<uint2*>(hi + hbase + (size_t)rk * kHeadDim + 4 * lane) =
            *reinterpret_cast<const uint2*>(hh);
        *reinterpret_cast<uint2*>(lo + hbase + (size_t)rk * kHeadDim + 4 * lane) =
            *reinterpret_cast<const uint2*>(ll);
      }
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) part[warp][4 * lane + e] = acc[e];
  if (lane == 0) cnt[warp] = nonzero;
  __syncthreads();
  if (threadIdx.x < kHeadDim) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kUThreads / 32; ++w) s += part[w][threadIdx.x];
    u[((size_t)h * S + sl) * kHeadDim + threadIdx.x] = s;
  }
  if (threadIdx.x == 0) {
    int c = 0;
    for (int w = 0; w < kUThreads / 32; ++w) c += cnt[w];
    nz[h * S + sl] = c;
  }
}

// ------------------------------------------------------------------------------- Gram tiles
constexpr int kGThreads = 12 * 32;   // TMA, MMA, 2 idle, 8 epilogue warps
constexpr int kGEpiWarp0 = 4, kGEpiWarps = 8;
constexpr int kOperandBytes = 4 * 16384;   // hi and lo of 128 rows: [part][64-column half][128 x 128 B]

struct GBars {
  uint64_t afull, afree;
  uint64_t bfull[2], bempty[2];
  uint64_t tfull[2], tempty[2];
  uint32_t tmem_base;
  int abort;
};

// The (head, row of tiles) items of one CTA: item m pairs rows m and nT-1-m of a head.
struct GramWalk {
  int nT, half, items, m, which, h, I;
  __device__ GramWalk(int nT_, int H) : nT(nT_), half((nT_ + 1) / 2), items(H * ((nT_ + 1) / 2)) {
    m = blockIdx.x;
    which = 0;
    set();
  }
  __device__ __forceinline__ bool valid() const { return m < items; }
  __device__ __forceinline__ void set() {
    if (m < items) {
      h = m / half;
      const int mi = m - h * half;
      I = which == 0 ? mi : nT - 1 - mi;
    }
  }
  __device__ __forceinline__ void next() {
    const int mi = m % half;
    if (which == 0 && nT - 1 - mi != mi) {
      which = 1;
    } else {
      which = 0;
      m += gridDim.x;
    }
    set();
  }
};

__device__ __forceinline__ void load_operand(unsigned char* dst, const CUtensorMap* tmHi,
                                             const CUtensorMap* tmLo, int row0, int h, uint64_t* bar) {
  tma_load_3d(dst, tmHi, 0, row0, h, bar);
  tma_load_3d(dst + 16384, tmHi, 64, row0, h, bar);
  tma_load_3d(dst + 32768, tmLo, 0, row0, h, bar);
  tma_load_3d(dst + 49152, tmLo, 64, row0, h, bar);
}

template <int B>
__global__ void __launch_bounds__(kGThreads, 1)
k_gram_tc(const __grid_constant__ CUtensorMap tmHi, const __grid_constant__ CUtensorMap tmLo,
          const int L, const int H, const int T, float* __restrict__ cells) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* base =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  unsigned char* sA = base;                      // 64 KB
  unsigned char* sB = sA + kOperandBytes;        // 2 x 64 KB
  GBars* bars = reinterpret_cast<GBars*>(sB + 2 * kOperandBytes);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nT = (L + kTile - 1) / kTile;
  volatile int* abort = &bars->abort;

  if (tid == 0) {
    mbar_init(&bars->afull, 1);
    mbar_init(&bars->afree, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->bfull[s], 1);
      mbar_init(&bars->bempty[s], 1);
      mbar_init(&bars->tfull[s], 1);
      mbar_init(&bars->tempty[s], kGEpiWarps);
    }
    bars->abort = 0;
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc(&bars->tmem_base, 256);
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tmHi);
    tma_prefetch_desc(&tmLo);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (warp == 0) {
    // -------------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int it = 0, rown = 0;
      bool ok = true;
      for (GramWalk w(nT, H); w.valid() && ok; w.next()) {
        if (rown > 0 && !mbar_wait(&bars->afree, (rown - 1) & 1, abort)) break;
        mbar_expect_tx(&bars->afull, kOperandBytes);
        load_operand(sA, &tmHi, &tmLo, w.I * kTile, w.h, &bars->afull);
        ++rown;
        for (int J = w.I; J < nT; ++J) {
          const int s = it & 1, ph = (it >> 1) & 1;
          if (!mbar_wait(&bars->bempty[s], ph ^ 1, abort)) {
            ok = false;
            break;
          }
          mbar_expect_tx(&bars->bfull[s], kOperandBytes);
          load_operand(sB + s * kOperandBytes, &tmHi, &tmLo, J * kTile, w.h, &bars->bfull[s]);
          ++it;
        }
      }
      if (*abort) {   // let the copies in flight land before the shared memory goes away
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 20000ull) {
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(128, kTile);
      const uint32_t a0 = umma_desc_lo(smem_u32(sA)), b0 = umma_desc_lo(smem_u32(sB));
      int it = 0, rown = 0;
      bool ok = true;
      for (GramWalk w(nT, H); w.valid() && ok; w.next()) {
        if (!mbar_wait(&bars->afull, rown & 1, abort)) break;
        ++rown;
        for (int J = w.I; J < nT; ++J) {
          const int s = it & 1, ph = (it >> 1) & 1;
          if (!mbar_wait(&bars->bfull[s], ph, abort) || !mbar_wait(&bars->tempty[s], ph ^ 1, abort)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t bs = b0 + (uint32_t)s * (kOperandBytes >> 4);
          // x^.y^ = hi.hi + hi.lo + lo.hi (lo.lo is below 2^-17): parts (A, B) = (0,0), (0,1), (1,0)
#pragma unroll
          for (int seg = 0; seg < 3; ++seg) {
            const uint32_t pa = (seg == 2 ? 32768u : 0u) >> 4, pb = (seg == 1 ? 32768u : 0u) >> 4;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint32_t o = (uint32_t)((ks >> 2) * (16384 >> 4) + (ks & 3) * 2);
              if (seg == 0 && ks == 0)
                umma_bf16_lo<0>(tmem + s * 128, a0 + pa + o, bs + pb + o, idesc);
              else
                umma_bf16_lo<1>(tmem + s * 128, a0 + pa + o, bs + pb + o, idesc);
            }
          }
          umma_commit(&bars->bempty[s]);
          umma_commit(&bars->tfull[s]);
          ++it;
        }
        umma_commit(&bars->afree);
      }
    }
  } else if (warp >= kGEpiWarp0) {
    // -------------------------------------------------------------------- epilogue
    // warp % 4 = TMEM lane quarter (32 rows of the tile), (warp - 4) / 4 = 64-column half.
    const int quarter = warp & 3, ch = (warp - kGEpiWarp0) >> 2;
    const int r = quarter * 32 + lane;
    constexpr int G = 32 / B;   // cells per 32-column chunk and row group
    int it = 0;
    bool ok = true;
    for (GramWalk w(nT, H); w.valid() && ok; w.next()) {
      const int i = w.I * kTile + r;            // row of the matrix
      const int ci = i / B;                     // its cell row
      const int nI = min(B, L - ci * B);
      float* out = cells + (size_t)w.h * T * T;
      for (int J = w.I; J < nT; ++J) {
        const int s = it & 1, ph = (it >> 1) & 1;
        if (!mbar_wait(&bars->tfull[s], ph, abort)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + s * 128 + ch * 64;
#pragma unroll 1
        for (int k = 0; k < 2; ++k) {
          uint32_t v[32];
          tmem_ld32(taddr + k * 32, v);
          tmem_ld_wait();
          tmem_ld_fence(v);
          const int c0 = ch * 64 + k * 32;      // first column of the chunk inside the tile
          if (J == w.I) {                       // the pairs i == j are left out
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (c0 + j == r) v[j] = 0u;
          }
          float sgrp[G];
#pragma unroll
          for (int g = 0; g < G; ++g) {
            float t = __uint_as_float(v[g * B]);
#pragma unroll
            for (int e = 1; e < B; ++e) t += __uint_as_float(v[g * B + e]);
            sgrp[g] = t;
          }
#pragma unroll
          for (int o = 1; o < B; o <<= 1)
#pragma unroll
            for (int g = 0; g < G; ++g) sgrp[g] += __shfl_xor_sync(0xffffffffu, sgrp[g], o);
          if (B == 1 && (T & 3) == 0 && ci < T) {
            // one row per thread: 16-byte stores along the row, the mirrored cells lane by lane
            // (consecutive lanes, consecutive addresses)
            const int cj0 = J * kTile + c0;
            if (cj0 < T) {
#pragma unroll
              for (int g = 0; g < 32; g += 4) {
                if (cj0 + g < T) {
                  float4 q4;
                  q4.x = ci != cj0 + g ? sgrp[g] : 0.f;
                  q4.y = ci != cj0 + g + 1 ? sgrp[g + 1] : 0.f;
                  q4.z = ci != cj0 + g + 2 ? sgrp[g + 2] : 0.f;
                  q4.w = ci != cj0 + g + 3 ? sgrp[g + 3] : 0.f;
                  *reinterpret_cast<float4*>(out + (size_t)ci * T + cj0 + g) = q4;
                }
              }
              if (J != w.I) {
#pragma unroll
                for (int g = 0; g < 32; ++g)
                  if (cj0 + g < T) out[(size_t)(cj0 + g) * T + ci] = sgrp[g];
              }
            }
          } else if ((lane & (B - 1)) == 0 && ci < T) {
            const int cj0 = (J * kTile + c0) / B;
#pragma unroll
            for (int g = 0; g < G; ++g) {
              const int cj = cj0 + g;
              if (cj < T) {
                const int nJ = min(B, L - cj * B);
                const float pairs = ci != cj ? (float)(nI * nJ) : (float)(nI * (nI - 1));
                const float val = pairs > 0.f ? sgrp[g] / pairs : 0.f;
                out[(size_t)ci * T + cj] = val;
                if (J != w.I) out[(size_t)cj * T + ci] = val;   // the mirrored tile
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->tempty[s]);
        ++it;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 256);
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

template <int B>
cudaError_t launch_gram(const CUtensorMap& tmHi, const CUtensorMap& tmLo, int L, int H, int T,
                        float* cells, cudaStream_t s) {
  static bool done[64] = {false};
  const size_t smem = 1024 + 3 * (size_t)kOperandBytes + sizeof(GBars);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !done[dev]) {
    e = cudaFuncSetAttribute(k_gram_tc<B>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) done[dev] = true;
  }
  const int nT = (L + kTile - 1) / kTile;
  const int items = H * ((nT + 1) / 2);
  const int grid = items < device_sm_count() ? items : device_sm_count();
  k_gram_tc<B><<<grid, kGThreads, smem, s>>>(tmHi, tmLo, L, H, T, cells);
  return cudaGetLastError();
}

}  // namespace

bool similarity_dense_block(int block) {
  return block == 1 || block == 2 || block == 4 || block == 8 || block == 16;
}

size_t similarity_dense_workspace(int heads, int L) {
  const size_t S = ((size_t)L + kURows - 1) / kURows;
  return 2 * align256((size_t)heads * L * kHeadDim * 2) + align256((size_t)heads * S * kHeadDim * 4) +
         align256((size_t)heads * S * 4);
}

// Dense route of mixkv_similarity_map.  u_out / nz_out / slices_out: the per-slice unit-row sums
// for the head mean.
cudaError_t launch_similarity_dense(const void* X, int heads, int L, int block, void* workspace,
                                    float* cells, float** u_out, int** nz_out, int* slices_out,
                                    cudaStream_t s) {
  unsigned char* wsb = reinterpret_cast<unsigned char*>(workspace);
  __nv_bfloat16* hi = reinterpret_cast<__nv_bfloat16*>(wsb);
  wsb += align256((size_t)heads * L * kHeadDim * 2);
  __nv_bfloat16* lo = reinterpret_cast<__nv_bfloat16*>(wsb);
  wsb += align256((size_t)heads * L * kHeadDim * 2);
  const int S = (L + kURows - 1) / kURows;
  float* u = reinterpret_cast<float*>(wsb);
  wsb += align256((size_t)heads * S * kHeadDim * 4);
  int* nz = reinterpret_cast<int*>(wsb);
  k_unit_rows<<<dim3((unsigned)S, (unsigned)heads), kUThreads, 0, s>>>(
      reinterpret_cast<const __nv_bfloat16*>(X), L, hi, lo, u, nz);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  CUtensorMap tmHi, tmLo;
  const unsigned long long dims[3] = {(unsigned long long)kHeadDim, (unsigned long long)L,
                                      (unsigned long long)heads};
  const unsigned long long strides[2] = {(unsigned long long)kHeadDim * 2,
                                         (unsigned long long)L * kHeadDim * 2};
  const unsigned box[3] = {64, (unsigned)kTile, 1};
  if (!encode_bf16_map(&tmHi, hi, 3, dims, strides, box) ||
      !encode_bf16_map(&tmLo, lo, 3, dims, strides, box))
    return cudaErrorInvalidValue;
  const int T = (L + block - 1) / block;
  switch (block) {
    case 1: e = launch_gram<1>(tmHi, tmLo, L, heads, T, cells, s); break;
    case 2: e = launch_gram<2>(tmHi, tmLo, L, heads, T, cells, s); break;
    case 4: e = launch_gram<4>(tmHi, tmLo, L, heads, T, cells, s); break;
    case 8: e = launch_gram<8>(tmHi, tmLo, L, heads, T, cells, s); break;
    default: e = launch_gram<16>(tmHi, tmLo, L, heads, T, cells, s); break;
  }
  *u_out = u;
  *nz_out = nz;
  *slices_out = S;
  return e;
}

}  // namespace mixkv
