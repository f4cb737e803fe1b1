// The two passes over K (and the one pass over V) of the MixKV scoring step as persistent,
// warp-specialised sm_100a kernels: TMA tile loads into 128-byte-swizzled shared memory,
// tcgen05.mma (bf16 x bf16 -> fp32) with accumulators in tensor memory, and an epilogue that
// reads the accumulators back with tcgen05.ld.
//
//   pass 1  logits with the window queries on the M side (one query row per TMEM lane), so
//           the running softmax (max, sum) of a row is thread-local; alongside, key norms and
//           the sum of unit keys from the shared-memory tile, and value norms streamed from
//           global memory.
//   pass 2  logits with the keys on the M side (one key per TMEM lane), normalised with the
//           finished row statistics, so the column sum over window rows and query heads is
//           thread-local -> s_ex_raw.  The mean unit key rides along as three extra bf16
//           "query" rows (hi / lo / lo2 split) -> K_i . kbar -> s_div.
//
// Paper: extrinsic importance and diversity of Sec. 3.2, redundancy of Eq. 3-4.
#include <cuda.h>

#include "tc_common.cuh"

namespace mixkv {

namespace {

constexpr int kStages = 4;                 // K tile ring
constexpr int kTileBytes = kTile * 256;    // 128 keys x 128 bf16
constexpr int kHalfBytes = kTile * 128;    // one 64-column half of a K tile

// warp roles
constexpr int kWarpTma = 0, kWarpMma = 1;
constexpr int kEpiWarp0 = 4, kEpiWarps = 8;      // warps 4..11: warp % 4 = TMEM lane quarter
constexpr int kEpiThreads = kEpiWarps * 32;

struct PipeBars {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint64_t qfull;
  uint64_t qfree;
  uint64_t kbready;
  uint32_t tmem_base;
  int abort;
  int vote[4][2];
};

// Named barrier among n threads that also agrees on whether to stop: the leader samples the
// CTA abort flag before the barrier and everybody reads that sample after it, so a group
// never splits around a later barrier.
__device__ __forceinline__ bool group_sync_stop(int id, int n, bool leader, volatile int* abort,
                                                volatile int* slots, int it) {
  if (leader) slots[it & 1] = *abort;
  named_bar_sync(id, n);
  return slots[it & 1] != 0;
}

__device__ __forceinline__ void raise(int* status, volatile int* abort) {
  *abort = 1;
  if (status) atomicExch(status, MIXKV_ERR_TIMEOUT);
}

// ======================================================================== pass 1
// grid = g1 persistent CTAs, 18 warps: TMA, MMA, 2 idle, 8 epilogue, 4 key-statistics,
// 2+2 value-norm warps.
constexpr int kP1Threads = 18 * 32;
constexpr int kKsWarp0 = 12;   // warps 12..15

template <int MB>
__global__ void __launch_bounds__(kP1Threads, 1)
k_pass1_tc(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
           const SeqTable st, const __nv_bfloat16* __restrict__ V, const Workspace ws,
           const float scale_log2e, const int use_vnorm, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* base =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  constexpr int QR = MB * 128;                 // query rows the MMA reads
  unsigned char* sQ = base;                    // 2 halves x [QR x 128 B]
  unsigned char* sK = sQ + 2 * QR * 128;       // kStages x 32 KB
  float* skinv = reinterpret_cast<float*>(sK + kStages * kTileBytes);  // [kStages][128]
  float* sks = skinv + kStages * 128;          // [2][128] key-sum exchange
  float* svr = sks + 256;                      // [16] value-stat exchange
  PipeBars* bars = reinterpret_cast<PipeBars*>(svr + 16);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int NQ = st.NQ, W = st.W, H = st.H;
  const int lo = cta_first_tile(blockIdx.x, st.nt1, st.g1);
  const int hi = cta_first_tile(blockIdx.x + 1, st.nt1, st.g1);
  volatile int* abort = &bars->abort;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1 + 4);   // MMA commit + 4 key-statistics warps
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->tfull[s], 1);
      mbar_init(&bars->tempty[s], kEpiThreads);
    }
    mbar_init(&bars->qfull, 1);
    mbar_init(&bars->qfree, 1);
    mbar_init(&bars->kbready, 1);
    bars->abort = 0;
    mbar_init_fence();
  }
  // rows of the query tile beyond NQ are never loaded: clear them once
  for (int i = tid; i < 2 * (QR - NQ) * 8; i += kP1Threads) {
    const int half = i / ((QR - NQ) * 8), rem = i % ((QR - NQ) * 8);
    const int r = NQ + rem / 8, c = rem % 8;
    *reinterpret_cast<uint4*>(sQ + half * QR * 128 + sw128_offset(r, c)) = make_uint4(0, 0, 0, 0);
  }
  fence_proxy_async_smem();
  if (warp == kWarpMma) tmem_alloc(&bars->tmem_base, MB * 256);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (warp == kWarpTma) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tmK);
      tma_prefetch_desc(&tmQ);
      int it = 0, segn = 0, prev_bh = -1;
      for (int id = lo; id < hi; ++id) {
        const TileCoord tc = tile_coord(st.tile1_start, st.batch, H, id);
        if (tc.bh != prev_bh) {
          if (segn > 0 && !mbar_wait(&bars->qfree, (segn - 1) & 1, abort)) break;
          mbar_expect_tx(&bars->qfull, NQ * 256);
          tma_load_2d(sQ, &tmQ, 0, tc.bh * NQ, &bars->qfull);
          tma_load_2d(sQ + QR * 128, &tmQ, 64, tc.bh * NQ, &bars->qfull);
          ++segn;
          prev_bh = tc.bh;
        }
        const int s = it % kStages, ph = (it / kStages) & 1;
        if (!mbar_wait(&bars->empty[s], ph ^ 1, abort)) break;
        mbar_expect_tx(&bars->full[s], kTileBytes);
        const int y = st.cu[tc.b] + tc.t * kTile;
        tma_load_3d(sK + s * kTileBytes, &tmK, 0, y, tc.h, &bars->full[s]);
        tma_load_3d(sK + s * kTileBytes + kHalfBytes, &tmK, 64, y, tc.h, &bars->full[s]);
        ++it;
      }
      if (*abort) {  // let the copies in flight land before the CTA goes away
        raise(status, abort);
        for (int k = max(0, it - kStages); k < it; ++k) {
          const unsigned long long t0 = global_ns();
          while (!mbar_try(&bars->full[k % kStages], (k / kStages) & 1) &&
                 global_ns() - t0 < kWaitLimitNs) {
          }
        }
      }
    }
  } else if (warp == kWarpMma) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(128, kTile);
      int it = 0, segn = 0, prev_bh = -1;
      for (int id = lo; id < hi; ++id) {
        const TileCoord tc = tile_coord(st.tile1_start, st.batch, H, id);
        if (tc.bh != prev_bh) {
          if (!mbar_wait(&bars->qfull, segn & 1, abort)) break;
          ++segn;
          prev_bh = tc.bh;
        }
        const int s = it % kStages, ph = (it / kStages) & 1, ts = it & 1, tph = (it >> 1) & 1;
        if (!mbar_wait(&bars->full[s], ph, abort)) break;
        if (!mbar_wait(&bars->tempty[ts], tph ^ 1, abort)) break;
        tc_fence_after();
        const uint32_t kaddr = smem_u32(sK + s * kTileBytes);
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint64_t da =
                umma_desc_sw128(smem_u32(sQ) + (ks >> 2) * QR * 128 + mb * 16384 + (ks & 3) * 32);
            const uint64_t db = umma_desc_sw128(kaddr + (ks >> 2) * kHalfBytes + (ks & 3) * 32);
            umma_bf16(tmem + ts * (MB * 128) + mb * 128, da, db, idesc, ks > 0);
          }
        }
        umma_commit(&bars->empty[s]);
        umma_commit(&bars->tfull[ts]);
        bool last = id + 1 == hi;
        if (!last) last = tile_coord(st.tile1_start, st.batch, H, id + 1).bh != tc.bh;
        if (last) umma_commit(&bars->qfree);
        ++it;
      }
      if (*abort) raise(status, abort);
    }
  } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kEpiWarps) {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3, wg = (warp - kEpiWarp0) >> 2;
    const int row = (MB == 2 ? wg * 128 : 0) + quarter * 32 + lane;
    const int unit = MB == 2 ? 0 : wg;
    constexpr int NC = MB == 2 ? 128 : 64;       // columns (keys) this thread reduces per tile
    const int col0 = MB == 2 ? wg * 128 : wg * 64;
    const bool warp_on = (MB == 2 ? wg * 128 : 0) + quarter * 32 < NQ;
    const int jrow = row % W;
    float m_run = -1e30f, z_run = 0.f;
    int it = 0, prev_bh = -1, seg_first = lo;
    for (int id = lo; id < hi; ++id) {
      const TileCoord tc = tile_coord(st.tile1_start, st.batch, H, id);
      if (tc.bh != prev_bh) {
        m_run = -1e30f;
        z_run = 0.f;
        seg_first = id;
        prev_bh = tc.bh;
      }
      const int L = st.cu[tc.b + 1] - st.cu[tc.b], P = L - W;
      const int ts = it & 1, tph = (it >> 1) & 1;
      if (!mbar_wait(&bars->tfull[ts], tph, abort)) break;
      tc_fence_after();
      if (warp_on) {
        const int k0 = tc.t * kTile + (MB == 2 ? 0 : wg * 64);
        const bool need_mask = tc.t * kTile + kTile > P;
        const int lim = P + jrow;   // last key this row may see
        const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + ts * (MB * 128) + col0;
#pragma unroll 1
        for (int c0 = 0; c0 < NC; c0 += 32) {
          uint32_t ra[16], rb[16];
          tmem_ld16(taddr + c0, ra);
          tmem_ld16(taddr + c0 + 16, rb);
          tmem_ld_wait();
          tmem_ld_fence(ra);
          tmem_ld_fence(rb);
          if (need_mask) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              if (k0 + c0 + j > lim) ra[j] = 0xff800000u;        // -inf
              if (k0 + c0 + 16 + j > lim) rb[j] = 0xff800000u;
            }
          }
          float mx = fmaxf(__uint_as_float(ra[0]), __uint_as_float(rb[0]));
#pragma unroll
          for (int j = 1; j < 16; ++j)
            mx = fmaxf(mx, fmaxf(__uint_as_float(ra[j]), __uint_as_float(rb[j])));
          const float mn = fmaxf(m_run, mx * scale_log2e);
          if (mn > m_run) {
            z_run *= ex2(m_run - mn);
            m_run = mn;
          }
          float z0 = 0.f, z1 = 0.f;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            z0 += ex2(fmaf(__uint_as_float(ra[j]), scale_log2e, -m_run));
            z1 += ex2(fmaf(__uint_as_float(rb[j]), scale_log2e, -m_run));
          }
          z_run += z0 + z1;
        }
      }
      tc_fence_before();
      mbar_arrive(&bars->tempty[ts]);
      bool last = id + 1 == hi;
      if (!last) last = tile_coord(st.tile1_start, st.batch, H, id + 1).bh != tc.bh;
      if (last && row < NQ)
        ws.rowstat[((size_t)seg_first * 2 + unit) * NQ + row] = make_float2(m_run, z_run);
      ++it;
    }
  } else if (warp >= kKsWarp0 && warp < kKsWarp0 + 4) {
    // ------------------------------------------------------------------ key statistics
    const int kt = tid - kKsWarp0 * 32;          // 0..127: key row of the tile (norm phase)
    const int wd = kt & 63, hk = kt >> 6;        // word (dims 2wd, 2wd+1) and key half (sum phase)
    float a0 = 0.f, a1 = 0.f;
    int it = 0, prev_bh = -1, seg_first = lo;
    for (int id = lo; id < hi; ++id) {
      const TileCoord tc = tile_coord(st.tile1_start, st.batch, H, id);
      if (tc.bh != prev_bh) {
        a0 = a1 = 0.f;
        seg_first = id;
        prev_bh = tc.bh;
      }
      const int L = st.cu[tc.b + 1] - st.cu[tc.b];
      const int s = it % kStages, ph = (it / kStages) & 1;
      mbar_wait(&bars->full[s], ph, abort);
      const unsigned char* tile = sK + s * kTileBytes;
      float ss = 0.f;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint4 u = *reinterpret_cast<const uint4*>(tile + half * kHalfBytes + sw128_offset(kt, c));
          const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(p2[e]);
            ss = fmaf(f.x, f.x, ss);
            ss = fmaf(f.y, f.y, ss);
          }
        }
      }
      const int i = tc.t * kTile + kt;
      const float inv = (i < L && ss > 0.f) ? 1.0f / sqrtf(ss) : 0.f;
      skinv[s * 128 + kt] = inv;
      if (i < L) ws.kinv[(size_t)tc.h * st.Ltot + st.cu[tc.b] + i] = inv;
      if (group_sync_stop(2, 128, kt == 0, abort, bars->vote[0], it)) break;
      {
        const unsigned char* colbase = tile + (wd >> 5) * kHalfBytes + (wd & 3) * 4;
        const int chunk = (wd & 31) >> 2;
#pragma unroll 8
        for (int rr = 0; rr < 64; ++rr) {
          const int r = hk * 64 + rr;
          const float2 f = __bfloat1622float2(
              *reinterpret_cast<const __nv_bfloat162*>(colbase + sw128_offset(r, chunk)));
          const float w = skinv[s * 128 + r];
          a0 = fmaf(f.x, w, a0);
          a1 = fmaf(f.y, w, a1);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->empty[s]);
      bool last = id + 1 == hi;
      if (!last) last = tile_coord(st.tile1_start, st.batch, H, id + 1).bh != tc.bh;
      if (last) {
        sks[hk * 128 + 2 * wd] = a0;
        sks[hk * 128 + 2 * wd + 1] = a1;
        named_bar_sync(2, 128);
        ws.ksum[(size_t)seg_first * kHeadDim + kt] = sks[kt] + sks[128 + kt];
        named_bar_sync(2, 128);
      }
      ++it;
    }
  } else if (use_vnorm) {
    // ------------------------------------------------------------------ value norms
    // warps 2, 3, 16, 17: each takes a quarter of the tile's rows, half a warp per row
    const int vw = warp < 4 ? warp - 2 : warp - 14;   // 0..3
    const int hw = lane >> 4, hl = lane & 15;
    float vmin = INFINITY, vmax = -INFINITY, vsum = 0.f;
    int prev_bh = -1, seg_first = lo;
    for (int id = lo; id < hi; ++id) {
      const TileCoord tc = tile_coord(st.tile1_start, st.batch, H, id);
      if (tc.bh != prev_bh) {
        vmin = INFINITY, vmax = -INFINITY, vsum = 0.f;
        seg_first = id;
        prev_bh = tc.bh;
      }
      const int P = st.cu[tc.b + 1] - st.cu[tc.b] - W;
      const size_t row0 = (size_t)tc.h * st.Ltot + st.cu[tc.b];
      const size_t poff = (size_t)tc.h * st.Ptot + (st.cu[tc.b] - tc.b * W);
      const int ibase = tc.t * kTile + vw * 32 + hw;
      if (tc.t * kTile + vw * 32 < P) {
#pragma unroll 1
        for (int kb = 0; kb < 16; kb += 8) {
          uint4 u[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const int i = ibase + 2 * (kb + k);
            u[k] = make_uint4(0, 0, 0, 0);
            if (i < P)
              u[k] = __ldg(reinterpret_cast<const uint4*>(V + (row0 + i) * kHeadDim) + hl);
          }
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const int i = ibase + 2 * (kb + k);
            const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&u[k]);
            float ss = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 f = __bfloat1622float2(p2[e]);
              ss = fmaf(f.x, f.x, ss);
              ss = fmaf(f.y, f.y, ss);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
            if (i < P && hl == 0) {
              const float n = sqrtf(ss);
              ws.vnorm[poff + i] = n;
              vmin = fminf(vmin, n);
              vmax = fmaxf(vmax, n);
              vsum += n;
            }
          }
        }
      }
      bool last = id + 1 == hi;
      if (!last) last = tile_coord(st.tile1_start, st.batch, H, id + 1).bh != tc.bh;
      if (last) {
        const float a = warp_min(vmin), b2 = warp_max(vmax), c2 = warp_sum(vsum);
        if (lane == 0) {
          svr[vw] = a;
          svr[4 + vw] = b2;
          svr[8 + vw] = c2;
        }
        named_bar_sync(3, 128);
        if (vw == 0 && lane == 0) {
          ws.vstat[seg_first] = make_float4(
              fminf(fminf(svr[0], svr[1]), fminf(svr[2], svr[3])),
              fmaxf(fmaxf(svr[4], svr[5]), fmaxf(svr[6], svr[7])),
              (svr[8] + svr[9]) + (svr[10] + svr[11]), 0.f);
        }
        named_bar_sync(3, 128);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kWarpMma) tmem_dealloc(tmem, MB * 256);
  if (tid == 0 && bars->abort && status) atomicExch(status, MIXKV_ERR_TIMEOUT);
}

// ======================================================================== pass 2
// grid = g2 persistent CTAs, 12 warps: TMA, MMA, 2 preparation, 8 epilogue.
constexpr int kP2Threads = 12 * 32;

__global__ void __launch_bounds__(kP2Threads, 1)
k_pass2_tc(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
           const SeqTable st, const Workspace ws, float* __restrict__ s_div_out,
           const float scale_log2e, const int use_vnorm, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* base =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  const int NQ = st.NQ, W = st.W, H = st.H;
  const int NB = NQ + kExtraRows;             // rows of the B operand
  unsigned char* sQ = base;                   // 2 halves x [NB x 128 B]
  unsigned char* sK = sQ + 2 * (kMaxNQ + kExtraRows) * 128;  // kStages x 32 KB
  float* sbq = reinterpret_cast<float*>(sK + kStages * kTileBytes);  // [256]
  float* sx = sbq + 256;                      // [2][128] partial sums WG0 -> WG1
  float* sred = sx + 256;                     // [32]
  float* sksp = sred + 32;                    // [2][128] unit-key sums of the two prep warps
  float2* spart = reinterpret_cast<float2*>(sksp + 256);   // [8][256] per-warp row statistics
  PipeBars* bars = reinterpret_cast<PipeBars*>(spart + 8 * 256);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int lo = cta_first_tile(blockIdx.x, st.nt2, st.g2);
  const int hi = cta_first_tile(blockIdx.x + 1, st.nt2, st.g2);
  volatile int* abort = &bars->abort;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->tfull[s], 1);
      mbar_init(&bars->tempty[s], kEpiThreads);
    }
    mbar_init(&bars->qfull, 1);
    mbar_init(&bars->qfree, 1);
    mbar_init(&bars->kbready, 2);
    bars->abort = 0;
    mbar_init_fence();
  }
  if (warp == kWarpMma) tmem_alloc(&bars->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (warp == kWarpTma) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tmK);
      tma_prefetch_desc(&tmQ);
      int it = 0, segn = 0, prev_bh = -1;
      for (int id = lo; id < hi; ++id) {
        const TileCoord tc = tile_coord(st.tile2_start, st.batch, H, id);
        if (tc.bh != prev_bh) {
          if (segn > 0 && !mbar_wait(&bars->qfree, (segn - 1) & 1, abort)) break;
          mbar_expect_tx(&bars->qfull, NQ * 256);
          tma_load_2d(sQ, &tmQ, 0, tc.bh * NQ, &bars->qfull);
          tma_load_2d(sQ + NB * 128, &tmQ, 64, tc.bh * NQ, &bars->qfull);
          ++segn;
          prev_bh = tc.bh;
        }
        const int s = it % kStages, ph = (it / kStages) & 1;
        if (!mbar_wait(&bars->empty[s], ph ^ 1, abort)) break;
        mbar_expect_tx(&bars->full[s], kTileBytes);
        const int y = st.cu[tc.b] + tc.t * kTile;
        tma_load_3d(sK + s * kTileBytes, &tmK, 0, y, tc.h, &bars->full[s]);
        tma_load_3d(sK + s * kTileBytes + kHalfBytes, &tmK, 64, y, tc.h, &bars->full[s]);
        ++it;
      }
      if (*abort) {
        raise(status, abort);
        for (int k = max(0, it - kStages); k < it; ++k) {
          const unsigned long long t0 = global_ns();
          while (!mbar_try(&bars->full[k % kStages], (k / kStages) & 1) &&
                 global_ns() - t0 < kWaitLimitNs) {
          }
        }
      }
    }
  } else if (warp == kWarpMma) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(128, NB);
      int it = 0, segn = 0, prev_bh = -1;
      for (int id = lo; id < hi; ++id) {
        const TileCoord tc = tile_coord(st.tile2_start, st.batch, H, id);
        if (tc.bh != prev_bh) {
          if (!mbar_wait(&bars->qfull, segn & 1, abort)) break;
          if (!mbar_wait(&bars->kbready, segn & 1, abort)) break;
          ++segn;
          prev_bh = tc.bh;
        }
        const int s = it % kStages, ph = (it / kStages) & 1, ts = it & 1, tph = (it >> 1) & 1;
        if (!mbar_wait(&bars->full[s], ph, abort)) break;
        if (!mbar_wait(&bars->tempty[ts], tph ^ 1, abort)) break;
        tc_fence_after();
        const uint32_t kaddr = smem_u32(sK + s * kTileBytes);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t da = umma_desc_sw128(kaddr + (ks >> 2) * kHalfBytes + (ks & 3) * 32);
          const uint64_t db = umma_desc_sw128(smem_u32(sQ) + (ks >> 2) * NB * 128 + (ks & 3) * 32);
          umma_bf16(tmem + ts * 256, da, db, idesc, ks > 0);
        }
        umma_commit(&bars->empty[s]);
        umma_commit(&bars->tfull[ts]);
        bool last = id + 1 == hi;
        if (!last) last = tile_coord(st.tile2_start, st.batch, H, id + 1).bh != tc.bh;
        if (last) umma_commit(&bars->qfree);
        ++it;
      }
      if (*abort) raise(status, abort);
    }
  } else if (warp == 2 || warp == 3) {
    // ------------------------------------------------------------------ preparation
    // Per segment: merge pass 1's unit-key sums of this (b, h) into the mean unit key, write
    // its bf16 hi / lo / lo2 split into the three extra B rows, and publish rbar (Eq. 4) and
    // the value-norm statistics once per (b, h).
    const int pt = tid - 64;   // 0..63 -> dims 2pt, 2pt+1
    int segn = 0, prev_bh = -1;
    for (int id = lo; id < hi; ++id) {
      const TileCoord tc = tile_coord(st.tile2_start, st.batch, H, id);
      if (tc.bh == prev_bh) continue;
      prev_bh = tc.bh;
      const int L = st.cu[tc.b + 1] - st.cu[tc.b];
      const int per_head = (st.tile1_start[tc.b + 1] - st.tile1_start[tc.b]) / H;
      const int T0 = st.tile1_start[tc.b] + tc.h * per_head;
      // pass 1 left one partial sum per segment of this (b, h): segment e starts at T0 for
      // e = 0 and at the first tile of CTA c0 + e otherwise
      const int c0 = tile_owner(T0, st.nt1, st.g1);
      const int nseg = tile_owner(T0 + per_head - 1, st.nt1, st.g1) - c0 + 1;
      {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
        for (int e = warp - 2; e < nseg; e += 2) {
          const int start = e == 0 ? T0 : cta_first_tile(c0 + e, st.nt1, st.g1);
          const float4 f = *reinterpret_cast<const float4*>(ws.ksum + (size_t)start * kHeadDim + 4 * lane);
          acc.x += f.x, acc.y += f.y, acc.z += f.z, acc.w += f.w;
        }
        named_bar_sync(4, 64);   // the previous segment's readers of sksp are done
        *reinterpret_cast<float4*>(sksp + (warp - 2) * 128 + 4 * lane) = acc;
        named_bar_sync(4, 64);
      }
      const float s0 = sksp[2 * pt] + sksp[128 + 2 * pt];
      const float s1 = sksp[2 * pt + 1] + sksp[128 + 2 * pt + 1];
      const bool owner = tc.t == 0;
      if (owner) {
        float n2 = warp_sum(s0 * s0 + s1 * s1);
        if (lane == 0) sred[warp] = n2;
      }
      const float invL = 1.0f / (float)L;
      float kb[2] = {s0 * invL, s1 * invL};
      __nv_bfloat16 parts[3][2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        parts[0][e] = __float2bfloat16_rn(kb[e]);
        const float r1 = kb[e] - __bfloat162float(parts[0][e]);
        parts[1][e] = __float2bfloat16_rn(r1);
        parts[2][e] = __float2bfloat16_rn(r1 - __bfloat162float(parts[1][e]));
      }
      if (segn > 0) {   // the previous segment's MMAs must be done with the B rows
        if (pt == 0) mbar_wait(&bars->qfree, (segn - 1) & 1, abort);
        if (group_sync_stop(4, 64, pt == 0, abort, bars->vote[1], segn)) break;
      }
      {
        const int col = 2 * pt, half = col >> 6, cin = col & 63;
        unsigned char* hb = sQ + half * NB * 128 + (cin & 7) * 2;
#pragma unroll
        for (int e = 0; e < kExtraRows; ++e) {
          __nv_bfloat162 v2;
          v2.x = e < 3 ? parts[e][0] : __float2bfloat16_rn(0.f);
          v2.y = e < 3 ? parts[e][1] : __float2bfloat16_rn(0.f);
          if (e < 3 || segn == 0)
            *reinterpret_cast<__nv_bfloat162*>(hb + sw128_offset(NQ + e, cin >> 3)) = v2;
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->kbready);
      if (owner) {
        named_bar_sync(4, 64);
        if (pt == 0) {
          const double n2 = (double)sred[2] + (double)sred[3];
          const double T = (double)L;
          ws.rbar[tc.bh] = (float)((n2 - T) / (T * (T - 1.0)));   // Eq. 4
        }
        if (use_vnorm && warp == 3) {
          float a = INFINITY, b2 = -INFINITY, c2 = 0.f;
          for (int e = lane; e < nseg; e += 32) {
            const int start = e == 0 ? T0 : cta_first_tile(c0 + e, st.nt1, st.g1);
            const float4 v = ws.vstat[start];
            a = fminf(a, v.x);
            b2 = fmaxf(b2, v.y);
            c2 += v.z;
          }
          a = warp_min(a);
          b2 = warp_max(b2);
          c2 = warp_sum(c2);
          if (lane == 0) ws.vfinal[tc.bh] = make_float4(a, b2, c2, 0.f);
        }
        named_bar_sync(4, 64);
      }
      ++segn;
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3, wg = (warp - kEpiWarp0) >> 2;
    const int et = tid - kEpiWarp0 * 32;        // 0..255
    const int key = quarter * 32 + lane;
    const int CA = ((NQ + 31) / 32) * 16;       // columns of warpgroup 0; warpgroup 1 takes the rest
    const int cbeg = wg == 0 ? 0 : CA, cend = wg == 0 ? CA : NQ;
    float dmin = INFINITY, dmax = -INFINITY, dsum = 0.f;
    int it = 0, prev_bh = -1, seg_first = lo;
    for (int id = lo; id < hi; ++id) {
      const TileCoord tc = tile_coord(st.tile2_start, st.batch, H, id);
      const int L = st.cu[tc.b + 1] - st.cu[tc.b], P = L - W;
      if (tc.bh != prev_bh) {
        // merge pass 1's per-segment softmax statistics of this (b, h) into one log2
        // normaliser per window row (the 1/W of the window mean folded in)
        named_bar_sync(1, kEpiThreads);
        {
          const int per_head = (st.tile1_start[tc.b + 1] - st.tile1_start[tc.b]) / H;
          const int T0 = st.tile1_start[tc.b] + tc.h * per_head;
          const int c0 = tile_owner(T0, st.nt1, st.g1);
          const int nseg = tile_owner(T0 + per_head - 1, st.nt1, st.g1) - c0 + 1;
          const int nunits = NQ <= 128 ? 2 : 1;
          const int ew = warp - kEpiWarp0;
          float M[8], Z[8];
#pragma unroll
          for (int r = 0; r < 8; ++r) M[r] = -1e30f, Z[r] = 0.f;
          for (int k = ew; k < nseg * nunits; k += kEpiWarps) {
            const int e = k / nunits, u = k - e * nunits;
            const int start = e == 0 ? T0 : cta_first_tile(c0 + e, st.nt1, st.g1);
            const float2* src = ws.rowstat + ((size_t)start * 2 + u) * NQ;
#pragma unroll
            for (int r = 0; r < 8; ++r) {
              const int q = lane + 32 * r;
              if (q < NQ) {
                const float2 mz = src[q];
                const float mn = fmaxf(M[r], mz.x);
                Z[r] = Z[r] * ex2(M[r] - mn) + mz.y * ex2(mz.x - mn);
                M[r] = mn;
              }
            }
          }
#pragma unroll
          for (int r = 0; r < 8; ++r) spart[ew * 256 + lane + 32 * r] = make_float2(M[r], Z[r]);
          named_bar_sync(1, kEpiThreads);
          if (et < NQ) {
            float Mx = -1e30f;
#pragma unroll
            for (int w = 0; w < kEpiWarps; ++w) Mx = fmaxf(Mx, spart[w * 256 + et].x);
            float Zs = 0.f;
#pragma unroll
            for (int w = 0; w < kEpiWarps; ++w) {
              const float2 mz = spart[w * 256 + et];
              Zs += mz.y * exp2f(mz.x - Mx);
            }
            sbq[et] = Mx + log2f(Zs * (float)W);
          }
        }
        dmin = INFINITY, dmax = -INFINITY, dsum = 0.f;
        seg_first = id;
        prev_bh = tc.bh;
        named_bar_sync(1, kEpiThreads);
      }
      const int ts = it & 1, tph = (it >> 1) & 1;
      const int ikey = tc.t * kTile + key;
      float kinv_i = 0.f;
      if (wg == 1 && ikey < P) kinv_i = ws.kinv[(size_t)tc.h * st.Ltot + st.cu[tc.b] + ikey];
      const bool ok = mbar_wait(&bars->tfull[ts], tph, abort);
      tc_fence_after();
      const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + ts * 256;
      float acc0 = 0.f, acc1 = 0.f, dot = 0.f;
      if (ok && cbeg < cend) {
        // 16-column chunks, the next one in flight while this one is reduced
        uint32_t ra[16], rb[16];
        tmem_ld16(taddr + cbeg, ra);
#pragma unroll 1
        for (int c0 = cbeg; c0 < cend; c0 += 32) {
          tmem_ld_wait();
          tmem_ld_fence(ra);
          if (c0 + 16 < cend) tmem_ld16(taddr + c0 + 16, rb);
#pragma unroll
          for (int j = 0; j < 16; j += 4) {
            const float4 nb = *reinterpret_cast<const float4*>(sbq + c0 + j);
            acc0 += ex2(fmaf(__uint_as_float(ra[j]), scale_log2e, -nb.x));
            acc1 += ex2(fmaf(__uint_as_float(ra[j + 1]), scale_log2e, -nb.y));
            acc0 += ex2(fmaf(__uint_as_float(ra[j + 2]), scale_log2e, -nb.z));
            acc1 += ex2(fmaf(__uint_as_float(ra[j + 3]), scale_log2e, -nb.w));
          }
          if (c0 + 16 < cend) {
            tmem_ld_wait();
            tmem_ld_fence(rb);
            if (c0 + 32 < cend) tmem_ld16(taddr + c0 + 32, ra);
#pragma unroll
            for (int j = 0; j < 16; j += 4) {
              const float4 nb = *reinterpret_cast<const float4*>(sbq + c0 + 16 + j);
              acc0 += ex2(fmaf(__uint_as_float(rb[j]), scale_log2e, -nb.x));
              acc1 += ex2(fmaf(__uint_as_float(rb[j + 1]), scale_log2e, -nb.y));
              acc0 += ex2(fmaf(__uint_as_float(rb[j + 2]), scale_log2e, -nb.z));
              acc1 += ex2(fmaf(__uint_as_float(rb[j + 3]), scale_log2e, -nb.w));
            }
          }
        }
      }
      if (wg == 1 && ok) {
        uint32_t r[16];
        tmem_ld16(taddr + NQ, r);
        tmem_ld_wait();
        tmem_ld_fence(r);
        dot = (__uint_as_float(r[0]) + __uint_as_float(r[1])) + __uint_as_float(r[2]);
      }
      tc_fence_before();
      mbar_arrive(&bars->tempty[ts]);
      if (wg == 0) sx[ts * 128 + key] = acc0 + acc1;
      if (group_sync_stop(1, kEpiThreads, et == 0, abort, bars->vote[2], it)) break;
      if (wg == 1) {
        const int i = tc.t * kTile + key;
        if (i < P) {
          const size_t poff = (size_t)tc.h * st.Ptot + (st.cu[tc.b] - tc.b * W);
          ws.s_ex_raw[poff + i] = (acc0 + acc1) + sx[ts * 128 + key];
          const float sd = -dot * kinv_i;
          s_div_out[poff + i] = sd;
          dmin = fminf(dmin, sd);
          dmax = fmaxf(dmax, sd);
          dsum += sd;
        }
        bool last = id + 1 == hi;
        if (!last) last = tile_coord(st.tile2_start, st.batch, H, id + 1).bh != tc.bh;
        if (last) {
          const float a = warp_min(dmin), b2 = warp_max(dmax), c2 = warp_sum(dsum);
          if (lane == 0) {
            sred[8 + quarter] = a;
            sred[12 + quarter] = b2;
            sred[16 + quarter] = c2;
          }
          named_bar_sync(5, 128);
          if (quarter == 0 && lane == 0) {
            ws.dstat[seg_first] = make_float4(
                fminf(fminf(sred[8], sred[9]), fminf(sred[10], sred[11])),
                fmaxf(fmaxf(sred[12], sred[13]), fmaxf(sred[14], sred[15])),
                (sred[16] + sred[17]) + (sred[18] + sred[19]), 0.f);
          }
          named_bar_sync(5, 128);
        }
      }
      ++it;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kWarpMma) tmem_dealloc(tmem, 512);
  if (tid == 0 && bars->abort && status) atomicExch(status, MIXKV_ERR_TIMEOUT);
}

// -------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// K as a 3-D tensor (d, Ltot, H) with boxes of 64 x 128 x 1; Q as 2-D (d, batch*H*NQ) with
// boxes of 64 x NQ.  Rows past the end of the tensor read as zero.
bool make_maps(const LaunchCtx& c, const void* K, const void* Q, CUtensorMap* tmK,
               CUtensorMap* tmQ) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  {
    cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)c.st.Ltot, (cuuint64_t)c.st.H};
    cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)c.st.Ltot * kHeadDim * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)kTile, 1};
    cuuint32_t es[3] = {1, 1, 1};
    if (enc(tmK, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(K), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  {
    cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)c.st.batch * c.st.H * c.st.NQ};
    cuuint64_t strides[1] = {(cuuint64_t)kHeadDim * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)c.st.NQ};
    cuuint32_t es[2] = {1, 1};
    if (enc(tmQ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(Q), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  return true;
}

size_t pass1_smem(int MB) {
  return 1024 + (size_t)2 * MB * 128 * 128 + kStages * kTileBytes + kStages * 128 * 4 + 256 * 4 +
         16 * 4 + sizeof(PipeBars) + 64;
}
size_t pass2_smem() {
  return 1024 + (size_t)2 * (kMaxNQ + kExtraRows) * 128 + kStages * kTileBytes + 256 * 4 +
         256 * 4 + 32 * 4 + 256 * 4 + 8 * 256 * 8 + sizeof(PipeBars) + 64;
}

}  // namespace

int device_sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
      n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

cudaError_t launch_pass1(const LaunchCtx& c, const void* K, const void* V, const void* Q,
                         int* status) {
  CUtensorMap tmK, tmQ;
  if (!make_maps(c, K, Q, &tmK, &tmQ)) return cudaErrorInvalidValue;
  const int MB = c.st.NQ <= 128 ? 1 : 2;
  const size_t smem = pass1_smem(MB);
  auto k = MB == 1 ? k_pass1_tc<1> : k_pass1_tc<2>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  k<<<c.st.g1, kP1Threads, smem, c.stream>>>(tmK, tmQ, c.st, (const __nv_bfloat16*)V, c.ws,
                                             c.scale_log2e, c.p.use_vnorm, status);
  return cudaGetLastError();
}

cudaError_t launch_pass2(const LaunchCtx& c, const void* K, const void* Q, float* s_div_out,
                         int* status) {
  CUtensorMap tmK, tmQ;
  if (!make_maps(c, K, Q, &tmK, &tmQ)) return cudaErrorInvalidValue;
  const size_t smem = pass2_smem();
  cudaError_t e = cudaFuncSetAttribute(k_pass2_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  k_pass2_tc<<<c.st.g2, kP2Threads, smem, c.stream>>>(tmK, tmQ, c.st, c.ws, s_div_out,
                                                      c.scale_log2e, c.p.use_vnorm, status);
  return cudaGetLastError();
}

}  // namespace mixkv
