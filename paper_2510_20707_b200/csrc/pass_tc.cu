// The two passes over K of the MixKV scoring step as persistent, warp-specialised sm_100a
// kernels: TMA tile loads into 128-byte-swizzled shared memory, tcgen05.mma (bf16 x bf16 ->
// fp32) with accumulators in tensor memory, and epilogues that read the accumulators back with
// tcgen05.ld.
//
//   pass 1  K from HBM.  Logits with the window queries on the M side (one query row per TMEM
//           lane), so the running softmax (max, sum) of a row is thread-local; alongside, key
//           norms and the sum of unit keys from the shared-memory tile.
//   pass 2  K again (served by L2), V from HBM.  At the start of a (sequence, head) segment the
//           CTA folds pass 1's per-CTA partials: the softmax statistics become one log2
//           normaliser per window row, the unit-key sums become the mean unit key (bf16 hi /
//           lo / lo2 rows) and the redundancy of Eq. 4.  Logits with the keys on the M side (one key
//           per TMEM lane), normalised with the finished row statistics, so the column sum over
//           window rows and query heads is thread-local -> s_ex_raw.  The mean unit key rides
//           along as three extra bf16 "query" rows -> K_i . kbar -> s_div.  Value norms are
//           computed from V tiles staged next to the K tiles.
//
// Paper: extrinsic importance, VNorm and diversity of Sec. 3.2, redundancy of Eq. 3-4.
#include <cuda.h>

#include "tc_common.cuh"

namespace mixkv {

namespace {

constexpr int kTileBytes = kTile * 256;    // 128 keys x 128 bf16
constexpr int kHalfBytes = kTile * 128;    // one 64-column half of a K tile

// warp roles (16 warps per CTA)
constexpr int kThreads = 16 * 32;
constexpr int kWarpTma = 0, kWarpMma = 1;
constexpr int kEpiWarp0 = 4, kEpiWarps = 8;      // warps 4..11: warp % 4 = TMEM lane quarter
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kAuxWarp0 = 12;                    // warps 12..15: key statistics / value norms

// Named barrier among n threads that also agrees on whether to stop: the leader samples the
// CTA abort flag before the barrier and everybody reads that sample after it, so a group
// never splits around a later barrier.
__device__ __forceinline__ bool group_sync_stop(int id, int n, bool leader, volatile int* abort,
                                                volatile int* slots, int it) {
  if (leader) slots[it & 1] = *abort;
  named_bar_sync(id, n);
  return slots[it & 1] != 0;
}

// Counts a delivered segment of a (layer, sequence, head) whose partial results come from
// `nseg` CTAs; true in the CTA that delivers the last one.  Called by one thread after a CTA
// barrier that follows the writes of the partial results: the release half of the atomic
// publishes them, the acquire half lets the last arrival read everybody's.  The word holds
// (tag << 16 | arrivals).  A word with another tag is left over from an earlier call, or was
// never written, and the first arrival of this call replaces it: the caller's workspace needs
// no clearing between calls.  Once the word carries the tag an arrival is one atomic add (no
// retries when the CTAs of a head finish together).
__device__ __forceinline__ bool arrive_last(unsigned long long* word, const unsigned long long tag,
                                            const int nseg) {
  unsigned long long cur = *reinterpret_cast<volatile unsigned long long*>(word);
  for (;;) {
    if ((cur >> 16) == tag) {
      unsigned long long old;
      asm volatile("atom.add.acq_rel.gpu.global.u64 %0, [%1], %2;"
                   : "=l"(old)
                   : "l"(word), "l"(1ull)
                   : "memory");
      return (int)((old + 1ull) & 0xffffull) == nseg;
    }
    __threadfence();   // release for the plain compare-and-swap below
    const unsigned long long seen = atomicCAS(word, cur, (tag << 16) | 1ull);
    if (seen == cur) return nseg == 1;
    cur = seen;   // another CTA replaced the stale word first (or it changed): look again
  }
}

__device__ __forceinline__ void raise(int* status, volatile int* abort) {
  *abort = 1;
  if (status) atomicExch(status, MIXKV_ERR_TIMEOUT);
}

// After an abort: let the copies in flight land before the CTA (and its shared memory) goes
// away.  `it` loads were issued into a ring of `stages` barriers.
__device__ __forceinline__ void drain_ring(uint64_t* full, int stages, int it) {
  for (int k = max(0, it - stages); k < it; ++k) {
    const unsigned long long t0 = global_ns();
    while (!mbar_try(&full[k % stages], (k / stages) & 1) && global_ns() - t0 < kWaitLimitNs) {
    }
  }
}

// Packed fp32 pairs (one instruction for two lanes of arithmetic).
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
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

constexpr size_t kSmemLimit = 227 * 1024;   // dynamic shared memory a CTA may ask for

// ======================================================================== pass 1
// Key-statistics warps (from warp 12 on): 8 for one 128-row query block, where their latency
// chains set the pace, 4 for two blocks, where the epilogue does.  One tile = 8 pairs of 8-row
// batches, spread evenly over the warps.
__host__ __device__ constexpr int p1_aux_warps(int MB) { return MB == 2 ? 4 : 8; }
__host__ __device__ constexpr int p1_threads(int MB) { return (kAuxWarp0 + p1_aux_warps(MB)) * 32; }
constexpr int kP1MaxStages = 6;
// K tile ring: as deep as shared memory allows next to the query tile (the deeper the ring, the
// more bytes in flight towards HBM)
__host__ __device__ constexpr int p1_stages(int MB) { return 5; }

struct P1Bars {
  uint64_t full[kP1MaxStages];
  uint64_t empty[kP1MaxStages];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint64_t qfull;
  uint64_t qfree;
  uint32_t tmem_base;
  int abort;
  int vote[2];
  int last;   // this CTA delivered the last segment of the head at hand
};

// ---- per-head folds at the end of pass 1 (once per (layer, sequence, head), in the CTA that
// delivers the head's last segment)
//
// All segments' softmax (max, sum) of window row q -> minus the log2 of the row's normaliser.
// NU partial results per segment and row.
template <int NU>
__device__ __forceinline__ float fold_row_stats(const float2* rowstat, const SegList& sl,
                                                const int NQ, const int q) {
  const int total = sl.nseg * NU;
  float Mx = -1e30f, Zs = 0.f;
#pragma unroll 1
  for (int i0 = 0; i0 < total; i0 += 20) {   // twenty loads in flight
    float2 v[20];
#pragma unroll
    for (int k = 0; k < 20; ++k) {
      const int i = i0 + k;
      v[k] = make_float2(-1e30f, 0.f);
      if (i < total) v[k] = __ldcg(rowstat + ((size_t)sl.start(i / NU) * 2 + (i % NU)) * NQ + q);
    }
#pragma unroll
    for (int k = 0; k < 20; ++k) {
      const float mn = fmaxf(Mx, v[k].x);
      Zs = Zs * ex2(Mx - mn) + v[k].y * ex2(v[k].x - mn);
      Mx = mn;
    }
  }
  return -(Mx + log2f(Zs));
}
// Sum over the head's segments of component kt of their unit-key sums.
__device__ __forceinline__ float fold_key_sums(const float* ksum, const SegList& sl, const int kt) {
  float sum = 0.f;
#pragma unroll 1
  for (int e0 = 0; e0 < sl.nseg; e0 += 20) {   // twenty loads in flight
    float v[20];
#pragma unroll
    for (int e = 0; e < 20; ++e)
      v[e] = e0 + e < sl.nseg ? __ldcg(ksum + (size_t)sl.start(e0 + e) * kHeadDim + kt) : 0.f;
#pragma unroll
    for (int e = 0; e < 20; ++e) sum += v[e];
  }
  return sum;
}
// Walks the segments of the CTA's tile range [lo, hi); every thread of the CTA calls it after
// the barrier that ends the tile loops.  Threads 0 .. NQ-1 fold the row statistics, threads
// 256 .. 383 the key sums.  `red` is shared scratch of four floats, `flag` a shared int.
template <int MB>
__device__ __forceinline__ void finish_heads(const SeqTable& st, const Workspace& ws, const int lo,
                                             const int hi, const unsigned long long call_tag,
                                             float* __restrict__ rbar_out, float* red, int* flag) {
  const int tid = threadIdx.x, lane = tid & 31;
  const int NQ = st.NQ, H = st.H;
  int id = lo;
  while (id < hi) {
    const TileIter ti(st.tile1_start, st.batch, H, st.nt1, id, hi);
    const int per_head = (st.tile1_start[ti.b + 1] - st.tile1_start[ti.b]) / H;
    const int L = st.cu[ti.b + 1] - st.cu[ti.b];
    const int unit = ti.unit();
    const SegList sl(ti.layer * st.nt1 + st.tile1_start[ti.b] + ti.h * per_head, per_head,
                     split1(st));
    if (tid == 0) *flag = arrive_last(ws.headcnt + unit, call_tag, sl.nseg);
    __syncthreads();
    const bool last = *flag != 0;
    if (last) {
      if (tid < NQ)
        ws.bq[(size_t)unit * NQ + tid] =
            fold_row_stats<MB == 1 ? 2 : 1>(ws.rowstat, sl, NQ, tid) - log2f((float)st.W);
      const int kt = tid - 256;
      float sum = 0.f;
      if (kt >= 0 && kt < kHeadDim) {
        sum = fold_key_sums(ws.ksum, sl, kt);
        ws.kbar[(size_t)unit * kHeadDim + kt] = sum / (float)L;
        const float n2 = warp_sum(sum * sum);
        if (lane == 0) red[kt >> 5] = n2;
      }
    }
    __syncthreads();   // `flag` may be rewritten; the four partial norms are in `red`
    if (last && tid == 256) {
      const double nn = ((double)red[0] + (double)red[1]) + ((double)red[2] + (double)red[3]);
      const double T = (double)L;
      const float r = (float)((nn - T) / (T * (T - 1.0)));   // Eq. 4
      ws.rbar[unit] = r;
      if (rbar_out) rbar_out[unit] = r;
    }
    __syncthreads();   // `red` is free again
    id += min(hi - id, per_head - ti.t);
  }
}

// One 32-column chunk of a logit row: running (max, sum) of the softmax in log2 units.
__device__ __forceinline__ void softmax_chunk(uint32_t (&r)[32], const bool need_mask,
                                              const int kbase, const int lim,
                                              const float scale_log2e, float& m_run,
                                              float& z_run) {
  if (need_mask) {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (kbase + j > lim) r[j] = 0xff800000u;   // -inf
  }
  float mx = max3(__uint_as_float(r[0]), __uint_as_float(r[1]), __uint_as_float(r[2]));
#pragma unroll
  for (int j = 3; j < 31; j += 2)
    mx = max3(mx, __uint_as_float(r[j]), __uint_as_float(r[j + 1]));
  mx = fmaxf(mx, __uint_as_float(r[31]));
  const float mn = fmaxf(m_run, mx * scale_log2e);
  if (mn > m_run) {
    z_run *= ex2(m_run - mn);
    m_run = mn;
  }
  const f32x2 sc2 = pack2(scale_log2e, scale_log2e), nm2 = pack2(-m_run, -m_run);
  f32x2 za = pack2(0.f, 0.f), zb = za;
#pragma unroll
  for (int j = 0; j < 32; j += 4) {
    float a0, a1, b0, b1;
    unpack2(fma2(pack2(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), sc2, nm2), a0, a1);
    unpack2(fma2(pack2(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3])), sc2, nm2), b0, b1);
    za = add2(za, pack2(ex2(a0), ex2(a1)));
    zb = add2(zb, pack2(ex2(b0), ex2(b1)));
  }
  float z0, z1;
  unpack2(add2(za, zb), z0, z1);
  z_run += z0 + z1;
}

// grid = g1 persistent CTAs: TMA, MMA, 2 idle, 8 epilogue, 4 or 8 key-statistics warps.
template <int MB>
__global__ void __launch_bounds__(p1_threads(MB), 1)
k_pass1(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
        const SeqTable st, const Workspace ws, const float scale_log2e,
        const unsigned long long call_tag, float* __restrict__ rbar_out, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* base =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  constexpr int QR = MB * 128;                 // query rows the MMA reads
  constexpr int kP1Stages = p1_stages(MB);
  constexpr int kP1AuxWarps = p1_aux_warps(MB);
  constexpr int kP1Threads = p1_threads(MB);
  unsigned char* sQ = base;                    // 2 halves x [QR x 128 B]
  unsigned char* sK = sQ + 2 * QR * 128;       // kP1Stages x 32 KB
  float* sks = reinterpret_cast<float*>(sK + kP1Stages * kTileBytes);  // [aux warps][128] key-sum exchange
  P1Bars* bars = reinterpret_cast<P1Bars*>(sks + kP1AuxWarps * 128);
  {
    // the carve-up above must fit behind the (1 KB aligned) base
    unsigned dyn;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    if ((size_t)(reinterpret_cast<unsigned char*>(bars + 1) - smem_dyn) > dyn) {
      if (threadIdx.x == 0 && status) atomicExch(status, MIXKV_ERR_CUDA);
      return;
    }
  }

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int NQ = st.NQ, W = st.W, H = st.H;
  const int lo = cta_first_tile(blockIdx.x, split1(st));
  const int hi = cta_first_tile(blockIdx.x + 1, split1(st));
  volatile int* abort = &bars->abort;

  pdl_launch_dependents();
  if (tid == 0) {
    for (int s = 0; s < kP1Stages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1 + kP1AuxWarps);   // MMA commit + the key-statistics warps
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->tfull[s], 1);
      mbar_init(&bars->tempty[s], kEpiThreads);
    }
    mbar_init(&bars->qfull, 1);
    mbar_init(&bars->qfree, 1);
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
  if (warp == kWarpTma && lane == 0) {
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmQ);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  pdl_wait();   // everything earlier in the stream is complete: global memory may be touched

  if (warp == kWarpTma) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int it = 0, segn = 0;
      bool seg_start = true;
      for (TileIter ti(st.tile1_start, st.batch, H, st.nt1, lo, hi); ti.valid(); ti.next()) {
        if (seg_start) {
          if (segn > 0 && !mbar_wait(&bars->qfree, (segn - 1) & 1, abort)) break;
          mbar_expect_tx(&bars->qfull, NQ * 256);
          tma_load_3d(sQ, &tmQ, 0, ti.bh() * NQ, ti.layer, &bars->qfull);
          tma_load_3d(sQ + QR * 128, &tmQ, 64, ti.bh() * NQ, ti.layer, &bars->qfull);
          ++segn;
        }
        seg_start = ti.seg_last();
        const int s = it % kP1Stages, ph = (it / kP1Stages) & 1;
        if (!mbar_wait(&bars->empty[s], ph ^ 1, abort)) break;
        mbar_expect_tx(&bars->full[s], kTileBytes);
        const int y = st.cu[ti.b] + ti.t * kTile;
        tma_load_4d(sK + s * kTileBytes, &tmK, 0, y, ti.h, ti.layer, &bars->full[s]);
        tma_load_4d(sK + s * kTileBytes + kHalfBytes, &tmK, 64, y, ti.h, ti.layer, &bars->full[s]);
        ++it;
      }
      if (*abort) {
        raise(status, abort);
        drain_ring(bars->full, kP1Stages, it);
      }
    }
  } else if (warp == kWarpMma) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(128, kTile);
      int it = 0, segn = 0;
      bool seg_start = true;
      for (TileIter ti(st.tile1_start, st.batch, H, st.nt1, lo, hi); ti.valid(); ti.next()) {
        if (seg_start) {
          if (!mbar_wait(&bars->qfull, segn & 1, abort)) break;
          ++segn;
        }
        seg_start = ti.seg_last();
        const int s = it % kP1Stages, ph = (it / kP1Stages) & 1, ts = it & 1, tph = (it >> 1) & 1;
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
        if (seg_start) umma_commit(&bars->qfree);
        ++it;
      }
      if (*abort) raise(status, abort);
    }
  } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kEpiWarps) {
    // ------------------------------------------------------------------ epilogue
    // MB == 2: warpgroup wg owns query rows wg*128 .. +127 and all 128 keys of the tile.
    // MB == 1: both warpgroups own rows 0 .. 127; wg takes the keys wg*64 .. +63.
    const int quarter = warp & 3, wg = (warp - kEpiWarp0) >> 2;
    const int row = (MB == 2 ? wg * 128 : 0) + quarter * 32 + lane;
    const int unit = MB == 2 ? 0 : wg;
    constexpr int NC = MB == 2 ? 128 : 64;       // columns (keys) this thread reduces per tile
    const int col0 = MB == 2 ? wg * 128 : wg * 64;
    const bool warp_on = (MB == 2 ? wg * 128 : 0) + quarter * 32 < NQ;
    const int jrow = row % W;
    float m_run = -1e30f, z_run = 0.f;
    int it = 0, seg_first = lo;
    bool seg_start = true;
    for (TileIter ti(st.tile1_start, st.batch, H, st.nt1, lo, hi); ti.valid(); ti.next()) {
      if (seg_start) {
        m_run = -1e30f;
        z_run = 0.f;
        seg_first = ti.id;
      }
      seg_start = ti.seg_last();
      const int L = st.cu[ti.b + 1] - st.cu[ti.b], P = L - W;
      const int ts = it & 1, tph = (it >> 1) & 1;
      if (!mbar_wait(&bars->tfull[ts], tph, abort)) break;
      tc_fence_after();
      if (warp_on) {
        const int k0 = ti.t * kTile + (MB == 2 ? 0 : wg * 64);
        const bool need_mask = ti.t * kTile + kTile > P;
        const int lim = P + jrow;   // last key this row may see
        const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + ts * (MB * 128) + col0;
#pragma unroll 1
        for (int c0 = 0; c0 < NC; c0 += 32) {   // kept rolled: the body must stay in the i-cache
          uint32_t ra[32];
          tmem_ld32(taddr + c0, ra);
          tmem_ld_wait();
          tmem_ld_fence(ra);
          softmax_chunk(ra, need_mask, k0 + c0, lim, scale_log2e, m_run, z_run);
        }
      }
      tc_fence_before();
      mbar_arrive(&bars->tempty[ts]);
      if (seg_start && row < NQ)
        ws.rowstat[((size_t)seg_first * 2 + unit) * NQ + row] = make_float2(m_run, z_run);
      ++it;
    }
  } else if (warp >= kAuxWarp0) {
    // ------------------------------------------------------------------ key statistics
    // Sixteen lanes share a key row (one 16-byte chunk each); a pair of 8-row batches is one
    // warp-wide step (one batch per 16-lane group).  Sweep 1 squares, a butterfly leaves the
    // squared norm of row r with lanes 2r and 2r+1, sweep 2 adds the rows scaled by 1/|k| into
    // eight per-thread sums (dims 8c .. 8c+7).
    const int aux_w = warp - kAuxWarp0;
    constexpr int kPairs = 8 / kP1AuxWarps;      // pairs of 8-row batches per warp and tile
    const int c = lane & 15, lg = lane >> 4;
    const int chalf = c >> 3, cc = c & 7;
    constexpr int aux_threads = kP1AuxWarps * 32;
    const int kt = tid - kAuxWarp0 * 32;
    f32x2 acc2[4];   // dims 8c .. 8c+7 as four packed pairs
#pragma unroll
    for (int e = 0; e < 4; ++e) acc2[e] = pack2(0.f, 0.f);
    int it = 0, seg_first = lo;
    bool seg_start = true;
    for (TileIter ti(st.tile1_start, st.batch, H, st.nt1, lo, hi); ti.valid(); ti.next()) {
      if (seg_start) {
#pragma unroll
        for (int e = 0; e < 4; ++e) acc2[e] = pack2(0.f, 0.f);
        seg_first = ti.id;
      }
      seg_start = ti.seg_last();
      const int L = st.cu[ti.b + 1] - st.cu[ti.b];
      const int s = it % kP1Stages, ph = (it / kP1Stages) & 1;
      const bool ok = mbar_wait(&bars->full[s], ph, abort);
      const unsigned char* tile = sK + s * kTileBytes + chalf * kHalfBytes;
#pragma unroll 1
      for (int bp = 0; bp < kPairs; ++bp) {   // kept rolled: the body must stay in the i-cache
        const int row0 = (2 * (aux_w * kPairs + bp) + lg) * 8;
        uint4 u[8];
        float p[8];
#pragma unroll
        for (int rr = 0; rr < 8; ++rr) {
          u[rr] = *reinterpret_cast<const uint4*>(tile + sw128_offset(row0 + rr, cc));
          const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&u[rr]);
          f32x2 sq = pack2(0.f, 0.f);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(p2[e]);
            const f32x2 f2 = pack2(f.x, f.y);
            sq = fma2(f2, f2, sq);
          }
          float s0, s1;
          unpack2(sq, s0, s1);
          p[rr] = s0 + s1;
        }
        if (bp == kPairs - 1) {   // the tile now lives in registers: hand the stage back
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars->empty[s]);
        }
#pragma unroll
        for (int o = 8; o >= 2; o >>= 1) {
          const bool up = (c & o) != 0;
#pragma unroll
          for (int k = 0; k < o / 2; ++k) {
            const float send = up ? p[k] : p[k + o / 2];
            const float keep = up ? p[k + o / 2] : p[k];
            p[k] = keep + __shfl_xor_sync(0xffffffffu, send, o);
          }
        }
        p[0] += __shfl_xor_sync(0xffffffffu, p[0], 1);
        const int i = ti.t * kTile + row0 + (c >> 1);
        const float inv = (ok && i < L && p[0] > 0.f) ? rsqrtf(p[0]) : 0.f;
        if (i < L && (c & 1) == 0) ws.kinv[kpos(st, ti.layer, ti.h, ti.b, i)] = inv;
#pragma unroll
        for (int rr = 0; rr < 8; ++rr) {
          const float w = __shfl_sync(0xffffffffu, inv, (lane & 16) | (rr << 1));
          const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&u[rr]);
          const f32x2 w2 = pack2(w, w);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(p2[e]);
            acc2[e] = fma2(pack2(f.x, f.y), w2, acc2[e]);
          }
        }
      }
      if (group_sync_stop(2, aux_threads, kt == 0, abort, bars->vote, it)) break;
      if (seg_start) {
        float acc[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) unpack2(acc2[e], acc[2 * e], acc[2 * e + 1]);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float v = acc[e] + __shfl_xor_sync(0xffffffffu, acc[e], 16);
          if (lane < 16) sks[aux_w * 128 + c * 8 + e] = v;
        }
        named_bar_sync(2, aux_threads);
        if (kt < kHeadDim) {
          float t = 0.f;
#pragma unroll
          for (int w = 0; w < kP1AuxWarps; ++w) t += sks[w * 128 + kt];
          ws.ksum[(size_t)seg_first * kHeadDim + kt] = t;
        }
        named_bar_sync(2, aux_threads);
      }
      ++it;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kWarpMma) tmem_dealloc(tmem, MB * 256);
  if (bars->abort) {
    if (tid == 0 && status) atomicExch(status, MIXKV_ERR_TIMEOUT);
    return;
  }
  // Every partial result of this CTA is written.  Its segments now count as delivered; the CTA
  // that delivers the last segment of a (layer, sequence, head) folds all of them, once, into
  // what pass 2 reads: one log2 normaliser per window row (the 1/W of the window mean folded
  // in), the mean unit key, the redundancy of Eq. 4.
  finish_heads<MB>(st, ws, lo, hi, call_tag, rbar_out, sks, &bars->last);
}

// ======================================================================== pass 2
constexpr int kP2KStages = 3;              // K tiles (32 KB each)
constexpr int kP2VStagesMax = 4;           // V half tiles: 64 rows, 16 KB each
constexpr int kVSubBytes = 64 * 256;
struct P2Bars {
  uint64_t kfull[kP2KStages];
  uint64_t kempty[kP2KStages];
  uint64_t vfull[kP2VStagesMax];
  uint64_t vempty[kP2VStagesMax];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint64_t qfull;
  uint64_t qfree;
  uint64_t kbready;
  uint32_t tmem_base;
  int abort;
  int vote[3][2];
};

// N logit columns of one key (registers r[0..N)): adds exp2(logit * scale - normaliser of the
// column) to acc; nb_smem holds the negated normalisers of these columns.
template <int N>
__device__ __forceinline__ void colsum_chunk(const uint32_t (&r)[N], const float* nb_smem,
                                             const f32x2 sc2, f32x2& acc) {
#pragma unroll
  for (int j = 0; j < N; j += 4) {
    const float4 nb = *reinterpret_cast<const float4*>(nb_smem + j);   // negated normalisers
    float a0, a1, b0, b1;
    unpack2(fma2(pack2(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), sc2, pack2(nb.x, nb.y)),
            a0, a1);
    unpack2(fma2(pack2(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3])), sc2,
                 pack2(nb.z, nb.w)),
            b0, b1);
    acc = add2(acc, pack2(ex2(a0), ex2(a1)));
    acc = add2(acc, pack2(ex2(b0), ex2(b1)));
  }
}

// grid = g2 persistent CTAs: K producer, MMA, V producer, 1 idle, 8 epilogue, 4 value-norm warps.
__global__ void __launch_bounds__(kThreads, 1)
k_pass2(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
        const __grid_constant__ CUtensorMap tmQ, const SeqTable st, const Workspace ws,
        float* __restrict__ s_div_out, const float scale_log2e,
        const int use_vnorm, const int pool_half, const int vstages, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* base =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  const int NQ = st.NQ, W = st.W, H = st.H;
  const int NB = NQ + kExtraRows;             // rows of the B operand
  unsigned char* sQ = base;                   // 2 halves x [NB x 128 B]
  unsigned char* sK = sQ + 2 * NB * 128;      // kP2KStages x 32 KB
  unsigned char* sV = sK + kP2KStages * kTileBytes;   // vstages x 16 KB
  float* sbq = reinterpret_cast<float*>(sV + vstages * kVSubBytes);  // [2][256] negated normalisers
  float* sred = sbq + 512;                    // [64]: 2 x 16 epilogue, 16 value norms + 4 mean key
  P2Bars* bars = reinterpret_cast<P2Bars*>(sred + 64);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int lo = cta_first_tile(blockIdx.x, split2(st));
  const int hi = cta_first_tile(blockIdx.x + 1, split2(st));
  volatile int* abort = &bars->abort;
  constexpr int kWarpTmaV = 2;

  pdl_launch_dependents();
  if (tid == 0) {
    for (int s = 0; s < kP2KStages; ++s) {
      mbar_init(&bars->kfull[s], 1);
      mbar_init(&bars->kempty[s], 1);
    }
    for (int s = 0; s < kP2VStagesMax; ++s) {
      mbar_init(&bars->vfull[s], 1);
      mbar_init(&bars->vempty[s], 2);      // the two warps that read a half tile
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->tfull[s], 1);
      mbar_init(&bars->tempty[s], 128);    // the warpgroup that owns the accumulator stage
    }
    mbar_init(&bars->qfull, 1);
    mbar_init(&bars->qfree, 1);
    mbar_init(&bars->kbready, 4);          // the four warps that write the mean-key rows
    bars->abort = 0;
    mbar_init_fence();
  }
  if (warp == kWarpMma) tmem_alloc(&bars->tmem_base, 512);
  if (warp == kWarpTma && lane == 0) {
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmQ);
  }
  if (warp == kWarpTmaV && lane == 0) tma_prefetch_desc(&tmV);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  pdl_wait();

  if (warp == kWarpTma) {
    // ------------------------------------------------------------------ K / Q producer
    if (lane == 0) {
      int it = 0, segn = 0;
      bool seg_start = true;
      for (TileIter ti(st.tile2_start, st.batch, H, st.nt2, lo, hi); ti.valid(); ti.next()) {
        if (seg_start) {
          if (segn > 0 && !mbar_wait(&bars->qfree, (segn - 1) & 1, abort)) break;
          mbar_expect_tx(&bars->qfull, NQ * 256);
          tma_load_3d(sQ, &tmQ, 0, ti.bh() * NQ, ti.layer, &bars->qfull);
          tma_load_3d(sQ + NB * 128, &tmQ, 64, ti.bh() * NQ, ti.layer, &bars->qfull);
          ++segn;
        }
        seg_start = ti.seg_last();
        const int s = it % kP2KStages, ph = (it / kP2KStages) & 1;
        if (!mbar_wait(&bars->kempty[s], ph ^ 1, abort)) break;
        mbar_expect_tx(&bars->kfull[s], kTileBytes);
        const int y = st.cu[ti.b] + ti.t * kTile;
        tma_load_4d(sK + s * kTileBytes, &tmK, 0, y, ti.h, ti.layer, &bars->kfull[s]);
        tma_load_4d(sK + s * kTileBytes + kHalfBytes, &tmK, 64, y, ti.h, ti.layer, &bars->kfull[s]);
        ++it;
      }
      if (*abort) {
        raise(status, abort);
        drain_ring(bars->kfull, kP2KStages, it);
      }
    }
  } else if (warp == kWarpTmaV) {
    // ------------------------------------------------------------------ V producer
    if (lane == 0 && use_vnorm == MIXKV_INTRINSIC_VNORM) {
      int vit = 0;
      bool ok = true;
      for (TileIter ti(st.tile2_start, st.batch, H, st.nt2, lo, hi); ti.valid() && ok; ti.next()) {
        const int y = st.cu[ti.b] + ti.t * kTile;
        for (int sub = 0; sub < 2; ++sub) {
          const int vs = vit % vstages, vph = (vit / vstages) & 1;
          if (!mbar_wait(&bars->vempty[vs], vph ^ 1, abort)) {
            ok = false;
            break;
          }
          mbar_expect_tx(&bars->vfull[vs], kVSubBytes);
          unsigned char* dst = sV + vs * kVSubBytes;
          tma_load_4d(dst, &tmV, 0, y + sub * 64, ti.h, ti.layer, &bars->vfull[vs]);
          tma_load_4d(dst + kVSubBytes / 2, &tmV, 64, y + sub * 64, ti.h, ti.layer, &bars->vfull[vs]);
          ++vit;
        }
      }
      if (*abort) {
        raise(status, abort);
        drain_ring(bars->vfull, vstages, vit);
      }
    }
  } else if (warp == kWarpMma) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(128, NB);
      int it = 0, segn = 0;
      bool seg_start = true;
      for (TileIter ti(st.tile2_start, st.batch, H, st.nt2, lo, hi); ti.valid(); ti.next()) {
        if (seg_start) {
          if (!mbar_wait(&bars->qfull, segn & 1, abort)) break;
          if (!mbar_wait(&bars->kbready, segn & 1, abort)) break;
          ++segn;
        }
        seg_start = ti.seg_last();
        const int s = it % kP2KStages, ph = (it / kP2KStages) & 1, ts = it & 1, tph = (it >> 1) & 1;
        if (!mbar_wait(&bars->kfull[s], ph, abort)) break;
        if (!mbar_wait(&bars->tempty[ts], tph ^ 1, abort)) break;
        tc_fence_after();
        const uint32_t kaddr = smem_u32(sK + s * kTileBytes);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t da = umma_desc_sw128(kaddr + (ks >> 2) * kHalfBytes + (ks & 3) * 32);
          const uint64_t db = umma_desc_sw128(smem_u32(sQ) + (ks >> 2) * NB * 128 + (ks & 3) * 32);
          umma_bf16(tmem + ts * 256, da, db, idesc, ks > 0);
        }
        umma_commit(&bars->kempty[s]);
        umma_commit(&bars->tfull[ts]);
        if (seg_start) umma_commit(&bars->qfree);
        ++it;
      }
      if (*abort) raise(status, abort);
    }
  } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kEpiWarps) {
    // ------------------------------------------------------------------ epilogue
    // The two warpgroups take alternate tiles (warpgroup g owns accumulator stage g), one key
    // per thread and all G*W columns of it, so a tile needs no exchange between warpgroups and
    // the groups never wait for each other: each keeps its own copy of the normaliser table
    // and leaves its own partial score statistics.
    const int quarter = warp & 3, wg = (warp - kEpiWarp0) >> 2;
    const int gt = (tid - kEpiWarp0 * 32) & 127;   // thread inside the warpgroup
    const int gw = gt >> 5;                        // warp inside the warpgroup
    const int key = quarter * 32 + lane;
    const int nch = NQ / 16;
    float* mybq = sbq + wg * 256;
    const int barid = 1 + wg;                      // named barriers 1, 2: one per warpgroup
    const f32x2 sc2 = pack2(scale_log2e, scale_log2e);
    float dmin = INFINITY, dmax = -INFINITY, dsum = 0.f, exw = 0.f;
    int it = 0, seg_first = lo;
    bool seg_start = true;
    for (TileIter ti(st.tile2_start, st.batch, H, st.nt2, lo, hi); ti.valid(); ti.next()) {
      const int L = st.cu[ti.b + 1] - st.cu[ti.b], P = L - W;
      if (seg_start) {
        // pass 1 left one negated log2 normaliser per window row of this (layer, b, h)
        named_bar_sync(barid, 128);   // the previous segment's readers of mybq are done
        for (int q = gt; q < NQ; q += 128) mybq[q] = ws.bq[(size_t)ti.unit() * NQ + q];
        dmin = INFINITY, dmax = -INFINITY, dsum = 0.f, exw = 0.f;
        seg_first = ti.id;
        named_bar_sync(barid, 128);
      }
      seg_start = ti.seg_last();
      const int ts = it & 1;
      if (ts == wg) {   // this warpgroup's tile
        const int tph = (it >> 1) & 1;
        const int ikey = ti.t * kTile + key;
        float kinv_i = 0.f;
        if (ikey < P) kinv_i = ws.kinv[kpos(st, ti.layer, ti.h, ti.b, ikey)];
        const bool ok = mbar_wait(&bars->tfull[ts], tph, abort);
        tc_fence_after();
        const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + ts * 256;
        f32x2 acc = pack2(0.f, 0.f);
        float dot = 0.f;
        if (ok) {
          uint32_t rd[4];
          tmem_ld4(taddr + NQ, rd);
          // 32-column chunks (the other warpgroup's tile keeps the SM busy while this load is
          // in flight), then a 16-column rest; kept rolled: the body must stay in the i-cache
          const int n32 = nch >> 1;
#pragma unroll 1
          for (int ci = 0; ci < n32; ++ci) {
            uint32_t ra[32];
            tmem_ld32(taddr + ci * 32, ra);
            tmem_ld_wait();
            tmem_ld_fence(ra);
            colsum_chunk<32>(ra, mybq + ci * 32, sc2, acc);
          }
          if (nch & 1) {
            uint32_t rb[16];
            tmem_ld16(taddr + n32 * 32, rb);
            tmem_ld_wait();
            tmem_ld_fence(rb);
            colsum_chunk<16>(rb, mybq + n32 * 32, sc2, acc);
          }
          tmem_ld_wait();
          tmem_ld_fence(rd);
          dot = (__uint_as_float(rd[0]) + __uint_as_float(rd[1])) + __uint_as_float(rd[2]);
        }
        tc_fence_before();
        mbar_arrive(&bars->tempty[ts]);
        if (ok && ikey < P) {
          float acc0, acc1;
          unpack2(acc, acc0, acc1);
          const size_t poff = ppos(st, ti.layer, ti.h, ti.b, 0);
          const float ex = acc0 + acc1;
          ws.s_ex_raw[poff + ikey] = ex;
          const float sd = -dot * kinv_i;
          s_div_out[poff + ikey] = sd;
          dmin = fminf(dmin, sd);
          dmax = fmaxf(dmax, sd);
          dsum += sd;
          // number of pooling windows (centres in [0, P)) that cover this position
          const int cover = min(ikey, pool_half) + min(P - 1 - ikey, pool_half) + 1;
          exw = fmaf(ex, (float)cover, exw);
        }
      }
      if (group_sync_stop(barid, 128, gt == 0, abort, bars->vote[wg], it)) break;
      if (seg_start) {
        // this warpgroup's share of the segment's score statistics (neutral if it had no tile)
        const float a = warp_min(dmin), b2 = warp_max(dmax), c2 = warp_sum(dsum),
                    d2 = warp_sum(exw);
        float* sr = sred + wg * 16;
        if (lane == 0) {
          sr[gw] = a;
          sr[4 + gw] = b2;
          sr[8 + gw] = c2;
          sr[12 + gw] = d2;
        }
        named_bar_sync(barid, 128);
        if (gt == 0) {
          ws.dstat[(size_t)seg_first * 2 + wg] = make_float4(
              fminf(fminf(sr[0], sr[1]), fminf(sr[2], sr[3])),
              fmaxf(fmaxf(sr[4], sr[5]), fmaxf(sr[6], sr[7])),
              (sr[8] + sr[9]) + (sr[10] + sr[11]), (sr[12] + sr[13]) + (sr[14] + sr[15]));
        }
      }
      ++it;
    }
  } else if (warp >= kAuxWarp0) {
    // ------------------------------------------------------------------ mean key, value norms
    // At the start of a segment: write the bf16 hi / lo / lo2 split of the head's mean unit key
    // (pass 1) into the three extra B rows.  Per tile: warps 12, 13 read the first 64 rows of the V
    // tile, warps 14, 15 the last 64; one row per thread from the swizzled half tile.
    const int vt = tid - kAuxWarp0 * 32;         // 0..127
    const int sub = vt >> 6, vr = vt & 63;
    float vmin = INFINITY, vmax = -INFINITY, vsum = 0.f;
    int it = 0, segn = 0, seg_first = lo;
    bool seg_start = true;
    for (TileIter ti(st.tile2_start, st.batch, H, st.nt2, lo, hi); ti.valid(); ti.next()) {
      if (seg_start) {
        const float kb = ws.kbar[(size_t)ti.unit() * kHeadDim + vt];   // mean unit key (pass 1)
        __nv_bfloat16 parts[3];
        parts[0] = __float2bfloat16_rn(kb);
        const float r1 = kb - __bfloat162float(parts[0]);
        parts[1] = __float2bfloat16_rn(r1);
        parts[2] = __float2bfloat16_rn(r1 - __bfloat162float(parts[1]));
        if (segn > 0) {   // the previous segment's MMAs must be done with the B rows
          if (vt == 0) mbar_wait(&bars->qfree, (segn - 1) & 1, abort);
          named_bar_sync(4, 128);
        }
        {
          unsigned char* hb = sQ + (vt >> 6) * NB * 128 + (vt & 7) * 2;
          const int chunk = (vt & 63) >> 3;
#pragma unroll
          for (int e = 0; e < kExtraRows; ++e) {
            if (e < 3 || segn == 0)
              *reinterpret_cast<__nv_bfloat16*>(hb + sw128_offset(NQ + e, chunk)) =
                  e < 3 ? parts[e] : __float2bfloat16_rn(0.f);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->kbready);
        ++segn;
        vmin = INFINITY, vmax = -INFINITY, vsum = 0.f;
        seg_first = ti.id;
      }
      seg_start = ti.seg_last();
      if (use_vnorm == MIXKV_INTRINSIC_KNORM) {
        // key-norm ablation: the intrinsic term is minus the key norm, which pass 1 left as its
        // reciprocal; no V tile is loaded
        const int P = st.cu[ti.b + 1] - st.cu[ti.b] - W;
        const int i = ti.t * kTile + vt;
        if (i < P) {
          const float ki = ws.kinv[kpos(st, ti.layer, ti.h, ti.b, i)];
          const float n = ki > 0.f ? -1.0f / ki : 0.f;
          ws.vnorm[ppos(st, ti.layer, ti.h, ti.b, i)] = n;
          vmin = fminf(vmin, n);
          vmax = fmaxf(vmax, n);
          vsum += n;
        }
      } else if (use_vnorm) {
        const int P = st.cu[ti.b + 1] - st.cu[ti.b] - W;
        const int vit = 2 * it + sub;
        const int vs = vit % vstages, vph = (vit / vstages) & 1;
        const bool ok = mbar_wait(&bars->vfull[vs], vph, abort);
        const unsigned char* tile = sV + vs * kVSubBytes;
        f32x2 ss2[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
        if (ok) {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const uint4 u =
                  *reinterpret_cast<const uint4*>(tile + half * (kVSubBytes / 2) + sw128_offset(vr, c));
              const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float2 f = __bfloat1622float2(p2[e]);
                const f32x2 f2 = pack2(f.x, f.y);
                ss2[e & 1] = fma2(f2, f2, ss2[e & 1]);
              }
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->vempty[vs]);
        const int i = ti.t * kTile + sub * 64 + vr;
        if (ok && i < P) {
          float ss[4];
          unpack2(ss2[0], ss[0], ss[2]);
          unpack2(ss2[1], ss[1], ss[3]);
          const float n = sqrtf((ss[0] + ss[1]) + (ss[2] + ss[3]));
          ws.vnorm[ppos(st, ti.layer, ti.h, ti.b, i)] = n;
          vmin = fminf(vmin, n);
          vmax = fmaxf(vmax, n);
          vsum += n;
        }
      }
      if (group_sync_stop(3, 128, vt == 0, abort, bars->vote[2], it)) break;
      if (seg_start && use_vnorm) {
        const float a = warp_min(vmin), b2 = warp_max(vmax), c2 = warp_sum(vsum);
        const int vw = warp - kAuxWarp0;
        if (lane == 0) {
          sred[32 + vw] = a;
          sred[36 + vw] = b2;
          sred[40 + vw] = c2;
        }
        named_bar_sync(4, 128);
        if (vt == 0) {
          ws.vstat[seg_first] = make_float4(
              fminf(fminf(sred[32], sred[33]), fminf(sred[34], sred[35])),
              fmaxf(fmaxf(sred[36], sred[37]), fmaxf(sred[38], sred[39])),
              (sred[40] + sred[41]) + (sred[42] + sred[43]), 0.f);
        }
        named_bar_sync(4, 128);
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

// X [layers, H, Ltot, d] bf16 (layer stride given in elements) as a 4-D tensor (d, Ltot, H,
// layers) with boxes of 64 x rows x 1 x 1.  Rows past the end of the tensor read as zero.
bool map_kv(const LaunchCtx& c, const void* X, int box_rows, CUtensorMap* tm) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)c.st.Ltot, (cuuint64_t)c.st.H,
                        (cuuint64_t)c.st.layers};
  cuuint64_t strides[3] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)c.st.Ltot * kHeadDim * 2,
                           (cuuint64_t)c.kv_layer_stride * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t es[4] = {1, 1, 1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(X), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Q [layers, batch * H * NQ, d] bf16 as a 3-D tensor (d, rows, layers) with boxes of 64 x NQ x 1.
bool map_q(const LaunchCtx& c, const void* Q, CUtensorMap* tm) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)c.st.batch * c.st.H * c.st.NQ,
                        (cuuint64_t)c.st.layers};
  cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)c.q_layer_stride * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)c.st.NQ, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(Q), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t pass1_smem(int MB) {
  // up to 1023 bytes of alignment slack in front of the carve-up; never beyond the limit (the
  // kernel checks that its carve-up fits behind the aligned base)
  const size_t need = (size_t)2 * MB * 128 * 128 + (size_t)p1_stages(MB) * kTileBytes + p1_aux_warps(MB) * 128 * 4 +
                      sizeof(P1Bars);
  const size_t want = need + 1024;
  return want < kSmemLimit ? want : kSmemLimit;
}
size_t pass2_smem(int NQ, int vstages) {
  return 1024 + (size_t)2 * (NQ + kExtraRows) * 128 + kP2KStages * kTileBytes +
         (size_t)vstages * kVSubBytes + 512 * 4 + 64 * 4 + sizeof(P2Bars) + 64;
}

// cudaFuncSetAttribute once per (kernel, device).
template <typename F>
cudaError_t ensure_smem(F kernel, size_t smem, bool (&done)[64]) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !done[dev]) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) done[dev] = true;
  }
  return cudaSuccess;
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

cudaError_t launch_pass1(const LaunchCtx& c, const void* K, const void* Q, float* rbar_out,
                         int* status) {
  CUtensorMap tmK, tmQ;
  if (!map_kv(c, K, kTile, &tmK) || !map_q(c, Q, &tmQ)) return cudaErrorInvalidValue;
  static bool done1[64] = {false}, done2[64] = {false};
  if (c.st.NQ <= 128) {
    const size_t smem = pass1_smem(1);
    cudaError_t e = ensure_smem(k_pass1<1>, smem, done1);
    if (e != cudaSuccess) return e;
    return launch_pdl(k_pass1<1>, dim3(c.st.g1), dim3(p1_threads(1)), smem, c.stream, 1, tmK, tmQ, c.st,
                      c.ws, c.scale_log2e, c.call_tag, rbar_out, status);
  }
  const size_t smem = pass1_smem(2);
  cudaError_t e = ensure_smem(k_pass1<2>, smem, done2);
  if (e != cudaSuccess) return e;
  return launch_pdl(k_pass1<2>, dim3(c.st.g1), dim3(p1_threads(2)), smem, c.stream, 1, tmK, tmQ, c.st,
                    c.ws, c.scale_log2e, c.call_tag, rbar_out, status);
}

cudaError_t launch_pass2(const LaunchCtx& c, const void* K, const void* V, const void* Q,
                         float* s_div_out, int* status) {
  CUtensorMap tmK, tmV, tmQ;
  const void* Vsrc = c.p.use_vnorm == MIXKV_INTRINSIC_VNORM ? V : K;   // the V map is never used without VNorm
  if (!map_kv(c, K, kTile, &tmK) || !map_kv(c, Vsrc, 64, &tmV) || !map_q(c, Q, &tmQ))
    return cudaErrorInvalidValue;
  static bool done[64] = {false};
  cudaError_t e = ensure_smem(k_pass2, kSmemLimit, done);
  if (e != cudaSuccess) return e;
  int vstages = kP2VStagesMax;
  while (vstages > 2 && pass2_smem(c.st.NQ, vstages) > kSmemLimit) --vstages;
  const size_t smem = pass2_smem(c.st.NQ, vstages);
  return launch_pdl(k_pass2, dim3(c.st.g2), dim3(kThreads), smem, c.stream, 1, tmK, tmV, tmQ, c.st,
                    c.ws, s_div_out, c.scale_log2e, c.p.use_vnorm, c.p.pool_kernel >> 1,
                    vstages, status);
}

}  // namespace mixkv
