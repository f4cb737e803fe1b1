// The two passes over K of the MixKV scoring step as persistent, warp-specialised sm_100a
// kernels: TMA tile loads into 128-byte-swizzled shared memory, tcgen05.mma (bf16 x bf16 ->
// fp32) with accumulators in tensor memory, and epilogues that read the accumulators back with
// tcgen05.ld.
//
//   pass 1  K from HBM.  Logits with the window queries on the M side (one query row per TMEM
//           lane), so the running softmax (max, sum) of a row is thread-local; alongside, key
//           norms and the sum of unit keys from the shared-memory tile.  Every run of tiles
//           of one (layer, sequence, head) inside a CTA (a segment) leaves its partial
//           statistics.
//   pass 2  K again, V from HBM.  A CTA that starts on a (layer, sequence, head) first folds
//           that head's segments of pass 1: the softmax statistics become one log2 normaliser
//           per window row, the unit-key sums the mean unit key and the redundancy of Eq. 4
//           (every CTA that touches the head does this for itself: no CTA waits for another,
//           nothing is counted).  Logits with the keys on the M side (one key per TMEM lane),
//           normalised with those row statistics, so the column sum over window rows
//           and query heads is thread-local -> s_ex_raw.  The mean unit key rides
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

// Warp roles.  Warpgroup 0 (warps 0..3) holds the single-thread roles: TMA producer, MMA
// issuer, (pass 2) V producer.  Pass 1: warps 4..19 are the epilogue (all sixteen work on every
// tile), warps 20..27 compute the key statistics; register budgets per role are set with
// setmaxnreg (the single-thread roles hand most of theirs to the others).  Pass 2: warps 4..11
// are the epilogue (two warpgroups that own alternate tiles), warps 12..15 the value norms.  A
// warp's TMEM lane quarter is warp % 4.
constexpr int kWarpTma = 0, kWarpMma = 1;
constexpr int kP1WarpMma = 3;                    // pass 1: see k_pass1
constexpr int kEpiWarp0 = 4;
constexpr int kEpiWarps = 16;                    // warps 4..19
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kAuxWarp0 = kEpiWarp0 + kEpiWarps; // warps 20..: key statistics / value norms

// Registers per thread of the calling warpgroup from here on: N, where the kernel was launched
// with BASE (every warp of the warpgroup executes this).
template <int N, int BASE>
__device__ __forceinline__ void set_regs() {
  if constexpr (N < BASE) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
  if constexpr (N > BASE) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
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

// exp2 of both halves of t on the FMA pipe, for the share of the exponentials that the
// special-function unit (16 results per clock and SM, the bound of both passes) cannot take:
// t = j + f with j the nearest integer (the magic-number add leaves j in the low mantissa bits),
// 2^f by a cubic (relative error below 7.5e-5 on [-0.5, 0.5]), j added to the exponent field.
// t is clamped at -125 (a masked logit, -inf, gives 2^-125 instead of 0).
__device__ __forceinline__ f32x2 ex2_poly2(f32x2 t2) {
  float t0, t1;
  unpack2(t2, t0, t1);
  t2 = pack2(fmaxf(t0, -125.f), fmaxf(t1, -125.f));
  const f32x2 y = add2(t2, pack2(12582912.f, 12582912.f));             // 1.5 * 2^23 + j
  const f32x2 jf = add2(y, pack2(-12582912.f, -12582912.f));
  const f32x2 f = fma2(jf, pack2(-1.f, -1.f), t2);
  f32x2 p = fma2(pack2(0.0551716536f, 0.0551716536f), f, pack2(0.242611125f, 0.242611125f));
  p = fma2(p, f, pack2(0.693260968f, 0.693260968f));
  p = fma2(p, f, pack2(0.999928057f, 0.999928057f));
  float p0, p1, y0, y1;
  unpack2(p, p0, p1);
  unpack2(y, y0, y1);
  return pack2(__uint_as_float(__float_as_uint(p0) + (__float_as_uint(y0) << 23)),
               __uint_as_float(__float_as_uint(p1) + (__float_as_uint(y1) << 23)));
}
// Of every 16 pairs of exponentials, kPolyPairs go through ex2_poly2, spread evenly.
#ifndef MIXKV_POLY_PAIRS
#define MIXKV_POLY_PAIRS 0
#endif
constexpr int kPolyPairs = MIXKV_POLY_PAIRS;
__host__ __device__ constexpr bool poly_pair(int k) {
  return ((k % 16) * kPolyPairs) % 16 < kPolyPairs && kPolyPairs > 0;
}
__device__ __forceinline__ f32x2 ex2_pair(f32x2 t2, const bool poly) {
  if (poly) return ex2_poly2(t2);
  float a0, a1;
  unpack2(t2, a0, a1);
  return pack2(ex2(a0), ex2(a1));
}

// The two bf16 of a word as a packed fp32 pair (low half first), built in place in the 64-bit
// register (a pair assembled from two separate floats costs moves).
__device__ __forceinline__ f32x2 bf16x2_wide(const uint32_t w) {
  return ((unsigned long long)(w & 0xffff0000u) << 32) | (unsigned long long)(w << 16);
}

constexpr size_t kSmemLimit = 227 * 1024;   // dynamic shared memory a CTA may ask for

// ======================================================================== pass 1
// Eight key-statistics warps (from warp 20 on): one tile = 8 pairs of 8-row batches, one pair per
// warp.  28 warps per CTA.
__host__ __device__ constexpr int p1_aux_warps(int MB) { return 8; }
__host__ __device__ constexpr int p1_threads(int MB) { return (kAuxWarp0 + p1_aux_warps(MB)) * 32; }
constexpr int kP1MaxStages = 6;
constexpr int kP1XRows = 3 * 128;   // row statistics exchanged between the warpgroups of a query row
// K tile ring: as deep as shared memory allows next to the query tile (the deeper the ring, the
// more bytes in flight towards HBM)
// (the widest query tiles leave room for four)
__host__ __device__ constexpr int p1_stages(int NQ) { return NQ > 224 ? 4 : 5; }
// registers per thread: at launch, then per role (7 warpgroups: 40 + 4 * 72 + 2 * 88 = 7 * 72;
// the key-statistics warps hold a batch of eight key rows in registers between their two sweeps)
#ifndef P1_LEAD
#define P1_LEAD 40
#define P1_EPI 72
#define P1_AUX 88
#endif
constexpr int kP1RegsLaunch = 72, kP1RegsLead = P1_LEAD, kP1RegsEpi = P1_EPI, kP1RegsAux = P1_AUX;

struct P1Bars {
  uint64_t full[kP1MaxStages];
  uint64_t empty[kP1MaxStages];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint64_t qfull;
  uint64_t qfree;
  uint32_t tmem_base;
  int abort;
};

// (m, z) pairs of the same row merged: z0 2^m0 + z1 2^m1 under the larger reference.
__device__ __forceinline__ float2 merge_stats(const float2 a, const float2 b) {
  const float mn = fmaxf(a.x, b.x);
  return make_float2(mn, a.y * ex2(a.x - mn) + b.y * ex2(b.x - mn));
}

// ---- per-head folds (pass 2, at the start of a segment): what the segments of pass 1 left
// for a (layer, sequence, head) becomes what pass 2 needs of it.
//
// kFoldDepth loads are in flight per round: a head that a one-layer call spreads over a quarter
// of the GPU's CTAs is folded in one round trip to L2.
constexpr int kFoldDepth = 40;
// Window row q: the (reference, sum) pairs of all segments merged under the largest reference,
// returned as the negated log2 normaliser of the row with the 1/W of the window mean folded in.
__device__ __forceinline__ float fold_row_stats(const float2* rowstat, const SegList& sl,
                                                const int NQ, const int q, const float log2W) {
  float M = -1e30f, Z = 0.f;
#pragma unroll 1
  for (int e0 = 0; e0 < sl.nseg; e0 += kFoldDepth) {
    float2 v[kFoldDepth];
#pragma unroll
    for (int k = 0; k < kFoldDepth; ++k) {
      v[k] = make_float2(-1e30f, 0.f);
      if (e0 + k < sl.nseg) v[k] = __ldcg(rowstat + (size_t)sl.start(e0 + k) * NQ + q);
    }
    float mx = M;
#pragma unroll
    for (int k = 0; k < kFoldDepth; ++k) mx = fmaxf(mx, v[k].x);
    Z *= ex2(M - mx);
#pragma unroll
    for (int k = 0; k < kFoldDepth; ++k) Z = fmaf(v[k].y, ex2(v[k].x - mx), Z);
    M = mx;
  }
  return -(M + log2f(Z)) - log2W;
}
// Component kt of the unit-key sum over all segments of the head.
__device__ __forceinline__ float fold_key_sums(const float* ksum, const SegList& sl, const int kt) {
  float sum = 0.f;
#pragma unroll 1
  for (int e0 = 0; e0 < sl.nseg; e0 += kFoldDepth) {
    float v[kFoldDepth];
#pragma unroll
    for (int k = 0; k < kFoldDepth; ++k)
      v[k] = e0 + k < sl.nseg ? __ldcg(ksum + (size_t)sl.start(e0 + k) * kHeadDim + kt) : 0.f;
#pragma unroll
    for (int k = 0; k < kFoldDepth; ++k) sum += v[k];
  }
  return sum;
}
// The pass-1 segments of the head that tile iterator `ti` (of either pass) stands on.
__device__ __forceinline__ SegList pass1_segments(const SeqTable& st, const TileIter& ti) {
  const int per_head = (st.tile1_start[ti.b + 1] - st.tile1_start[ti.b]) / st.H;
  return SegList(ti.layer * st.nt1 + st.tile1_start[ti.b] + ti.h * per_head, per_head, split1(st));
}

// The running softmax statistics of a query row are a pair (m, z): z = sum over the keys seen
// so far of exp2(logit * c - m), where m is a REFERENCE in log2 units, a logit of the row seen
// earlier, not necessarily the largest one: z * 2^m is the same number whatever m is, fp32
// carries 2^±126 around it, and searching the maximum of every chunk costs a quarter of the
// epilogue's instructions on its critical path.
//
// Fast path, one 32-column chunk: the sum of exp2(logit * c - m) with the standing reference.
__device__ __forceinline__ float chunk_expsum(const uint32_t (&r)[32], const float scale_log2e,
                                              const float m_run) {
  const f32x2 sc2 = pack2(scale_log2e, scale_log2e), nm2 = pack2(-m_run, -m_run);
  f32x2 za = pack2(0.f, 0.f), zb = za;
#pragma unroll
  for (int j = 0; j < 32; j += 4) {
    const f32x2 ta = fma2(pack2(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), sc2, nm2);
    const f32x2 tb = fma2(pack2(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3])), sc2, nm2);
    za = add2(za, ex2_pair(ta, poly_pair(j / 2)));
    zb = add2(zb, ex2_pair(tb, poly_pair(j / 2 + 1)));
  }
  float z0, z1;
  unpack2(add2(za, zb), z0, z1);
  return z0 + z1;
}
// A chunk sum at or above this means a logit about 2^99 above the reference (or no reference
// yet): the chunk is redone on the slow path.  Below it nothing can overflow: 1024 chunks of a
// head add up to less than 2^110.
constexpr float kChunkSumLimit = 1e30f;

// Slow path: the chunk again from tensor memory with the causal mask and a maximum search; the
// reference moves up to the chunk's maximum if that is larger.  Taken for the first chunk of
// a segment, for the tiles that need the mask, and when the fast path's sum says that the
// reference is too low.  Every lane of the warp takes part (the load is warp-wide).  Returns
// the new (m, z).
__device__ __noinline__ float2 softmax_chunk_ref(const uint32_t taddr, const bool need_mask,
                                                 const int kbase, const int lim,
                                                 const float scale_log2e, float m_run,
                                                 float z_run) {
  uint32_t r[32];
  tmem_ld32(taddr, r);
  tmem_ld_wait();
  tmem_ld_fence(r);
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
  z_run += chunk_expsum(r, scale_log2e, m_run);
  return make_float2(m_run, z_run);
}

// grid = g1 persistent CTAs of 28 warps: TMA, 2 idle, MMA, 16 epilogue, 8 key-statistics.  The
// MMA issuer is warp 3: its scheduler carries the fewest busy warps (with G*W = 224 the last
// lane quarter of the second query block is padding), and a single dependent instruction
// stream that shares a scheduler with many busy warps issues slowly enough to pace the tile
// loop.
template <int MB>
__global__ void __launch_bounds__(p1_threads(MB), 1)
k_pass1(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
        const SeqTable st, const Workspace ws, const float scale_log2e,
        int* status) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* base =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  const int kP1Stages = p1_stages(st.NQ);
  constexpr int kP1AuxWarps = p1_aux_warps(MB);
  constexpr int NU = MB == 2 ? 2 : 4;   // warpgroups that share a query row
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int NQ = st.NQ, W = st.W, H = st.H;
  // The query tile holds exactly NQ rows per 64-column half.  The MMA reads MB * 128 rows: the
  // rows past NQ are whatever follows in shared memory (the next half, the K ring), they only
  // reach accumulator lanes that nobody reads.
  unsigned char* sQ = base;                    // 2 halves x [NQ x 128 B]
  unsigned char* sK = sQ + 2 * NQ * 128;       // kP1Stages x 32 KB
  float* sks = reinterpret_cast<float*>(sK + kP1Stages * kTileBytes);  // [aux warps][128] key-sum exchange
  float2* sxs = reinterpret_cast<float2*>(sks + kP1AuxWarps * 128);    // [kP1XRows] row statistics handed over
  P1Bars* bars = reinterpret_cast<P1Bars*>(sxs + kP1XRows);
  {
    // the carve-up above must fit behind the (1 KB aligned) base
    unsigned dyn;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    if ((size_t)(reinterpret_cast<unsigned char*>(bars + 1) - smem_dyn) > dyn) {
      if (threadIdx.x == 0 && status) atomicExch(status, MIXKV_ERR_CUDA);
      return;
    }
  }

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
      // every epilogue warp that owns query rows reads every tile; warps on padding rows (the
      // last lane quarters of the last block) neither wait nor arrive: a warp that polls a
      // barrier takes issue slots from the scheduler it shares with the MMA issuer
      mbar_init(&bars->tempty[s], (kEpiWarps / (MB * 4)) * ((NQ + 31) / 32));
    }
    mbar_init(&bars->qfull, 1);
    mbar_init(&bars->qfree, 1);
    bars->abort = 0;
    mbar_init_fence();
  }
  if (warp == kP1WarpMma) tmem_alloc(&bars->tmem_base, MB * 256);
  if (warp == kWarpTma && lane == 0) {
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmQ);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  pdl_wait();   // everything earlier in the stream is complete: global memory may be touched

  if (warp < kEpiWarp0) {
    set_regs<kP1RegsLead, kP1RegsLaunch>();
    if (warp == kWarpTma) {
      // ---------------------------------------------------------------- TMA producer
      if (lane == 0) {
        int it = 0, segn = 0;
        bool seg_start = true;
        for (TileIter ti(st.tile1_start, st.batch, H, st.nt1, lo, hi); ti.valid(); ti.next()) {
          if (seg_start) {
            if (segn > 0 && !mbar_wait(&bars->qfree, (segn - 1) & 1, abort)) break;
            mbar_expect_tx(&bars->qfull, NQ * 256);
            tma_load_3d(sQ, &tmQ, 0, ti.bh() * NQ, ti.layer, &bars->qfull);
            tma_load_3d(sQ + NQ * 128, &tmQ, 64, ti.bh() * NQ, ti.layer, &bars->qfull);
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
    } else if (warp == kP1WarpMma) {
      // ---------------------------------------------------------------- MMA issuer
      if (lane == 0) {
        constexpr uint32_t idesc = umma_idesc_bf16(128, kTile);
        const uint32_t q_lo = umma_desc_lo(smem_u32(sQ));
        const uint32_t k_lo = umma_desc_lo(smem_u32(sK));
        const uint32_t q_half = (uint32_t)(NQ * 128) >> 4;   // second 64-column half of the queries
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
          const uint32_t kb_lo = k_lo + (uint32_t)s * (kTileBytes >> 4);
          const uint32_t td = tmem + ts * (MB * 128);
#pragma unroll
          for (int mb = 0; mb < MB; ++mb) {
            // k-steps of 16 columns: 32 bytes apart inside a 64-column half
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint32_t a_lo = q_lo + (ks >> 2) * q_half + (uint32_t)(mb * (16384 >> 4) + (ks & 3) * 2);
              const uint32_t b_lo = kb_lo + (uint32_t)((ks >> 2) * (kHalfBytes >> 4) + (ks & 3) * 2);
              if (ks == 0)
                umma_bf16_lo<0>(td + mb * 128, a_lo, b_lo, idesc);
              else
                umma_bf16_lo<1>(td + mb * 128, a_lo, b_lo, idesc);
            }
          }
          umma_commit(&bars->empty[s]);
          umma_commit(&bars->tfull[ts]);
          if (seg_start) umma_commit(&bars->qfree);
          ++it;
        }
        if (*abort) raise(status, abort);
      }
    }
  } else if (warp < kAuxWarp0) {
    // ------------------------------------------------------------------ epilogue
    // All sixteen warps read every tile (two accumulator stages: the MMA of the next tile fills
    // the other stage meanwhile).  Warpgroup wg = 0..3:
    // MB == 2: query rows (wg / 2) * 128 .. +127, keys (wg % 2) * 64 .. +63 of the tile;
    // MB == 1: query rows 0 .. 127, keys wg * 32 .. +31.
    set_regs<kP1RegsEpi, kP1RegsLaunch>();
    const int wg = (warp - kEpiWarp0) >> 2, quarter = warp & 3;
    const int blk = MB == 2 ? wg >> 1 : 0;
    const int unit = MB == 2 ? wg & 1 : wg;      // which partial result of the row this is
    constexpr int NC = MB == 2 ? 64 : 32;        // columns (keys) this thread reduces per tile
    const int row = blk * 128 + quarter * 32 + lane;
    const int col0 = blk * 128 + unit * NC;
    const bool warp_on = blk * 128 + quarter * 32 < NQ;
    const int jrow = row % W;
    // The NU warpgroups that share a query row merge their statistics at the end of a segment:
    // units 1 .. NU-1 hand theirs over through shared memory, unit 0 merges and writes one pair
    // per row.  Named barriers 6 + blk ("handed over") and 8 + blk ("read").
    const int xrow = (unit > 0 ? unit - 1 : 0) * 128 + (MB == 2 ? blk * 128 : 0) + quarter * 32 + lane;
    constexpr int kXThreads = NU * 128;
    float m_run = -1e30f, z_run = 0.f;
    int it = 0, seg_first = lo, segs_done = 0;
    bool seg_start = true, no_ref = true;
    for (TileIter ti(st.tile1_start, st.batch, H, st.nt1, lo, hi); ti.valid(); ti.next()) {
      if (seg_start) {
        m_run = -1e30f;
        z_run = 0.f;
        no_ref = true;   // the segment's first chunk sets the reference
        seg_first = ti.id;
      }
      seg_start = ti.seg_last();
      const int L = st.cu[ti.b + 1] - st.cu[ti.b], P = L - W;
      const int ts = it & 1, tph = (it >> 1) & 1;
      // (after an abort the waits fail at once; the loop goes on without work so that the
      // segment-end barriers below stay matched)
      const bool ok = warp_on && mbar_wait(&bars->tfull[ts], tph, abort);
      if (ok) {
        tc_fence_after();
        const int k0 = ti.t * kTile + unit * NC;
        const bool need_mask = ti.t * kTile + kTile > P;
        const int lim = P + jrow;   // last key this row may see
        const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + ts * (MB * 128) + col0;
#pragma unroll 1
        for (int c0 = 0; c0 < NC; c0 += 32) {   // kept rolled: the body must stay in the i-cache
          bool slow = no_ref || need_mask;      // the same in every lane
          float zc = 0.f;
          if (!slow) {
            uint32_t ra[32];
            tmem_ld32(taddr + c0, ra);
            tmem_ld_wait();
            tmem_ld_fence(ra);
            zc = chunk_expsum(ra, scale_log2e, m_run);
            slow = __any_sync(0xffffffffu, !(zc < kChunkSumLimit));
          }
          if (slow) {
            const float2 mz =
                softmax_chunk_ref(taddr + c0, need_mask, k0 + c0, lim, scale_log2e, m_run, z_run);
            m_run = mz.x;
            z_run = mz.y;
            no_ref = false;
          } else {
            z_run += zc;
          }
        }
      }
      if (warp_on) {
        tc_fence_before();
        __syncwarp();   // one arrival per warp: 512 single arrivals on one word cost more than a chunk
        if (lane == 0) mbar_arrive(&bars->tempty[ts]);
      }
      if (seg_start) {   // (here: this was the segment's last tile)
        if (unit > 0) {
          if (segs_done > 0) named_bar_sync(8 + blk, kXThreads);   // the last hand-over was read
          sxs[xrow] = make_float2(m_run, z_run);
          named_bar_arrive(6 + blk, kXThreads);
        } else {
          named_bar_sync(6 + blk, kXThreads);
          float2 mz = make_float2(m_run, z_run);
#pragma unroll
          for (int u = 1; u < NU; ++u) mz = merge_stats(mz, sxs[xrow + (u - 1) * 128]);
          named_bar_arrive(8 + blk, kXThreads);
          if (row < NQ) ws.rowstat[(size_t)seg_first * NQ + row] = mz;
        }
        ++segs_done;
      }
      ++it;
    }
  } else {
    // ------------------------------------------------------------------ key statistics
    // Sixteen lanes share a key row (one 16-byte chunk each); a pair of 8-row batches is one
    // warp-wide step (one batch per 16-lane group).  Sweep 1 squares, a butterfly leaves the
    // squared norm of row r with lanes 2r and 2r+1, sweep 2 adds the rows scaled by 1/|k| into
    // eight per-thread sums (dims 8c .. 8c+7).
    set_regs<kP1RegsAux, kP1RegsLaunch>();
    const int aux_w = warp - kAuxWarp0;
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
      {
        const int row0 = (2 * aux_w + lg) * 8;
        uint4 u[8];
        float p[8];
#pragma unroll
        for (int rr = 0; rr < 8; ++rr) {
          u[rr] = *reinterpret_cast<const uint4*>(tile + sw128_offset(row0 + rr, cc));
          const uint32_t* p2 = reinterpret_cast<const uint32_t*>(&u[rr]);
          f32x2 sq = pack2(0.f, 0.f);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const f32x2 f2 = bf16x2_wide(p2[e]);
            sq = fma2(f2, f2, sq);
          }
          float s0, s1;
          unpack2(sq, s0, s1);
          p[rr] = s0 + s1;
        }
        // the tile now lives in registers: hand the stage back
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->empty[s]);
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
          const uint32_t* p2 = reinterpret_cast<const uint32_t*>(&u[rr]);
          const f32x2 w2 = pack2(w, w);
#pragma unroll
          for (int e = 0; e < 4; ++e) acc2[e] = fma2(bf16x2_wide(p2[e]), w2, acc2[e]);
        }
      }
      // (no barrier per tile: after an abort the waits fail at once and every warp still walks
      // the same tiles, so the segment-end barriers below stay matched)
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
  if (warp == kP1WarpMma) tmem_dealloc(tmem, MB * 256);
  if (tid == 0 && bars->abort && status) atomicExch(status, MIXKV_ERR_TIMEOUT);
  // every partial result of this CTA's segments is written: pass 2 folds them per head
}

// ======================================================================== pass 2
// Pass 2 streams K and V and sits at the HBM bound with sixteen warps: K/Q producer, MMA, V
// producer, 1 idle, two epilogue warpgroups that own alternate tiles (every thread one key and all
// of its G*W logit columns, so nothing is exchanged between warps), 4 value-norm warps.  More
// epilogue warps splitting the columns of a tile were measured slower (C3: 13.4 against 11.7 us per
// layer): the exchange of partial sums and the extra warps cost more than they hide.
constexpr int kP2Threads = 16 * 32;
constexpr int kP2EpiWarps = 8;                   // warps 4..11
constexpr int kP2AuxWarp0 = 12;                  // warps 12..15: value norms

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
__global__ void __launch_bounds__(kP2Threads, 1)
k_pass2(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
        const __grid_constant__ CUtensorMap tmQ, const SeqTable st, const Workspace ws,
        float* __restrict__ s_div_out, float* __restrict__ rbar_out, const float scale_log2e,
        const int use_vnorm, const int pool_half, const int vstages, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* base =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  const int NQ = st.NQ, W = st.W, H = st.H;
  const int NB = NQ + kExtraRows;             // rows of the B operand
  unsigned char* sQ = base;                   // 2 halves x [NB x 128 B]
  unsigned char* sK = sQ + 2 * NB * 128;      // kP2KStages x 32 KB
  unsigned char* sV = sK + kP2KStages * kTileBytes;   // vstages x 16 KB
  float* sbq = reinterpret_cast<float*>(sV + vstages * kVSubBytes);  // [256] negated normalisers (+ 256 spare)
  float* sred = sbq + 512;                    // [64]: 2 x 16 epilogue, 12 value norms, 4 mean key
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
  } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kP2EpiWarps) {
    // ------------------------------------------------------------------ epilogue
    // The two warpgroups take alternate tiles (warpgroup g owns accumulator stage g), one key
    // per thread and all G*W columns of it, so a tile needs no exchange between warpgroups and
    // inside a segment the groups never wait for each other; each leaves its own partial score
    // statistics.  At the start of a segment the 256 threads fold the row statistics of the
    // head together, one window row per thread, into the normaliser table both groups read.
    // Nobody leaves the tile loop early: after an abort every wait fails at once, so the
    // named barriers of the segment boundaries stay matched.
    const int quarter = warp & 3, wg = (warp - kEpiWarp0) >> 2;
    const int gt = (tid - kEpiWarp0 * 32) & 127;   // thread inside the warpgroup
    const int gw = gt >> 5;                        // warp inside the warpgroup
    const int key = quarter * 32 + lane;
    const int nch = NQ / 16;
    const int et = tid - kEpiWarp0 * 32;           // thread inside the epilogue, 0..255
    const float log2W = log2f((float)W);
    const int barid = 1 + wg;                      // named barriers 1, 2: one per warpgroup
    const f32x2 sc2 = pack2(scale_log2e, scale_log2e);
    float dmin = INFINITY, dmax = -INFINITY, dsum = 0.f, exw = 0.f;
    int it = 0, seg_first = lo;
    bool seg_start = true;
    for (TileIter ti(st.tile2_start, st.batch, H, st.nt2, lo, hi); ti.valid(); ti.next()) {
      const int L = st.cu[ti.b + 1] - st.cu[ti.b], P = L - W;
      if (seg_start) {
        named_bar_sync(5, kP2EpiWarps * 32);   // the previous segment's readers of sbq are done
        if (et < NQ) sbq[et] = fold_row_stats(ws.rowstat, pass1_segments(st, ti), NQ, et, log2W);
        dmin = INFINITY, dmax = -INFINITY, dsum = 0.f, exw = 0.f;
        seg_first = ti.id;
        named_bar_sync(5, kP2EpiWarps * 32);
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
            colsum_chunk<32>(ra, sbq + ci * 32, sc2, acc);
          }
          if (nch & 1) {
            uint32_t rb[16];
            tmem_ld16(taddr + n32 * 32, rb);
            tmem_ld_wait();
            tmem_ld_fence(rb);
            colsum_chunk<16>(rb, sbq + n32 * 32, sc2, acc);
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
  } else if (warp >= kP2AuxWarp0) {
    // ------------------------------------------------------------------ mean key, value norms
    // At the start of a segment: fold the unit-key sums of the head's pass-1 segments (one
    // dimension per thread) and write the bf16 hi / lo / lo2 split of the mean unit key into the
    // three extra B rows; the CTA that starts on the head's first tile also leaves the redundancy
    // of Eq. 4, which needs nothing but the squared norm of that sum.  Per tile: warps 12, 13 read the first 64 rows of the V
    // tile, warps 14, 15 the last 64; one row per thread from the swizzled half tile.
    const int vt = tid - kP2AuxWarp0 * 32;         // 0..127
    const int sub = vt >> 6, vr = vt & 63;
    float vmin = INFINITY, vmax = -INFINITY, vsum = 0.f;
    int it = 0, segn = 0, seg_first = lo;
    bool seg_start = true;
    for (TileIter ti(st.tile2_start, st.batch, H, st.nt2, lo, hi); ti.valid(); ti.next()) {
      if (seg_start) {
        const int L = st.cu[ti.b + 1] - st.cu[ti.b];
        const float ks = fold_key_sums(ws.ksum, pass1_segments(st, ti), vt);
        const float kb = ks / (float)L;   // mean unit key
        if (ti.t == 0) {                  // the same in all 128 threads
          const float n2 = warp_sum(ks * ks);
          if (lane == 0) sred[44 + (warp - kP2AuxWarp0)] = n2;
          named_bar_sync(4, 128);
          if (vt == 0) {
            const double nn = ((double)sred[44] + (double)sred[45]) + ((double)sred[46] + (double)sred[47]);
            const double T = (double)L;
            const float r = (float)((nn - T) / (T * (T - 1.0)));   // Eq. 4
            ws.rbar[ti.unit()] = r;
            if (rbar_out) rbar_out[ti.unit()] = r;
          }
        }
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
              const uint32_t* p2 = reinterpret_cast<const uint32_t*>(&u);
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const f32x2 f2 = bf16x2_wide(p2[e]);
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
      // The four warps stay within one tile of each other.  With an odd number of V stages the
      // two pairs of warps take turns on the same stage: a pair that ran ahead would wait for
      // a phase of vfull whose predecessor it never saw complete, and a parity wait on a
      // barrier that is still one phase behind returns at once.
      named_bar_sync(3, 128);
      if (seg_start && use_vnorm) {
        const float a = warp_min(vmin), b2 = warp_max(vmax), c2 = warp_sum(vsum);
        const int vw = warp - kP2AuxWarp0;
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

size_t pass1_smem(int MB, int NQ) {
  // up to 1023 bytes of alignment slack in front of the carve-up; never beyond the limit (the
  // kernel checks that its carve-up fits behind the aligned base)
  const size_t need = (size_t)2 * NQ * 128 + (size_t)p1_stages(NQ) * kTileBytes + p1_aux_warps(MB) * 128 * 4 +
                      kP1XRows * 8 + sizeof(P1Bars);
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

bool encode_bf16_map(void* tm, const void* base, int rank, const unsigned long long* dims,
                     const unsigned long long* strides_bytes, const unsigned* box) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  cuuint64_t d[5], st[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) d[i] = dims[i], bx[i] = box[i], es[i] = 1;
  for (int i = 0; i + 1 < rank; ++i) st[i] = strides_bytes[i];
  return enc(reinterpret_cast<CUtensorMap*>(tm), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
             const_cast<void*>(base), d, st, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

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

cudaError_t launch_pass1(const LaunchCtx& c, const void* K, const void* Q, int* status) {
  CUtensorMap tmK, tmQ;
  if (!map_kv(c, K, kTile, &tmK) || !map_q(c, Q, &tmQ)) return cudaErrorInvalidValue;
  static bool done1[64] = {false}, done2[64] = {false};
  if (c.st.NQ <= 128) {
    const size_t smem = pass1_smem(1, c.st.NQ);
    cudaError_t e = ensure_smem(k_pass1<1>, kSmemLimit, done1);
    if (e != cudaSuccess) return e;
    return launch_pdl(k_pass1<1>, dim3(c.st.g1), dim3(p1_threads(1)), smem, c.stream, 1, tmK, tmQ, c.st,
                      c.ws, c.scale_log2e, status);
  }
  const size_t smem = pass1_smem(2, c.st.NQ);
  cudaError_t e = ensure_smem(k_pass1<2>, kSmemLimit, done2);
  if (e != cudaSuccess) return e;
  return launch_pdl(k_pass1<2>, dim3(c.st.g1), dim3(p1_threads(2)), smem, c.stream, 1, tmK, tmQ, c.st,
                    c.ws, c.scale_log2e, status);
}

cudaError_t launch_pass2(const LaunchCtx& c, const void* K, const void* V, const void* Q,
                         float* s_div_out, float* rbar_out, int* status) {
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
  return launch_pdl(k_pass2, dim3(c.st.g2), dim3(kP2Threads), smem, c.stream, 1, tmK, tmV, tmQ, c.st,
                    c.ws, s_div_out, rbar_out, c.scale_log2e, c.p.use_vnorm, c.p.pool_kernel >> 1,
                    vstages, status);
}

}  // namespace mixkv
