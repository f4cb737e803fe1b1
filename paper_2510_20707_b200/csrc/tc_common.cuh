// Blackwell (sm_100a) building blocks used by the two K passes: mbarriers with bounded
// waits, TMA tile loads, tcgen05 (UMMA) descriptors / issue / commit, TMEM allocation and
// loads.  Every wait is bounded in wall-clock time: when it expires the waiting thread raises
// the CTA-wide abort flag and the kernel drains and returns with an error status instead of
// hanging.
#pragma once

#include <cuda.h>
#include <stdint.h>

#include "common.cuh"

namespace mixkv {

constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s per wait

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_init_fence() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return done != 0;
}

// Waits for the barrier phase `parity`.  Returns false (after raising *abort) when the time
// limit passes or another thread of the CTA has already aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 255u) == 0) {
      if (*abort) return false;
      if (global_ns() - t0 > kWaitLimitNs) {
        *abort = 1;
        return false;
      }
    }
  }
}

// TMA tile loads (no multicast); coordinates innermost first.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int x, int y,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], "
      "[%1, {%2, %3}], [%4];" ::"r"(smem_u32(dst)),
      "l"(tm), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* tm, int x, int y, int z,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], "
      "[%1, {%2, %3, %4}], [%5];" ::"r"(smem_u32(dst)),
      "l"(tm), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* tm, int x, int y, int z,
                                            int w, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], "
      "[%1, {%2, %3, %4, %5}], [%6];" ::"r"(smem_u32(dst)),
      "l"(tm), "r"(x), "r"(y), "r"(z), "r"(w), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 operand stored as rows of 128 bytes with
// the 128-byte swizzle (what a TMA box of 64 bf16 x rows writes): 8-row groups are 1024 bytes
// apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
  d |= (uint64_t)1 << 16;            // leading byte offset: unused for swizzled K-major
  d |= (uint64_t)(1024 >> 4) << 32;  // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;            // descriptor version (Blackwell)
  d |= (uint64_t)2 << 61;            // SWIZZLE_128B
  return d;
}

// Instruction descriptor: D f32, A and B bf16, both K-major, M x N tile.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same descriptor as two 32-bit halves: the high half is a constant, the low half is
// ((address >> 4) & 0x3fff) | 1 << 16, so stepping an operand by n bytes (n a multiple of 16,
// inside shared memory) is an integer add of n >> 4 to the low half: the issuing thread
// builds a descriptor with one add instead of a dozen 64-bit operations.
constexpr uint32_t kUmmaDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t saddr) {
  return ((saddr >> 4) & 0x3FFFu) | (1u << 16);
}
template <int ACC>
__device__ __forceinline__ void umma_bf16_lo(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo,
                                             uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(tmem_d),
      "r"(a_lo), "r"(b_lo), "r"(kUmmaDescHi), "r"(idesc), "n"(ACC)
      : "memory");
}
// Arrives on the barrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                   smem_u32(slot)),
               "r"(cols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols)
               : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread l of the warp gets lane (base lane + l).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t (&r)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// The registers written by tcgen05.ld are only valid after tcgen05.wait::ld.  This empty
// statement makes every later use of r depend on a point after the wait (volatile asm
// statements keep their order), so the compiler cannot hoist arithmetic above it.
__device__ __forceinline__ void tmem_ld_fence(uint32_t (&r)[16]) {
  asm volatile(""
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]),
                 "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]),
                 "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :
               : "memory");
}
__device__ __forceinline__ void tmem_ld_fence(uint32_t (&r)[32]) {
  asm volatile(""
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]),
                 "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]),
                 "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :
               : "memory");
  asm volatile(""
               : "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]),
                 "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]),
                 "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
__device__ __forceinline__ void tmem_ld_fence(uint32_t (&r)[4]) {
  asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]) : : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Arrives at a named barrier without waiting (the other side calls named_bar_sync with the
// same thread count); shared-memory writes before it are visible to the threads that sync.
__device__ __forceinline__ void named_bar_arrive(int id, int threads) {
  __threadfence_block();
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Byte offset of element (row r, 16-byte chunk c in 0..7) inside a [rows x 128 B] half tile
// written with the 128-byte swizzle (tile base 1024-byte aligned).
__device__ __forceinline__ uint32_t sw128_offset(int r, int c) {
  return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4));
}

// ---- persistent tile schedule shared by every role of a CTA ----------------------------
// Tiles are 128 consecutive keys of one (sequence, head), numbered in (b, h, t) order.
struct TileCoord {
  int b, h, t, bh;
};

__device__ __forceinline__ TileCoord tile_coord(const int* tile_start, int batch, int H,
                                                int id) {
  const int b = find_seq(tile_start, batch, id);
  const int per_head = (tile_start[b + 1] - tile_start[b]) / H;
  const int rem = id - tile_start[b];
  TileCoord c;
  c.b = b;
  c.h = rem / per_head;
  c.t = rem - c.h * per_head;
  c.bh = b * H + c.h;
  return c;
}
__host__ __device__ __forceinline__ Split split1(const SeqTable& st) {
  return Split{st.layers * st.nt1, st.g1, st.q1, st.r1};
}
__host__ __device__ __forceinline__ Split split2(const SeqTable& st) {
  return Split{st.layers * st.nt2, st.g2, st.q2, st.r2};
}
// First tile of CTA c.
__host__ __device__ __forceinline__ int cta_first_tile(int c, const Split& sp) {
  return c * sp.q + (c < sp.r ? c : sp.r);
}
// CTA whose contiguous range contains tile t.
__host__ __device__ __forceinline__ int tile_owner(int t, const Split& sp) {
  const int big = sp.r * (sp.q + 1);
  return t < big ? t / (sp.q + 1) : sp.r + (t - big) / sp.q;
}

// Walks the tiles [lo, hi) of one CTA in (layer, b, h, t) order without dividing per tile.
// Tile ids run over all layers: id = layer * nt + (tile of the layer).
struct TileIter {
  int id, hi, layer, b, h, t, per_head, H, batch, nt;
  const int* tile_start;
  __device__ TileIter(const int* tile_start_, int batch_, int H_, int nt_, int lo, int hi_)
      : id(lo), hi(hi_), H(H_), batch(batch_), nt(nt_), tile_start(tile_start_) {
    layer = b = h = t = 0;
    per_head = 1;
    if (lo < hi_) {
      layer = lo / nt_;
      const TileCoord c = tile_coord(tile_start_, batch_, H_, lo - layer * nt_);
      b = c.b, h = c.h, t = c.t;
      per_head = (tile_start_[b + 1] - tile_start_[b]) / H_;
    }
  }
  __device__ __forceinline__ bool valid() const { return id < hi; }
  // (sequence, head) of the tile inside its layer, and over all layers
  __device__ __forceinline__ int bh() const { return b * H + h; }
  __device__ __forceinline__ int unit() const { return (layer * batch + b) * H + h; }
  // last tile of a segment: a run of tiles of one (layer, b, h) inside this CTA's range
  __device__ __forceinline__ bool seg_last() const { return id + 1 == hi || t + 1 == per_head; }
  __device__ __forceinline__ void next() {
    ++id;
    if (++t == per_head) {
      t = 0;
      if (++h == H) {
        h = 0;
        if (++b == batch) {
          b = 0;
          ++layer;
        }
        if (id < hi) per_head = (tile_start[b + 1] - tile_start[b]) / H;
      }
    }
  }
};

// Segments of one (b, h) when its tiles [T0, T0 + per_head) lie in a tile list split
// contiguously over CTAs: segment e starts at T0 for e = 0 and at the first tile of CTA
// c0 + e otherwise (c0 = CTA that owns T0).
struct SegList {
  int T0, c0, nseg;
  Split sp;
  __device__ SegList(int T0_, int per_head, const Split& sp_) : T0(T0_), sp(sp_) {
    c0 = tile_owner(T0_, sp_);
    nseg = tile_owner(T0_ + per_head - 1, sp_) - c0 + 1;
  }
  __device__ __forceinline__ int start(int e) const {
    return e == 0 ? T0 : cta_first_tile(c0 + e, sp);
  }
};

}  // namespace mixkv
