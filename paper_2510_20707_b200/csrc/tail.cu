// Everything after the two K passes: the per-head scalars, pooling, the head-wise mix (Eq. 2,
// Eq. 5), budgets, per-head top-B selection and the gather (Algorithm 1, step 2 and the TopB
// line).  The fixed-budget layer call runs all of it in ONE kernel, k_tail: a cluster of eight
// CTAs per (sequence, head) mixes the scores of its slice, finds the selection threshold by
// radix passes whose histograms are combined through distributed shared memory, compacts the
// kept positions in ascending order and copies the kept K / V rows.
#include <cooperative_groups.h>

#include "tc_common.cuh"

namespace cg = cooperative_groups;

namespace mixkv {

namespace {

// ------------------------------------------------------------------- per-head scalars
// Everything Eq. 2 / Eq. 5 need besides the per-position values, folded from the per-segment
// partials pass 2 left behind.  Computed by one warp; the five results go to sc[0..4]:
//   s_in_scaled  = (|V_i| - sc[0]) * sc[1]
//   s_div_scaled = (s_div_i - sc[2]) * sc[3]
//   sc[4]        = redundancy used by the mix
__device__ void head_scalars(const SeqTable& st, const Workspace& ws, const int layer, const int b,
                             const int h, const int pool_k, const int pool_mode, const int use_vnorm,
                             const float eps, const float* __restrict__ rbar_in, const int lane,
                             float* sc) {
  const int unit = (layer * st.batch + b) * st.H + h;
  const int P = st.cu[b + 1] - st.cu[b] - st.W;
  float dmin = INFINITY, dmax = -INFINITY, dsum = 0.f, exw = 0.f;
  float vmin = INFINITY, vmax = -INFINITY, vsum = 0.f;
  float rbar = 0.f;
  if (lane == 0) rbar = rbar_in ? rbar_in[unit] : ws.rbar[unit];
  {
    const int per_head = (st.tile2_start[b + 1] - st.tile2_start[b]) / st.H;
    const SegList sl(layer * st.nt2 + st.tile2_start[b] + h * per_head, per_head, split2(st));
    // lanes take segments side by side, two per lane and round; all loads of a round are
    // issued before the first is used
    for (int e0 = lane; e0 < sl.nseg; e0 += 64) {
      float4 d4[2], e4[2], v4[2];
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int e = e0 + 32 * k;
        d4[k] = e4[k] = make_float4(INFINITY, -INFINITY, 0.f, 0.f);
        v4[k] = d4[k];
        if (e < sl.nseg) {
          const int start = sl.start(e);
          d4[k] = ws.dstat[(size_t)start * 2];
          e4[k] = ws.dstat[(size_t)start * 2 + 1];
          if (use_vnorm) v4[k] = ws.vstat[start];
        }
      }
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        dmin = fminf(dmin, fminf(d4[k].x, e4[k].x));
        dmax = fmaxf(dmax, fmaxf(d4[k].y, e4[k].y));
        dsum += d4[k].z + e4[k].z;
        exw += d4[k].w + e4[k].w;
        vmin = fminf(vmin, v4[k].x);
        vmax = fmaxf(vmax, v4[k].y);
        vsum += v4[k].z;
      }
    }
  }
  float ex;
  if (pool_mode == MIXKV_POOL_AVG) {
    // sum of the zero-padded average-pooled score = sum of raw[m] * (windows covering m) / k
    ex = warp_sum(exw) / (float)pool_k;
  } else {
    float e = 0.f;
    for (int c = st.pchunk_start[b] + lane; c < st.pchunk_start[b + 1]; c += 32)
      e += ws.exsum[((size_t)layer * st.H + h) * st.pchunks_total + c];
    ex = warp_sum(e);
  }
  dmin = warp_min(dmin);
  dmax = warp_max(dmax);
  dsum = warp_sum(dsum);
  vmin = warp_min(vmin);
  vmax = warp_max(vmax);
  vsum = warp_sum(vsum);
  if (lane == 0) {
    const float invP = 1.0f / (float)P;
    const float mean_ex = ex * invP;
    float v0 = 0.f, cin = 0.f, mean_imp = mean_ex;
    if (use_vnorm) {
      const float vinv = 1.0f / (vmax - vmin + eps);
      const float mean_in = (vsum * invP - vmin) * vinv;
      const float a_in = mean_ex / (mean_in + eps);
      v0 = vmin;
      cin = vinv * a_in;
      mean_imp = mean_ex + mean_in * a_in;
    }
    const float dinv = 1.0f / (dmax - dmin + eps);
    const float mean_dn = (dsum * invP - dmin) * dinv;
    const float a_div = mean_imp / (mean_dn + eps);
    sc[0] = v0;
    sc[1] = cin;
    sc[2] = dmin;
    sc[3] = dinv * a_div;
    sc[4] = rbar;
  }
}

// Pooled attention score at one position from a staged window w[0..k) (centre at w[k/2]);
// positions outside the candidates were staged as 0 (average) or -inf (max).
__device__ __forceinline__ float pool_window(const float* w, const int k, const int mode,
                                             const float invk) {
  if (mode == MIXKV_POOL_AVG) {
    float v = 0.f;
    for (int u = 0; u < k; ++u) v += w[u];
    return v * invk;
  }
  float v = -INFINITY;
  for (int u = 0; u < k; ++u) v = fmaxf(v, w[u]);
  return v;
}

__device__ __forceinline__ float mix_one(const float ex, const float vn, const float dv,
                                         const float* sc, const int use_vnorm,
                                         const int mix_mode) {
  float imp = ex;
  if (use_vnorm) imp += (vn - sc[0]) * sc[1];
  const float dsc = (dv - sc[2]) * sc[3];
  const float r = sc[4];
  switch (mix_mode) {
    case MIXKV_MIX_HEADWISE: return (1.0f - r) * imp + r * dsc;   // Eq. 5
    case MIXKV_MIX_IMPORTANCE_ONLY: return imp;
    case MIXKV_MIX_DIVERSITY_ONLY: return dv;
    default: return imp + dsc;
  }
}

struct MixParams {
  int pool_k, pool_mode, use_vnorm, mix_mode;
  float eps;
};

// --------------------------------------------------------------------------- poolsum
// Max pooling only: per-chunk sums of the pooled score (its mean enters Eq. 2).
__global__ void __launch_bounds__(256)
k_poolsum(const SeqTable st, const Workspace ws, const int k) {
  __shared__ float tile[kPChunk + 64];
  __shared__ float sred[8];
  pdl_launch_dependents();
  pdl_wait();
  const int pcx = blockIdx.x, h = blockIdx.y, layer = blockIdx.z;
  const int b = find_seq(st.pchunk_start, st.batch, pcx);
  const int P = st.cu[b + 1] - st.cu[b] - st.W;
  const int p0 = (pcx - st.pchunk_start[b]) * kPChunk;
  const int p1 = min(p0 + kPChunk, P);
  const size_t poff = ppos(st, layer, h, b, 0);
  const int half = k >> 1;
  for (int t = threadIdx.x; t < (p1 - p0) + 2 * half; t += 256) {
    const int i = p0 - half + t;
    tile[t] = (i >= 0 && i < P) ? ws.s_ex_raw[poff + i] : -INFINITY;
  }
  __syncthreads();
  float sum = 0.f;
  for (int t = threadIdx.x; t < p1 - p0; t += 256) sum += pool_window(tile + t, k, MIXKV_POOL_MAX, 0.f);
  sum = warp_sum(sum);
  if ((threadIdx.x & 31) == 0) sred[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
    for (int w = 0; w < 8; ++w) s += sred[w];
    ws.exsum[((size_t)layer * st.H + h) * st.pchunks_total + pcx] = s;
  }
}

// --------------------------------------------------------------------------- mixpool
// Pooling and the mix over a grid of position chunks (the scores entry point, adaptive budgets).
__global__ void __launch_bounds__(256)
k_mixpool(const SeqTable st, const Workspace ws, const float* __restrict__ s_div,
          const float* __restrict__ rbar_in, float* __restrict__ s_ex_out,
          float* __restrict__ s_comp, const MixParams mp) {
  __shared__ float tile[kPChunk + 64];
  __shared__ float sc[8];
  pdl_launch_dependents();
  pdl_wait();
  const int pcx = blockIdx.x, h = blockIdx.y, layer = blockIdx.z;
  const int b = find_seq(st.pchunk_start, st.batch, pcx);
  const int P = st.cu[b + 1] - st.cu[b] - st.W;
  const int p0 = (pcx - st.pchunk_start[b]) * kPChunk;
  const int p1 = min(p0 + kPChunk, P);
  const size_t poff = ppos(st, layer, h, b, 0);
  const int half = mp.pool_k >> 1;
  const float pad = mp.pool_mode == MIXKV_POOL_AVG ? 0.f : -INFINITY;
  if (threadIdx.x < 32)
    head_scalars(st, ws, layer, b, h, mp.pool_k, mp.pool_mode, mp.use_vnorm, mp.eps, rbar_in,
                 threadIdx.x, sc);
  // a chunk is eight rounds of 256 positions (+ the pooling halo in a ninth); every load of the
  // chunk is issued before the first use
  constexpr int kRounds = kPChunk / 256;
  const int nstage = (p1 - p0) + 2 * half;
  float raw[kRounds + 1], vn[kRounds], dv[kRounds];
#pragma unroll
  for (int e = 0; e <= kRounds; ++e) {
    const int t = e * 256 + threadIdx.x, i = p0 - half + t;
    raw[e] = (t < nstage && i >= 0 && i < P) ? ws.s_ex_raw[poff + i] : pad;
  }
#pragma unroll
  for (int e = 0; e < kRounds; ++e) {
    const int i = p0 + e * 256 + threadIdx.x;
    vn[e] = (mp.use_vnorm && i < p1) ? ws.vnorm[poff + i] : 0.f;
    dv[e] = i < p1 ? s_div[poff + i] : 0.f;
  }
#pragma unroll
  for (int e = 0; e <= kRounds; ++e) {
    const int t = e * 256 + threadIdx.x;
    if (t < nstage) tile[t] = raw[e];
  }
  __syncthreads();
  const float invk = 1.0f / (float)mp.pool_k;
#pragma unroll
  for (int e = 0; e < kRounds; ++e) {
    const int t = e * 256 + threadIdx.x, i = p0 + t;
    if (i < p1) {
      const float ex = pool_window(tile + t, mp.pool_k, mp.pool_mode, invk);
      if (s_ex_out) s_ex_out[poff + i] = ex;
      s_comp[poff + i] = mix_one(ex, vn[e], dv[e], sc, mp.use_vnorm, mp.mix_mode);
    }
  }
}

// ------------------------------------------------------------------- radix selection
// Order-preserving map float -> uint32 (larger float, larger key); -0 is folded into +0 so
// that equal floats have equal keys.
__device__ __forceinline__ unsigned order_key(float f) {
  unsigned u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Adds the 32 digits of a warp (0xffffffff = none) to a shared-memory histogram.  The digit of
// the lowest lane, then the digit of the lowest lane left, are counted with one vote and one add
// each (the first passes of a selection see one or two digits almost everywhere); what is left
// after that is spread over the bins and is added lane by lane.
__device__ __forceinline__ void count_digits(int* hist, const unsigned digit, const int lane) {
  unsigned left = 0xffffffffu;
#pragma unroll
  for (int round = 0; round < 2; ++round) {
    const int src = __ffs(left) - 1;                       // lowest lane not counted yet
    const unsigned d = __shfl_sync(0xffffffffu, digit, src);
    const unsigned same = __ballot_sync(0xffffffffu, digit == d) & left;
    if (lane == src && d != 0xffffffffu) atomicAdd(&hist[d], __popc(same));
    left &= ~same;
    if (left == 0) return;                                 // uniform across the warp
  }
  if (((left >> lane) & 1u) && digit != 0xffffffffu) atomicAdd(&hist[digit], 1);
}

// Adds eight digits per lane (0xffffffff = none) to a shared-memory histogram.  A lane first counts
// how many of its own digits equal its first live one (the leading digits of a selection put
// almost every key of a CTA into two or three bins: one add per key on those words would
// serialise the CTA).  Then, as in count_digits, the first digit of the lowest lane and that of
// the lowest lane left are added with one vote, one warp sum and one add each; the lanes left
// after that add their own count, and the digits that differ from a lane's first go in one by
// one.
__device__ __forceinline__ void count_digits8(int* hist, const unsigned (&dg)[8], const int lane) {
  unsigned d0 = 0xffffffffu;
#pragma unroll
  for (int e = 0; e < 8; ++e)
    if (d0 == 0xffffffffu) d0 = dg[e];
  int c0 = 0;
#pragma unroll
  for (int e = 0; e < 8; ++e) c0 += (dg[e] == d0);
  unsigned left = 0xffffffffu;
#pragma unroll
  for (int round = 0; round < 2; ++round) {
    const int src = __ffs(left) - 1;                       // lowest lane not counted yet
    const unsigned d = __shfl_sync(0xffffffffu, d0, src);
    const bool mine = d0 == d && ((left >> lane) & 1u);
    const unsigned same = __ballot_sync(0xffffffffu, mine);
    const int tot = __reduce_add_sync(0xffffffffu, mine ? c0 : 0);
    if (lane == src && d != 0xffffffffu) atomicAdd(&hist[d], tot);
    left &= ~same;
    if (left == 0) break;                                  // uniform across the warp
  }
  if (((left >> lane) & 1u) && d0 != 0xffffffffu) atomicAdd(&hist[d0], c0);
#pragma unroll
  for (int e = 0; e < 8; ++e)
    if (dg[e] != 0xffffffffu && dg[e] != d0) atomicAdd(&hist[dg[e]], 1);
}

// Threshold of the `want` largest keys of a set spread over the CTAs of a cluster (one CTA: a
// cluster of one): the want-th largest key and how many keys equal to it are still needed.  All
// threads of all CTAs take part; key_at(e), e < total, gives the keys of this CTA (any order).
// A first sweep finds the smallest and the largest key: the bits they share are the same in
// every key and are skipped, so the first digit pass already sees digits that differ (scores of
// one sequence share sign and most of the exponent; counting those bits would send every warp
// to the same one or two bins).  Then digit passes of up to 8 bits, most significant first:
// every CTA counts its keys, the histograms are added up through distributed shared memory
// after a cluster barrier and every CTA finds the digit itself.  The first pass leaves one bin
// to search; when its keys fit `list` (list_cap entries of shared memory) the second pass
// copies this CTA's share of them there while it counts, and the later passes read the list
// instead of all keys.  hist: 2 x 256 ints of shared memory, zeroed here.  Returns through
// tau / need_eq (same in every thread of the cluster).
template <typename KeyAt>
__device__ __forceinline__ void radix_threshold(const KeyAt& key_at, const int total, const int want,
                                                cg::cluster_group& cluster, int (*hist)[256],
                                                unsigned* list, const int list_cap, unsigned* tau,
                                                int* need_eq) {
  __shared__ unsigned s_prefix, s_lo[32], s_hi[32], s_range[2];
  __shared__ int s_remaining, s_cand, s_fill, htot[256];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  const int cs = (int)cluster.num_blocks();
  for (int t = threadIdx.x; t < 512; t += blockDim.x) hist[t >> 8][t & 255] = 0;
  unsigned lo = 0xffffffffu, hi = 0u;
  for (int e = threadIdx.x; e < total; e += blockDim.x) {
    const unsigned key = key_at(e);
    lo = min(lo, key);
    hi = max(hi, key);
  }
  lo = __reduce_min_sync(0xffffffffu, lo);
  hi = __reduce_max_sync(0xffffffffu, hi);
  if (lane == 0) s_lo[warp] = lo, s_hi[warp] = hi;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 0; w < nwarps; ++w) lo = min(lo, s_lo[w]), hi = max(hi, s_hi[w]);
    s_range[0] = lo, s_range[1] = hi;
  }
  cluster.sync();
  lo = 0xffffffffu, hi = 0u;
  for (int r = 0; r < cs; ++r) {
    const unsigned* rr = cluster.map_shared_rank(&s_range[0], r);
    lo = min(lo, rr[0]);
    hi = max(hi, rr[1]);
  }
  const unsigned diff = lo ^ hi;
  int top = (hi >= lo && diff) ? 32 - __clz(diff) : 0;   // the low `top` bits differ between keys
  unsigned mask = top == 32 ? 0u : ~((1u << top) - 1u);
  unsigned prefix = hi & mask;
  int remaining = want;
  int n_list = -1;        // >= 0: this CTA's candidates are in `list`
  bool build = false;     // this pass copies the candidates to `list`
  for (int pass = 0; top > 0; ++pass) {
    const int bits = min(8, top), shift = top - bits, buf = pass & 1;
    const unsigned dmask = (1u << bits) - 1u;
    if (threadIdx.x == 0) s_prefix = prefix, s_remaining = remaining, s_cand = 0, s_fill = 0;
    __syncthreads();
    if (n_list >= 0) {
      for (int e0 = 0; e0 < n_list; e0 += blockDim.x) {   // uniform trip count: full-warp votes
        const int e = e0 + threadIdx.x;
        unsigned digit = 0xffffffffu;
        if (e < n_list) {
          const unsigned key = list[e];
          if ((key & mask) == prefix) digit = (key >> shift) & dmask;
        }
        count_digits(hist[buf], digit, lane);
      }
    } else {
      for (int e0 = 0; e0 < total; e0 += blockDim.x) {   // uniform trip count: full-warp votes
        const int e = e0 + threadIdx.x;
        unsigned digit = 0xffffffffu, key = 0u;
        if (e < total) {
          key = key_at(e);
          if ((key & mask) == prefix) digit = (key >> shift) & dmask;
        }
        count_digits(hist[buf], digit, lane);
        if (build) {   // one shared-memory add per warp reserves the slots of its candidates
          const unsigned m = __ballot_sync(0xffffffffu, digit != 0xffffffffu);
          if (m) {
            const int leader = __ffs(m) - 1;
            int base = 0;
            if (lane == leader) base = atomicAdd(&s_fill, __popc(m));
            base = __shfl_sync(0xffffffffu, base, leader);
            if (digit != 0xffffffffu) list[base + __popc(m & ((1u << lane) - 1u))] = key;
          }
        }
      }
    }
    cluster.sync();
    if (threadIdx.x < 256) {
      int tot = 0;
      for (int r = 0; r < cs; ++r) tot += *cluster.map_shared_rank(&hist[buf][threadIdx.x], r);
      htot[threadIdx.x] = tot;
      hist[buf ^ 1][threadIdx.x] = 0;   // every CTA is past its reads of the other buffer
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      // lane l owns bins 8l .. 8l+7; `above` = keys in higher bins
      int h8[8], mine = 0;
#pragma unroll
      for (int k = 0; k < 8; ++k) h8[k] = htot[8 * lane + k], mine += h8[k];
      // suffix sum over lanes: keys in the bins of higher lanes
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_down_sync(0xffffffffu, incl, o);
        if (lane + o < 32) incl += v;
      }
      int above = incl - mine;
#pragma unroll
      for (int k = 7; k >= 0; --k) {
        if (above < remaining && remaining <= above + h8[k]) {
          s_prefix = prefix | ((unsigned)(8 * lane + k) << shift);
          s_remaining = remaining - above;
          s_cand = h8[k];
        }
        above += h8[k];
      }
    }
    __syncthreads();
    prefix = s_prefix;
    remaining = s_remaining;
    mask |= dmask << shift;
    top = shift;
    if (build) {
      n_list = s_fill;   // the list holds this CTA's keys under the prefix before this pass; the
      build = false;     // next passes narrow the prefix inside it
    } else if (n_list < 0 && pass == 0 && s_cand <= list_cap) {
      build = true;
    }
    __syncthreads();
  }
  *tau = prefix;
  *need_eq = remaining;
}

constexpr int kBudgetCluster = 8;

// Head budgets of one sequence under the adaptive rule (see mixkv.h).  One CTA per (sequence,
// layer) when the call has many of them, else a cluster of kBudgetCluster CTAs, each with a
// slice of the positions of every head.  A CTA turns its H * n pooled scores into
// order-preserving keys once and keeps them in shared memory when they fit (cache_cap keys);
// otherwise every pass reads them from global memory.
__global__ void __launch_bounds__(1024)
k_budget(const SeqTable st, const float* __restrict__ scores, int* __restrict__ counts,
         const int Bp, const int floor_slots, const int cache_cap, const int list_cap) {
  extern __shared__ unsigned bkeys[];   // [cache_cap] keys, then [list_cap] candidates
  __shared__ int hist[2][256];
  __shared__ int s_gt[64], s_eq[64], t_gt[64], t_eq[64];
  cg::cluster_group cluster = cg::this_cluster();
  const int cs = (int)cluster.num_blocks(), crank = (int)cluster.block_rank();
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x / cs, layer = blockIdx.y, H = st.H;
  counts += (size_t)layer * st.batch * H;
  const int P = st.cu[b + 1] - st.cu[b] - st.W;
  const long long total = (long long)H * P;
  long long N = (long long)H * (Bp - floor_slots);
  if (N > total) N = total;
  const float* base = scores + ppos(st, layer, 0, b, 0);
  const size_t stride = (size_t)st.Ptot;
  if (N <= 0) {   // the same in every CTA of the cluster
    if (crank == 0)
      for (int h = threadIdx.x; h < H; h += blockDim.x) counts[b * H + h] = min(floor_slots, P);
    return;
  }
  // this CTA's slice of every head: positions [p0, p0 + n)
  const int chunk = (P + cs - 1) / cs;
  const int p0 = min(crank * chunk, P), n = min(chunk, P - p0);
  const int local = H * n;
  const bool cached = local <= cache_cap;
  if (cached) {
    for (int h = 0; h < H; ++h) {
      const float* row = base + (size_t)h * stride + p0;
      for (int i0 = 0; i0 < n; i0 += 8 * blockDim.x) {   // eight loads in flight per thread
        float v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int i = i0 + k * blockDim.x + threadIdx.x;
          v[k] = i < n ? row[i] : 0.f;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int i = i0 + k * blockDim.x + threadIdx.x;
          if (i < n) bkeys[h * n + i] = order_key(v[k]);
        }
      }
    }
    __syncthreads();
  }
  auto key_at = [&](const int e) -> unsigned {
    if (cached) return bkeys[e];
    const int h = e / n;
    return order_key(base[(size_t)h * stride + p0 + (e - h * n)]);
  };
  unsigned tau;
  int need_eq;
  radix_threshold(key_at, local, (int)N, cluster, hist, bkeys + cache_cap, list_cap, &tau, &need_eq);
  for (int h = threadIdx.x; h < H; h += blockDim.x) s_gt[h] = 0, s_eq[h] = 0;
  __syncthreads();
  for (int h = 0; h < H; ++h) {
    int gt = 0, eq = 0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      const unsigned key = key_at(h * n + i);
      gt += key > tau;
      eq += key == tau;
    }
    for (int o = 16; o > 0; o >>= 1) {
      gt += __shfl_xor_sync(0xffffffffu, gt, o);
      eq += __shfl_xor_sync(0xffffffffu, eq, o);
    }
    if ((threadIdx.x & 31) == 0) {
      atomicAdd(&s_gt[h], gt);
      atomicAdd(&s_eq[h], eq);
    }
  }
  cluster.sync();   // every CTA's per-head counts are complete
  if (crank == 0) {
    for (int h = threadIdx.x; h < H; h += blockDim.x) {
      int g = 0, q = 0;
      for (int r = 0; r < cs; ++r) {
        g += *cluster.map_shared_rank(&s_gt[h], r);
        q += *cluster.map_shared_rank(&s_eq[h], r);
      }
      t_gt[h] = g, t_eq[h] = q;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int rem = need_eq;  // equal-to-threshold elements go to the lower (head, position) first
      for (int h = 0; h < H; ++h) {
        const int take = min(t_eq[h], rem);
        rem -= take;
        counts[b * H + h] = min(floor_slots + t_gt[h] + take, P);
      }
    }
  }
  cluster.sync();   // the peers' shared memory stays alive until rank 0 has read it
}

// ------------------------------------------------------------------------------ tail
constexpr int kTailCluster = 8;
constexpr int kTailThreads = 512;
constexpr int kTailCacheCap = 16384;       // positions a CTA of a cluster keeps in shared memory
constexpr int kTailCacheCapSolo = 40960;   // positions a CTA that owns a whole head keeps
constexpr int kTailListCap = 2048;         // keys of the threshold bin a lone CTA lists after two digits

struct TailKernelArgs {
  const float* scores;        // select on these (FUSED == false)
  const float* s_div;         // FUSED: parts of the mix
  const float* rbar_in;
  float* s_comp_out;          // FUSED: mixed scores are written here
  const int* counts_dev;      // adaptive budgets; nullptr = fixed
  int* counts_out;
  int* idx;
  int* idx_offsets;
  int* out_row_offsets;       // may be nullptr
  const __nv_bfloat16* K;     // gather when K_out != nullptr
  const __nv_bfloat16* V;
  __nv_bfloat16* K_out;
  __nv_bfloat16* V_out;
  int Bp;                     // B - W
  int cached;                 // keys of the slice fit the shared-memory cache
  long long kv_layer_stride;  // elements between consecutive layers of K (V)
  int idx_cap;                // index-list entries reserved per layer
  int out_rows_cap;           // output rows reserved per layer
  MixParams mp;
};

// Selected rows of (b', h') pairs before bh, fixed budgets.
__device__ __forceinline__ int fixed_offset(const SeqTable& st, int bh, int Bp) {
  const int b = bh / st.H, h = bh % st.H;
  int off = 0;
  for (int x = 0; x < b; ++x) off += st.H * min(Bp, st.cu[x + 1] - st.cu[x] - st.W);
  if (b < st.batch) off += h * min(Bp, st.cu[b + 1] - st.cu[b] - st.W);
  return off;
}

// Shared-memory slot of local position j: one pad word per 32 keeps both the strided walk
// (thread t, t + 512, ...) and the contiguous runs of the compaction free of bank conflicts.
__device__ __forceinline__ int kslot(int j) { return j + (j >> 5); }

// T threads per CTA; the cluster size (1 or kTailCluster CTAs per (layer, sequence, head)) is read
// from the launch: many independent heads fill the GPU with one CTA each and need no cluster
// traffic at all, a call with few heads spreads each head over a cluster.
template <bool FUSED, int T>
__global__ void __launch_bounds__(T, T == 512 ? 2 : 1)
k_tail(const SeqTable st, const Workspace ws, const TailKernelArgs a) {
  extern __shared__ __align__(16) unsigned char tail_smem[];
  __shared__ int hist[2][256];
  __shared__ int s_scan[32][2];
  __shared__ __align__(8) int s_tot[2];
  __shared__ int s_sel[3];      // digit, remaining, keys in the digit's bin
  __shared__ int s_nlist;
  __shared__ int s_off;
  __shared__ float sc[8];
  cg::cluster_group cluster = cg::this_cluster();
  const int crank = (int)cluster.block_rank();
  const int cs = (int)cluster.num_blocks();
  const int BH = st.batch * st.H;
  const int unit = blockIdx.x / cs;                    // (layer, sequence, head)
  const int layer = unit / BH, bh = unit % BH, b = bh / st.H, h = bh % st.H;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int W = st.W;
  const int P = st.cu[b + 1] - st.cu[b] - W;
  const size_t poff = ppos(st, layer, h, b, 0);
  // this layer's slices of the per-layer arrays
  const int* counts_dev = a.counts_dev ? a.counts_dev + (size_t)layer * BH : nullptr;
  int* counts_out = a.counts_out ? a.counts_out + (size_t)layer * BH : nullptr;
  int* idx_offsets = a.idx_offsets + (size_t)layer * (BH + 1);
  int* out_row_offsets = a.out_row_offsets ? a.out_row_offsets + (size_t)layer * (BH + 1) : nullptr;
  // slice of this CTA: positions [c0, c0 + n)
  const int chunk = (P + cs - 1) / cs;
  const int R = (chunk + T - 1) / T;   // positions per thread
  const int c0 = min(crank * chunk, P);
  const int n = min(chunk, P - c0);
  unsigned* skeys = reinterpret_cast<unsigned*>(tail_smem);            // [kslot(chunk) + 1]
  float* sraw = reinterpret_cast<float*>(skeys + kslot(chunk) + 1);    // FUSED: [8 T + 64] stage; else [kTailListCap]

  pdl_launch_dependents();
  pdl_wait();

  // ---- budget and output offsets of this (b, h)
  if (tid < 32) {
    int off = 0, cnt;
    if (counts_dev) {
      for (int t = lane; t < bh; t += 32) off += counts_dev[t];
      for (int o = 16; o > 0; o >>= 1) off += __shfl_xor_sync(0xffffffffu, off, o);
      cnt = counts_dev[bh];
    } else {
      off = fixed_offset(st, bh, a.Bp);
      cnt = min(a.Bp, P);
    }
    if (lane == 0) {
      s_off = off;
      s_nlist = 0;
      s_sel[1] = cnt;
      if (crank == 0) {
        idx_offsets[bh] = off;
        if (counts_out) counts_out[bh] = cnt;
        if (out_row_offsets) out_row_offsets[bh] = off + bh * W;
        if (bh == BH - 1) {
          idx_offsets[BH] = off + cnt;
          if (out_row_offsets) out_row_offsets[BH] = off + cnt + BH * W;
        }
      }
    }
  }
  for (int t = tid; t < 256; t += T) hist[0][t] = 0;   // visible after the next CTA barrier
  const float* src = a.scores;
  const bool cached = FUSED || a.cached;
  float held[8];   // FUSED, R <= 8: mixed scores kept until the selection is done
  if (FUSED) {
    // ---- pooling and mix of this slice (Eq. 2, Eq. 5) in blocks of 8 T consecutive positions:
    // thread t takes positions t, t + T, ... of the block
    const int half = a.mp.pool_k >> 1;
    const bool avg = a.mp.pool_mode == MIXKV_POOL_AVG;
    const float pad = avg ? 0.f : -INFINITY;
    const float invk = 1.0f / (float)a.mp.pool_k;
    if (warp == 1)
      head_scalars(st, ws, layer, b, h, a.mp.pool_k, a.mp.pool_mode, a.mp.use_vnorm, a.mp.eps,
                   a.rbar_in, lane, sc);
    // The block and its pooling halo (62 positions at most) are nine rounds of T raw scores.
    // They are loaded one block ahead: the raw scores of block b + 1 fly while block b is pooled
    // and mixed, and the two per-position terms of a block are asked for before its pooling and
    // used after it.
    float raw[9];
    auto load_raw = [&](const int j0) {
      const int nstage = min(8 * T, n - j0) + 2 * half;
#pragma unroll
      for (int e = 0; e < 9; ++e) {
        const int t = e * T + tid, i = c0 + j0 - half + t;
        raw[e] = (j0 < n && t < nstage && i >= 0 && i < P) ? ws.s_ex_raw[poff + i] : pad;
      }
    };
    load_raw(0);
    for (int j0 = 0; j0 < n; j0 += 8 * T) {
      const int nb = min(8 * T, n - j0);   // positions of this block
      float vn[8], dv[8];
      const int nstage = nb + 2 * half;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int jb = e * T + tid;
        vn[e] = (a.mp.use_vnorm && jb < nb) ? ws.vnorm[poff + c0 + j0 + jb] : 0.f;
        dv[e] = jb < nb ? a.s_div[poff + c0 + j0 + jb] : 0.f;
      }
      __syncthreads();                     // the previous block's readers of sraw are done
#pragma unroll
      for (int e = 0; e < 9; ++e) {
        const int t = e * T + tid;
        if (t < nstage) sraw[t] = raw[e];
      }
      load_raw(j0 + 8 * T);
      __syncthreads();
      // the eight pooling windows advance together (same order of additions as pool_window),
      // so their shared-memory loads overlap instead of forming eight serial chains
      float ex[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) ex[e] = avg ? 0.f : -INFINITY;
      for (int u = 0; u < a.mp.pool_k; ++u) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int jb = min(e * T + tid, nb - 1);
          const float w = sraw[jb + u];
          ex[e] = avg ? ex[e] + w : fmaxf(ex[e], w);
        }
      }
      unsigned top[8];   // leading digit of the block's keys: the first digit pass, taken here
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int jb = e * T + tid;
        held[e] = 0.f;
        top[e] = 0xffffffffu;
        if (jb < nb) {
          held[e] = mix_one(avg ? ex[e] * invk : ex[e], vn[e], dv[e], sc, a.mp.use_vnorm,
                            a.mp.mix_mode);
          const unsigned key = order_key(held[e]);
          skeys[kslot(j0 + jb)] = key;
          top[e] = key >> 24;
          if (R > 8) a.s_comp_out[poff + c0 + j0 + jb] = held[e];
        }
      }
      count_digits8(hist[0], top, lane);
    }
    src = a.s_comp_out;
  } else if (a.cached) {
    for (int j = tid; j < n; j += T) skeys[kslot(j)] = order_key(src[poff + c0 + j]);
  }
  __syncthreads();
  const int want = s_sel[1];
  int* out = a.idx + (size_t)layer * a.idx_cap + s_off;
  auto key_at = [&](int j) -> unsigned {
    return cached ? skeys[kslot(j)] : order_key(src[poff + c0 + j]);
  };

  bool all = false;
  unsigned tau = 0;
  int need_eq = 0;
  if (want >= P) {
    all = true;     // keep every candidate
  } else if (want > 0) {
    // ---- threshold: the want-th largest key of the head, four 8-bit digit passes
    unsigned prefix = 0, mask = 0;
    int remaining = want;
    // up to eight keys per thread stay in registers for the four passes; their votes are
    // independent, so the eight chains of a pass overlap
    const bool inreg = cached && R <= 8;
    unsigned rk[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int j = e * T + tid;
      rk[e] = (inreg && j < n) ? skeys[kslot(j)] : 0u;
    }
    auto count_digit = [&](const unsigned digit, const int buf) {
      count_digits(hist[buf], digit, lane);
    };
    // Threads 0..255 bring the number of keys in their bin: the bin that holds the left-th
    // largest key goes to s_sel[0], how many keys are still needed from inside it to s_sel[1],
    // its size to s_sel[2].  All threads call it; it ends on a CTA barrier.
    auto find_digit = [&](const int tot, const int left) {
      int incl = tot;   // suffix sums over the 256 bins: this bin and those above it
      if (tid < 256) {
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_down_sync(0xffffffffu, incl, o);
          if (lane + o < 32) incl += v;
        }
        if (lane == 0) s_scan[warp][0] = incl;
      }
      __syncthreads();
      if (tid < 256) {
        int above = incl - tot;
        for (int w = warp + 1; w < 8; ++w) above += s_scan[w][0];
        if (above < left && left <= above + tot) {
          s_sel[0] = tid;
          s_sel[1] = left - above;
          s_sel[2] = tot;
        }
      }
      __syncthreads();
    };
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass, buf = pass & 1;
      if (FUSED && pass == 0) {
        // the leading digits were counted while the keys were made
      } else if (inreg) {
        unsigned dg[8];
#pragma unroll
        for (int e = 0; e < 8; ++e)
          dg[e] = (e * T + tid < n && (rk[e] & mask) == prefix) ? (rk[e] >> shift) & 255u
                                                                : 0xffffffffu;
        if (R > 4) {   // R is the same in every thread
          count_digits8(hist[buf], dg, lane);
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (e < R) count_digit(dg[e], buf);
        }
      } else {
        for (int e0 = 0; e0 < R; e0 += 8) {   // same trip count in every lane: full-warp votes
          unsigned dg[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const int j = (e0 + e) * T + tid;
            dg[e] = 0xffffffffu;
            if (e0 + e < R && j < n) {
              const unsigned key = key_at(j);
              if ((key & mask) == prefix) dg[e] = (key >> shift) & 255u;
            }
          }
          count_digits8(hist[buf], dg, lane);
        }
      }
      cluster.sync();
      // every CTA adds up the cluster's histograms and finds the digit itself
      int tot = 0;
      if (tid < 256) {
        int part[kTailCluster];
#pragma unroll
        for (int r = 0; r < kTailCluster; ++r)
          part[r] = r < cs ? *cluster.map_shared_rank(&hist[buf][tid], r) : 0;
#pragma unroll
        for (int r = 0; r < kTailCluster; ++r) tot += part[r];
        hist[buf ^ 1][tid] = 0;   // every CTA is past its reads of the other buffer
      }
      find_digit(tot, remaining);
      prefix |= (unsigned)s_sel[0] << shift;
      remaining = s_sel[1];
      mask |= 255u << shift;
      // A CTA that owns a whole head and keeps its keys in shared memory: two digits fix sign,
      // exponent and seven mantissa bits, and the bin that holds the threshold is small.  Its
      // keys (their low 16 bits) go to a list and the last two digits are searched there, two
      // sweeps over a few hundred entries instead of two over all keys.  (With a cluster the
      // sweeps are short already and a list costs as much as the two histogram exchanges.)
      if (cs == 1 && pass == 1 && !inreg && cached && s_sel[2] <= kTailListCap) {
        unsigned* list = reinterpret_cast<unsigned*>(sraw);   // after the keys; the pooling stage is free by now
        for (int e = 0; e < R; ++e) {
          const int j = e * T + tid;
          if (j < n) {
            const unsigned key = skeys[kslot(j)];
            if ((key & mask) == prefix) list[atomicAdd(&s_nlist, 1)] = key & 0xffffu;
          }
        }
        if (tid < 256) hist[1][tid] = 0;   // hist[0] is zero already
        __syncthreads();
        const int nl = s_nlist;
        for (int e = tid; e < nl; e += T) atomicAdd(&hist[0][(list[e] >> 8) & 255u], 1);
        __syncthreads();
        find_digit(tid < 256 ? hist[0][tid] : 0, remaining);
        const unsigned hi8 = (unsigned)s_sel[0];
        remaining = s_sel[1];
        for (int e = tid; e < nl; e += T)
          if (((list[e] >> 8) & 255u) == hi8) atomicAdd(&hist[1][list[e] & 255u], 1);
        __syncthreads();
        find_digit(tid < 256 ? hist[1][tid] : 0, remaining);
        prefix |= (hi8 << 8) | (unsigned)s_sel[0];
        remaining = s_sel[1];
        break;
      }
    }
    tau = prefix;
    need_eq = remaining;
  }

  // ---- ordered compaction: thread t owns the run [t*R, (t+1)*R) of the slice; it keeps the
  // positions with key > tau, plus the first need_eq (in position order) with key == tau
  if (want > 0) {
    const int r0 = min(tid * R, n), r1 = min(r0 + R, n);
    int gt = 0, eq = 0;
    if (all) {
      gt = r1 - r0;
    } else {
      for (int j = r0; j < r1; ++j) {
        const unsigned key = key_at(j);
        gt += key > tau;
        eq += key == tau;
      }
    }
    int gt_inc = gt, eq_inc = eq;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, gt_inc, o);
      const int y = __shfl_up_sync(0xffffffffu, eq_inc, o);
      if (lane >= o) gt_inc += x, eq_inc += y;
    }
    __syncthreads();   // the threshold search is done with s_scan
    if (lane == 31) s_scan[warp][0] = gt_inc, s_scan[warp][1] = eq_inc;
    __syncthreads();
    int gt_before = gt_inc - gt, eq_before = eq_inc - eq;
    for (int w = 0; w < warp; ++w) gt_before += s_scan[w][0], eq_before += s_scan[w][1];
    if (tid == T - 1) {
      s_tot[0] = gt_before + gt;
      s_tot[1] = eq_before + eq;
    }
    cluster.sync();
    {
      int2 before[kTailCluster];
#pragma unroll
      for (int r = 0; r < kTailCluster; ++r)
        before[r] = r < crank ? *reinterpret_cast<const int2*>(cluster.map_shared_rank(&s_tot[0], r))
                              : make_int2(0, 0);
#pragma unroll
      for (int r = 0; r < kTailCluster; ++r) gt_before += before[r].x, eq_before += before[r].y;
    }
    // most runs hold no kept position at all: their second walk is skipped
    const bool writes = all || gt > 0 || (eq > 0 && eq_before < need_eq);
    for (int j = r0; writes && j < r1; ++j) {
      const int i = c0 + j;
      if (all) {
        out[gt_before++] = i;
        continue;
      }
      const unsigned key = key_at(j);
      if (key > tau) {
        out[gt_before + min(eq_before, need_eq)] = i;
        ++gt_before;
      } else if (key == tau) {
        if (eq_before < need_eq) out[gt_before + eq_before] = i;
        ++eq_before;
      }
    }
  }
  // the index list is complete (and visible to the cluster) after this barrier; it also keeps
  // every CTA's shared memory alive until its peers have read it
  cluster.sync();
  if (FUSED && R <= 8) {
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int j = e * T + tid;
      if (j < n) a.s_comp_out[poff + c0 + j] = held[e];
    }
  }

  // ---- gather: selected rows in ascending position order, then the W window rows
  if (a.K_out) {
    const int n_sel = max(want, 0) < P ? max(want, 0) : P;
    const int rows = n_sel + W;
    const __nv_bfloat16* Ksrc = a.K + (size_t)layer * a.kv_layer_stride;
    const __nv_bfloat16* Vsrc = a.V + (size_t)layer * a.kv_layer_stride;
    const size_t srow0 = (size_t)h * st.Ltot + st.cu[b];
    const size_t drow0 = (size_t)layer * a.out_rows_cap + (size_t)(s_off + bh * W);
    const int hw = tid >> 4, l = tid & 15;                       // half-warps, 16 B per lane
    const int rows_per_sweep = cs * (T / 16);
    for (int rb = crank * (T / 16) + hw; rb < rows; rb += 2 * rows_per_sweep) {
      const int ra = rb + rows_per_sweep;
      const int sa = rb < n_sel ? __ldcg(out + rb) : P + (rb - n_sel);
      const int sb = ra < rows ? (ra < n_sel ? __ldcg(out + ra) : P + (ra - n_sel)) : -1;
      const uint4 k0 = __ldg(reinterpret_cast<const uint4*>(Ksrc + (srow0 + sa) * kHeadDim) + l);
      const uint4 v0 = __ldg(reinterpret_cast<const uint4*>(Vsrc + (srow0 + sa) * kHeadDim) + l);
      uint4 k1 = make_uint4(0, 0, 0, 0), v1 = k1;
      if (sb >= 0) {
        k1 = __ldg(reinterpret_cast<const uint4*>(Ksrc + (srow0 + sb) * kHeadDim) + l);
        v1 = __ldg(reinterpret_cast<const uint4*>(Vsrc + (srow0 + sb) * kHeadDim) + l);
      }
      reinterpret_cast<uint4*>(a.K_out + (drow0 + rb) * kHeadDim)[l] = k0;
      reinterpret_cast<uint4*>(a.V_out + (drow0 + rb) * kHeadDim)[l] = v0;
      if (sb >= 0) {
        reinterpret_cast<uint4*>(a.K_out + (drow0 + ra) * kHeadDim)[l] = k1;
        reinterpret_cast<uint4*>(a.V_out + (drow0 + ra) * kHeadDim)[l] = v1;
      }
    }
  }
}

int floor_slots(const mixkv_params& p) {
  const int Bp = p.budget - p.window;
  int f = (int)floor((double)p.ada_floor * (double)Bp);
  if (f > Bp) f = Bp;
  if (f < 0) f = 0;
  return f;
}

MixParams mix_params(const mixkv_params& p) {
  MixParams mp;
  mp.pool_k = p.pool_kernel;
  mp.pool_mode = p.pool_mode;
  mp.use_vnorm = p.use_vnorm;
  mp.mix_mode = p.mix_mode;
  mp.eps = p.eps;
  return mp;
}

}  // namespace

cudaError_t launch_poolsum(const LaunchCtx& c) {
  return launch_pdl(k_poolsum, dim3(c.st.pchunks_total, c.st.H, c.st.layers), dim3(256), 0,
                    c.stream, 1, c.st,
                    c.ws, c.p.pool_kernel);
}

cudaError_t launch_mixpool(const LaunchCtx& c, const float* s_div, const float* rbar_in,
                           float* s_ex_out, float* s_comp) {
  return launch_pdl(k_mixpool, dim3(c.st.pchunks_total, c.st.H, c.st.layers), dim3(256), 0,
                    c.stream, 1, c.st,
                    c.ws, s_div, rbar_in, s_ex_out, s_comp, mix_params(c.p));
}

// Budgets chosen by the caller (rows to keep per (layer, sequence, head), window included) ->
// candidates to select: minus the window, at least 0, at most B - W and the candidates there are.
__global__ void __launch_bounds__(256)
k_given_budgets(const SeqTable st, const int* __restrict__ budgets, int* __restrict__ counts,
                const int Bp) {
  pdl_launch_dependents();
  pdl_wait();
  const int layer = blockIdx.x, BH = st.batch * st.H;
  for (int t = threadIdx.x; t < BH; t += blockDim.x) {
    const int b = t / st.H;
    const int P = st.cu[b + 1] - st.cu[b] - st.W;
    const int c = budgets[(size_t)layer * BH + t] - st.W;
    counts[(size_t)layer * BH + t] = max(0, min(c, min(Bp, P)));
  }
}

cudaError_t launch_given_budgets(const LaunchCtx& c, const int* budgets, int* counts) {
  return launch_pdl(k_given_budgets, dim3(c.st.layers), dim3(256), 0, c.stream, 1, c.st, budgets,
                    counts, c.p.budget - c.p.window);
}

cudaError_t launch_budget(const LaunchCtx& c, const float* scores, int* counts) {
  // few (sequence, layer) pairs: a cluster of CTAs each; many: one CTA each
  const int cs = c.st.batch * c.st.layers < device_sm_count() / kBudgetCluster ? kBudgetCluster : 1;
  const size_t chunk = ((size_t)c.max_prefix + cs - 1) / cs;
  // the keys of a CTA's slice of the longest sequence in shared memory when they fit
  const size_t want = (size_t)c.st.H * chunk * 4;
  const size_t cap_bytes = 200 * 1024;
  const size_t key_bytes = want <= cap_bytes - 16 * 1024 ? want : 0;
  // the rest, up to 16 K entries, holds the candidates left after the first digit pass
  size_t list_bytes = cap_bytes - key_bytes;
  if (list_bytes > 64 * 1024) list_bytes = 64 * 1024;
  if (list_bytes > want) list_bytes = want;
  const size_t smem = key_bytes + list_bytes;
  if (smem > 48 * 1024) {
    static bool done[64] = {false};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !done[dev]) {
      e = cudaFuncSetAttribute(k_budget, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)cap_bytes);
      if (e != cudaSuccess) return e;
      if (dev >= 0 && dev < 64) done[dev] = true;
    }
  }
  return launch_pdl(k_budget, dim3(c.st.batch * cs, c.st.layers), dim3(1024), smem, c.stream, cs,
                    c.st, scores, counts, c.p.budget - c.p.window, floor_slots(c.p),
                    (int)(key_bytes / 4), (int)(list_bytes / 4));
}

// Launch shape of k_tail: many (layer, sequence, head) units -> one 1024-thread CTA each; few ->
// a cluster of kTailCluster 512-thread CTAs each.  Returns false when the keys of a slice do not
// fit the shared-memory cache under either shape.
struct TailShape {
  int cs, threads, chunk;
  bool cached;
};

TailShape tail_shape(const LaunchCtx& c) {
  const int units = c.st.layers * c.st.batch * c.st.H;
  TailShape t;
  t.cs = 1, t.threads = 1024, t.chunk = c.max_prefix;
  if (units >= device_sm_count() / 2 && t.chunk <= kTailCacheCapSolo) {
    t.cached = true;
    return t;
  }
  t.cs = kTailCluster, t.threads = kTailThreads;
  t.chunk = (c.max_prefix + kTailCluster - 1) / kTailCluster;
  t.cached = t.chunk <= kTailCacheCap;
  return t;
}

bool tail_can_fuse(const LaunchCtx& c) { return tail_shape(c).cached; }

template <bool FUSED, int T>
cudaError_t launch_tail_t(const LaunchCtx& c, const TailKernelArgs& a, const TailShape& sh,
                          size_t smem) {
  static size_t have[64] = {0};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (smem > 48 * 1024 && (dev < 0 || dev >= 64 || have[dev] < smem)) {
    const size_t ask = 216 * 1024;
    e = cudaFuncSetAttribute(k_tail<FUSED, T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)ask);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) have[dev] = ask;
  }
  const dim3 grid(c.st.layers * c.st.batch * c.st.H * sh.cs);
  return launch_pdl(k_tail<FUSED, T>, grid, dim3(T), smem, c.stream, sh.cs, c.st, c.ws, a);
}

cudaError_t launch_tail(const LaunchCtx& c, const TailArgs& t) {
  TailKernelArgs a;
  a.scores = t.scores;
  a.s_div = t.s_div;
  a.rbar_in = t.rbar_in;
  a.s_comp_out = t.s_comp_out;
  a.counts_dev = t.counts_dev;
  a.counts_out = t.counts_out;
  a.idx = t.idx;
  a.idx_offsets = t.idx_offsets;
  a.out_row_offsets = t.out_row_offsets;
  a.K = (const __nv_bfloat16*)t.K;
  a.V = (const __nv_bfloat16*)t.V;
  a.K_out = (__nv_bfloat16*)t.K_out;
  a.V_out = (__nv_bfloat16*)t.V_out;
  a.Bp = c.p.budget - c.p.window;
  a.kv_layer_stride = c.kv_layer_stride;
  a.idx_cap = c.idx_cap;
  a.out_rows_cap = c.out_rows_cap;
  a.mp = mix_params(c.p);
  const TailShape sh = tail_shape(c);
  const bool fused = t.scores == nullptr;
  a.cached = sh.cached ? 1 : 0;
  if (fused && !a.cached) return cudaErrorInvalidValue;   // callers check tail_can_fuse() first
  size_t smem = 0;
  if (a.cached) smem += ((size_t)sh.chunk + (sh.chunk >> 5) + 1) * 4;
  if (fused) smem += ((size_t)8 * sh.threads + 64) * 4;          // pooling stage, later the key list
  else if (a.cached) smem += (size_t)kTailListCap * 4;           // key list of a lone CTA
  if (sh.threads == 1024)
    return fused ? launch_tail_t<true, 1024>(c, a, sh, smem) : launch_tail_t<false, 1024>(c, a, sh, smem);
  return fused ? launch_tail_t<true, 512>(c, a, sh, smem) : launch_tail_t<false, 512>(c, a, sh, smem);
}

}  // namespace mixkv
