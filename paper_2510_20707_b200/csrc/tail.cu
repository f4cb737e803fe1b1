// Everything after the two K passes: finishing the per-head statistics, pooling, the
// head-wise mix (Eq. 2, Eq. 5), budgets, per-head top-B selection and the gather
// (Algorithm 1, step 2 and the TopB line).
#include "tc_common.cuh"

namespace mixkv {

namespace {

// ----------------------------------------------------------------------------- pool
// 1-D pooling of the raw attention score over the candidate positions of one sequence,
// stride 1, half-width k/2; average pooling pads with zeros and divides by k.
__global__ void __launch_bounds__(256)
k_pool(const SeqTable st, const Workspace ws, float* __restrict__ s_ex_out, const int k,
       const int mode) {
  __shared__ float tile[kPChunk + 64];
  __shared__ float sred[8];
  const int pcx = blockIdx.x, h = blockIdx.y;
  const int b = find_seq(st.pchunk_start, st.batch, pcx);
  const int P = st.cu[b + 1] - st.cu[b] - st.W;
  const int p0 = (pcx - st.pchunk_start[b]) * kPChunk;
  const int p1 = min(p0 + kPChunk, P);
  const size_t poff = (size_t)h * st.Ptot + (st.cu[b] - b * st.W);
  const int half = k >> 1;
  const float pad = mode == 0 ? 0.f : -INFINITY;
  for (int t = threadIdx.x; t < (p1 - p0) + 2 * half; t += 256) {
    const int i = p0 - half + t;
    tile[t] = (i >= 0 && i < P) ? ws.s_ex_raw[poff + i] : pad;
  }
  __syncthreads();
  float sum = 0.f;
  const float invk = 1.0f / (float)k;
  for (int t = threadIdx.x; t < p1 - p0; t += 256) {
    float v;
    if (mode == 0) {
      v = 0.f;
      for (int u = 0; u < k; ++u) v += tile[t + u];
      v *= invk;
    } else {
      v = -INFINITY;
      for (int u = 0; u < k; ++u) v = fmaxf(v, tile[t + u]);
    }
    s_ex_out[poff + p0 + t] = v;
    sum += v;
  }
  sum = warp_sum(sum);
  if ((threadIdx.x & 31) == 0) sred[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
    for (int w = 0; w < 8; ++w) s += sred[w];
    ws.exsum[(size_t)h * st.pchunks_total + pcx] = s;
  }
}

// ------------------------------------------------------------------------------ mix
// Eq. 2 and Eq. 5.  Every CTA first rebuilds the scalars of its (sequence, head) from the
// per-chunk partials (a few dozen values), then mixes its slice.
__global__ void __launch_bounds__(256)
k_mix(const SeqTable st, const Workspace ws, const float* __restrict__ s_ex,
      const float* __restrict__ s_div, const float* __restrict__ rbar_in,
      float* __restrict__ s_comp, float* __restrict__ rbar_out, const int use_vnorm,
      const int mix_mode, const float eps) {
  __shared__ float sc[8];
  const int pcx = blockIdx.x, h = blockIdx.y;
  const int b = find_seq(st.pchunk_start, st.batch, pcx);
  const int bh = b * st.H + h;
  const int P = st.cu[b + 1] - st.cu[b] - st.W;
  const int p0 = (pcx - st.pchunk_start[b]) * kPChunk;
  const int p1 = min(p0 + kPChunk, P);
  const size_t poff = (size_t)h * st.Ptot + (st.cu[b] - b * st.W);
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    float ex = 0.f;
    for (int c = st.pchunk_start[b] + lane; c < st.pchunk_start[b + 1]; c += 32)
      ex += ws.exsum[(size_t)h * st.pchunks_total + c];
    float a = INFINITY, bb = -INFINITY, s = 0.f;
    {
      const int per_head = (st.tile2_start[b + 1] - st.tile2_start[b]) / st.H;
      const int U0 = st.tile2_start[b] + h * per_head;
      int k = 0;
      for (SegIter sg(U0, U0 + per_head, st.nt2, st.g2); sg.valid(); sg.next(), ++k) {
        if ((k & 31) == lane) {
          const float4 v = ws.dstat[sg.start];
          a = fminf(a, v.x);
          bb = fmaxf(bb, v.y);
          s += v.z;
        }
      }
    }
    ex = warp_sum(ex);
    a = warp_min(a);
    bb = warp_max(bb);
    s = warp_sum(s);
    if (lane == 0) {
      const float invP = 1.0f / (float)P;
      const float mean_ex = ex * invP;
      float vmin = 0.f, vinv = 0.f, a_in = 0.f, mean_imp = mean_ex;
      if (use_vnorm) {
        const float4 v = ws.vfinal[bh];
        vmin = v.x;
        vinv = 1.0f / (v.y - v.x + eps);
        const float mean_in = (v.z * invP - v.x) * vinv;
        a_in = mean_ex / (mean_in + eps);
        mean_imp = mean_ex + mean_in * a_in;
      }
      const float dinv = 1.0f / (bb - a + eps);
      const float mean_dn = (s * invP - a) * dinv;
      const float a_div = mean_imp / (mean_dn + eps);
      const float r = rbar_in ? rbar_in[bh] : ws.rbar[bh];
      sc[0] = vmin;
      sc[1] = vinv * a_in;     // s_in_scaled = (n - vmin) * sc[1]
      sc[2] = a;
      sc[3] = dinv * a_div;    // s_div_scaled = (s_div - dmin) * sc[3]
      sc[4] = r;
      if (rbar_out && pcx == st.pchunk_start[b]) rbar_out[bh] = ws.rbar[bh];
    }
  }
  __syncthreads();
  const float vmin = sc[0], cin = sc[1], dmin = sc[2], cdiv = sc[3], r = sc[4];
  for (int i = p0 + threadIdx.x; i < p1; i += 256) {
    const float ex = s_ex[poff + i];
    const float dv = s_div[poff + i];
    float imp = ex;
    if (use_vnorm) imp += (ws.vnorm[poff + i] - vmin) * cin;
    const float dsc = (dv - dmin) * cdiv;
    float c;
    switch (mix_mode) {
      case MIXKV_MIX_HEADWISE: c = (1.0f - r) * imp + r * dsc; break;
      case MIXKV_MIX_IMPORTANCE_ONLY: c = imp; break;
      case MIXKV_MIX_DIVERSITY_ONLY: c = dv; break;
      default: c = imp + dsc; break;
    }
    s_comp[poff + i] = c;
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

// Finds the key of the `want`-th largest element (1-based) among n_rows rows of `len` floats
// (row r at base + r*stride) and how many elements equal to it are still needed.  Four
// 8-bit digit passes, most significant first; all threads of the CTA take part.
// hist: 256 ints of shared memory.  Returns through tau / need_eq (same in every thread).
__device__ void radix_threshold(const float* base, size_t stride, int n_rows, int len, int want,
                                int* hist, unsigned* tau, int* need_eq) {
  __shared__ unsigned s_prefix;
  __shared__ int s_remaining;
  unsigned prefix = 0, mask = 0;
  int remaining = want;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int t = threadIdx.x; t < 256; t += blockDim.x) hist[t] = 0;
    __syncthreads();
    for (int r = 0; r < n_rows; ++r) {
      const float* row = base + (size_t)r * stride;
      for (int i = threadIdx.x; i < len; i += blockDim.x) {
        const unsigned key = order_key(row[i]);
        if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
      }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int cum = 0, d = 255;
      for (; d > 0; --d) {
        if (cum + hist[d] >= remaining) break;
        cum += hist[d];
      }
      s_prefix = prefix | ((unsigned)d << shift);
      s_remaining = remaining - cum;
    }
    __syncthreads();
    prefix = s_prefix;
    remaining = s_remaining;
    mask |= 255u << shift;
    __syncthreads();
  }
  *tau = prefix;
  *need_eq = remaining;
}

// Head budgets of one sequence.  Fixed: min(B - W, P).  Adaptive: see mixkv.h.
__global__ void __launch_bounds__(1024)
k_budget(const SeqTable st, const float* __restrict__ scores, int* __restrict__ counts,
         const int budget_mode, const int Bp, const int floor_slots) {
  __shared__ int hist[256];
  __shared__ int s_gt[64], s_eq[64];
  const int b = blockIdx.x, H = st.H;
  const int P = st.cu[b + 1] - st.cu[b] - st.W;
  if (budget_mode == MIXKV_BUDGET_FIXED) {
    for (int h = threadIdx.x; h < H; h += blockDim.x) counts[b * H + h] = min(Bp, P);
    return;
  }
  const long long total = (long long)H * P;
  long long N = (long long)H * (Bp - floor_slots);
  if (N > total) N = total;
  const float* base = scores + (st.cu[b] - b * st.W);
  if (N <= 0) {
    for (int h = threadIdx.x; h < H; h += blockDim.x) counts[b * H + h] = min(floor_slots, P);
    return;
  }
  unsigned tau;
  int need_eq;
  radix_threshold(base, (size_t)st.Ptot, H, P, (int)N, hist, &tau, &need_eq);
  for (int h = threadIdx.x; h < H; h += blockDim.x) s_gt[h] = 0, s_eq[h] = 0;
  __syncthreads();
  for (int h = 0; h < H; ++h) {
    int gt = 0, eq = 0;
    const float* row = base + (size_t)h * st.Ptot;
    for (int i = threadIdx.x; i < P; i += blockDim.x) {
      const unsigned key = order_key(row[i]);
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
  __syncthreads();
  if (threadIdx.x == 0) {
    int rem = need_eq;  // equal-to-threshold elements go to the lower (head, position) first
    for (int h = 0; h < H; ++h) {
      const int take = min(s_eq[h], rem);
      rem -= take;
      counts[b * H + h] = min(floor_slots + s_gt[h] + take, P);
    }
  }
}

// Per (sequence, head) top-b selection, ascending position order.
__global__ void __launch_bounds__(1024)
k_select(const SeqTable st, const float* __restrict__ scores, const int* __restrict__ counts,
         int* __restrict__ idx, int* __restrict__ idx_offsets, int* __restrict__ out_row_offsets) {
  __shared__ int hist[256];
  __shared__ int s_gt[32], s_eq[32];
  __shared__ int s_off;
  const int bh = blockIdx.x, b = bh / st.H, h = bh % st.H;
  const int BH = st.batch * st.H;
  const int P = st.cu[b + 1] - st.cu[b] - st.W;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // where this (b, h) starts in the packed outputs
  {
    int part = 0;
    for (int t = tid; t < bh; t += blockDim.x) part += counts[t];
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if (lane == 0) s_gt[warp] = part;
    __syncthreads();
    if (tid == 0) {
      int off = 0;
      for (int w = 0; w < 32; ++w) off += s_gt[w];
      s_off = off;
      idx_offsets[bh] = off;
      if (out_row_offsets) out_row_offsets[bh] = off + bh * st.W;
      if (bh == BH - 1) {
        idx_offsets[BH] = off + counts[bh];
        if (out_row_offsets) out_row_offsets[BH] = off + counts[bh] + BH * st.W;
      }
    }
    __syncthreads();
  }
  const int want = counts[bh];
  int* out = idx + s_off;
  if (want <= 0) return;
  if (want >= P) {
    for (int i = tid; i < P; i += blockDim.x) out[i] = i;
    return;
  }
  const float* row = scores + (size_t)h * st.Ptot + (st.cu[b] - b * st.W);
  unsigned tau;
  int need_eq;
  radix_threshold(row, 0, 1, P, want, hist, &tau, &need_eq);
  // ordered compaction: thread t owns the contiguous positions [t*per, (t+1)*per)
  const int per = (P + blockDim.x - 1) / blockDim.x;
  const int lo = min(tid * per, P), hi = min(lo + per, P);
  int gt = 0, eq = 0;
  for (int i = lo; i < hi; ++i) {
    const unsigned key = order_key(row[i]);
    gt += key > tau;
    eq += key == tau;
  }
  // exclusive scan of (gt, eq) over the CTA
  int gt_inc = gt, eq_inc = eq;
  for (int o = 1; o < 32; o <<= 1) {
    const int a = __shfl_up_sync(0xffffffffu, gt_inc, o);
    const int c = __shfl_up_sync(0xffffffffu, eq_inc, o);
    if (lane >= o) gt_inc += a, eq_inc += c;
  }
  if (lane == 31) s_gt[warp] = gt_inc, s_eq[warp] = eq_inc;
  __syncthreads();
  if (warp == 0) {
    int a = s_gt[lane], c = s_eq[lane];
    int ai = a, ci = c;
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, ai, o);
      const int y = __shfl_up_sync(0xffffffffu, ci, o);
      if (lane >= o) ai += x, ci += y;
    }
    s_gt[lane] = ai - a;
    s_eq[lane] = ci - c;
  }
  __syncthreads();
  int gt_before = s_gt[warp] + gt_inc - gt;
  int eq_before = s_eq[warp] + eq_inc - eq;
  for (int i = lo; i < hi; ++i) {
    const unsigned key = order_key(row[i]);
    if (key > tau) {
      out[gt_before + min(eq_before, need_eq)] = i;
      ++gt_before;
    } else if (key == tau) {
      if (eq_before < need_eq) out[gt_before + eq_before] = i;
      ++eq_before;
    }
  }
}

// --------------------------------------------------------------------------- gather
// One half-warp per output row (16 lanes x 16 bytes = one 256-byte bf16 row).
__global__ void __launch_bounds__(256)
k_gather(const SeqTable st, const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V,
         const int* __restrict__ idx, const int* __restrict__ idx_offsets,
         const int* __restrict__ out_row_offsets, __nv_bfloat16* __restrict__ K_out,
         __nv_bfloat16* __restrict__ V_out) {
  const int bh = blockIdx.y, b = bh / st.H, h = bh % st.H;
  const int n_sel = idx_offsets[bh + 1] - idx_offsets[bh];
  const int rows = n_sel + st.W;
  const int r = blockIdx.x * 16 + (threadIdx.x >> 4);
  if (r >= rows) return;
  const int P = st.cu[b + 1] - st.cu[b] - st.W;
  const int src = r < n_sel ? idx[idx_offsets[bh] + r] : P + (r - n_sel);
  const size_t srow = (size_t)h * st.Ltot + st.cu[b] + src;
  const size_t drow = (size_t)out_row_offsets[bh] + r;
  const int l = threadIdx.x & 15;
  const __nv_bfloat16* X = blockIdx.z == 0 ? K : V;
  __nv_bfloat16* Y = blockIdx.z == 0 ? K_out : V_out;
  reinterpret_cast<uint4*>(Y + drow * kHeadDim)[l] =
      __ldg(reinterpret_cast<const uint4*>(X + srow * kHeadDim) + l);
}

}  // namespace

cudaError_t launch_pool(const LaunchCtx& c, float* s_ex_out) {
  k_pool<<<dim3(c.st.pchunks_total, c.st.H), 256, 0, c.stream>>>(c.st, c.ws, s_ex_out,
                                                                 c.p.pool_kernel, c.p.pool_mode);
  return cudaGetLastError();
}

cudaError_t launch_mix(const LaunchCtx& c, const float* s_ex, const float* s_div,
                       const float* rbar_in, float* s_comp, float* rbar_out) {
  k_mix<<<dim3(c.st.pchunks_total, c.st.H), 256, 0, c.stream>>>(
      c.st, c.ws, s_ex, s_div, rbar_in, s_comp, rbar_out, c.p.use_vnorm, c.p.mix_mode, c.p.eps);
  return cudaGetLastError();
}

static int floor_slots(const mixkv_params& p) {
  const int Bp = p.budget - p.window;
  int f = (int)floor((double)p.ada_floor * (double)Bp);
  if (f > Bp) f = Bp;
  if (f < 0) f = 0;
  return f;
}

cudaError_t launch_budget(const LaunchCtx& c, const float* scores, int* counts) {
  const int threads = c.p.budget_mode == MIXKV_BUDGET_FIXED ? 64 : 1024;
  k_budget<<<c.st.batch, threads, 0, c.stream>>>(c.st, scores, counts, c.p.budget_mode,
                                                 c.p.budget - c.p.window, floor_slots(c.p));
  return cudaGetLastError();
}

cudaError_t launch_select(const LaunchCtx& c, const float* scores, const int* counts, int* idx,
                          int* idx_offsets, int* out_row_offsets) {
  k_select<<<c.st.batch * c.st.H, 1024, 0, c.stream>>>(c.st, scores, counts, idx, idx_offsets,
                                                       out_row_offsets);
  return cudaGetLastError();
}

cudaError_t launch_gather(const LaunchCtx& c, const void* K, const void* V, const int* idx,
                          const int* idx_offsets, const int* out_row_offsets, void* K_out,
                          void* V_out) {
  // upper bound of rows any (b, h) can own
  const int Bp = c.p.budget - c.p.window;
  long long max_sel = Bp;
  if (c.p.budget_mode == MIXKV_BUDGET_ADAPTIVE) {
    const int f = floor_slots(c.p);
    max_sel = (long long)f + (long long)c.st.H * (Bp - f);
  }
  if (max_sel > c.max_prefix) max_sel = c.max_prefix;
  const int max_rows = (int)max_sel + c.st.W;
  const dim3 grid((max_rows + 15) / 16, c.st.batch * c.st.H, 2);
  k_gather<<<grid, 256, 0, c.stream>>>(c.st, (const __nv_bfloat16*)K, (const __nv_bfloat16*)V, idx,
                                       idx_offsets, out_row_offsets, (__nv_bfloat16*)K_out,
                                       (__nv_bfloat16*)V_out);
  return cudaGetLastError();
}

}  // namespace mixkv
