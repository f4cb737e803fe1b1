// Redundancy analysis (the pairwise key / value similarity the paper plots as heat maps and
// summarises per head, Sec. 1 and Sec. 3.1): block-mean cosine similarity map of the rows of
// one tensor.  The mean of cos(x_i, x_j) over a cell (i in block I, j in block J) is
// u_I . u_J / (n_I n_J) with u_I the sum of the unit rows of block I, the same identity that
// turns the mean of the whole matrix into Eq. 4; so the map needs one streaming pass over the
// rows (HBM bound) and a small Gram matrix of the block sums, not the L x L matrix.  That is the
// route for coarse maps; with 1 .. 16 rows per cell the Gram of block sums is the L x L
// contraction itself and runs on the tensor cores (similarity_tc.cu).
#include "common.cuh"

namespace mixkv {
namespace {

constexpr int kSimThreads = 256;
constexpr int kSimRows = 256;   // rows one CTA of the first kernel reads

// grid (T * S, H): unit-row sum and number of non-zero rows of one slice (kSimRows rows at most;
// S slices per block) of one block of one head.  A warp takes four rows at a time (all loads in
// flight); lane l holds elements 4l .. 4l+3 of a row.  u, nz: [H, T * S, ...].
__global__ void __launch_bounds__(kSimThreads)
k_block_unit_sums(const __nv_bfloat16* __restrict__ X, const int L, const int block, const int S,
                  float* __restrict__ u, int* __restrict__ nz) {
  __shared__ float part[kSimThreads / 32][kHeadDim];
  __shared__ int cnt[kSimThreads / 32];
  const int I = blockIdx.x / S, sl = blockIdx.x % S, h = blockIdx.y, T = gridDim.x;   // T: slices per head
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b1 = min(L, (I + 1) * block);
  const int r0 = min(b1, I * block + sl * kSimRows), r1 = min(b1, r0 + kSimRows);
  const __nv_bfloat16* base = X + (size_t)h * L * kHeadDim;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  int nonzero = 0;
  constexpr int kW = kSimThreads / 32, kInFlight = 4;   // rows a warp loads before it reduces any
  for (int r = r0 + warp; r < r1; r += kInFlight * kW) {
    uint2 v[kInFlight];
#pragma unroll
    for (int k = 0; k < kInFlight; ++k) {
      const int rk = r + k * kW;
      v[k] = rk < r1 ? *reinterpret_cast<const uint2*>(base + (size_t)rk * kHeadDim + 4 * lane)
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
      const float inv = n2[k] > 0.f ? rsqrtf(n2[k]) : 0.f;
      nonzero += n2[k] > 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[e] = fmaf(f[k][e], inv, acc[e]);
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) part[warp][4 * lane + e] = acc[e];
  if (lane == 0) cnt[warp] = nonzero;
  __syncthreads();
  if (threadIdx.x < kHeadDim) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kSimThreads / 32; ++w) s += part[w][threadIdx.x];
    u[((size_t)h * T + blockIdx.x) * kHeadDim + threadIdx.x] = s;
  }
  if (threadIdx.x == 0) {
    int c = 0;
    for (int w = 0; w < kSimThreads / 32; ++w) c += cnt[w];
    nz[h * T + blockIdx.x] = c;
  }
}

// grid (T, H), 128 threads: adds the S slices of a block (blocks longer than kSimRows rows).
__global__ void __launch_bounds__(kHeadDim)
k_fold_slices(const float* __restrict__ us, const int* __restrict__ nzs, const int S,
              float* __restrict__ u, int* __restrict__ nz) {
  const int I = blockIdx.x, h = blockIdx.y, T = gridDim.x, c = threadIdx.x;
  float s = 0.f;
  for (int k = 0; k < S; ++k) s += us[(((size_t)h * T + I) * S + k) * kHeadDim + c];
  u[((size_t)h * T + I) * kHeadDim + c] = s;
  if (c == 0) {
    int z = 0;
    for (int k = 0; k < S; ++k) z += nzs[(h * T + I) * S + k];
    nz[h * T + I] = z;
  }
}

// grid (ceil(T/16), ceil(T/16), H), 16 x 16 threads: cells of the map.
__global__ void __launch_bounds__(256)
k_block_map(const float* __restrict__ u, const int* __restrict__ nz, const int L, const int block,
            const int T, float* __restrict__ cells) {
  __shared__ float ui[16][kHeadDim + 1], uj[16][kHeadDim + 1];
  const int h = blockIdx.z, I0 = blockIdx.y * 16, J0 = blockIdx.x * 16;
  const int ty = threadIdx.y, tx = threadIdx.x, t = ty * 16 + tx;
  {
    // thread t stages column t % 128 of rows t / 128, t / 128 + 2, ... : all sixteen loads in flight
    const int c = t & (kHeadDim - 1), rb = t >> 7;
    float a[8], b[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int r = rb + 2 * k;
      a[k] = I0 + r < T ? u[((size_t)h * T + I0 + r) * kHeadDim + c] : 0.f;
      b[k] = J0 + r < T ? u[((size_t)h * T + J0 + r) * kHeadDim + c] : 0.f;
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) ui[rb + 2 * k][c] = a[k], uj[rb + 2 * k][c] = b[k];
  }
  __syncthreads();
  const int I = I0 + ty, J = J0 + tx;
  if (I >= T || J >= T) return;
  float dot = 0.f;
#pragma unroll 8
  for (int c = 0; c < kHeadDim; ++c) dot = fmaf(ui[ty][c], uj[tx][c], dot);
  const float nI = (float)(min(L, (I + 1) * block) - I * block);
  const float nJ = (float)(min(L, (J + 1) * block) - J * block);
  float v;
  if (I != J) {
    v = dot / (nI * nJ);
  } else {   // the pairs i == j are left out: each non-zero row has cosine 1 with itself
    const float pairs = nI * (nI - 1.f);
    v = pairs > 0.f ? (dot - (float)nz[h * T + I]) / pairs : 0.f;
  }
  cells[((size_t)h * T + I) * T + J] = v;
}

// grid H, 1024 threads: mean over all ordered pairs i != j of the head (Eq. 4).  Eight groups of
// 128 threads walk the blocks side by side.
__global__ void __launch_bounds__(1024)
k_head_mean(const float* __restrict__ u, const int* __restrict__ nz, const int L, const int T,
            float* __restrict__ mean) {
  __shared__ float part[8][kHeadDim];
  __shared__ float red[4];
  __shared__ int zs[32];
  const int h = blockIdx.x, c = threadIdx.x & (kHeadDim - 1), g = threadIdx.x >> 7;
  float s = 0.f;
#pragma unroll 16
  for (int I = g; I < T; I += 8) s += u[((size_t)h * T + I) * kHeadDim + c];
  part[g][c] = s;
  int z = 0;
  for (int I = threadIdx.x; I < T; I += 1024) z += nz[h * T + I];
  for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
  if ((threadIdx.x & 31) == 0) zs[threadIdx.x >> 5] = z;
  __syncthreads();
  if (threadIdx.x < kHeadDim) {
    float t = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) t += part[k][c];
    const float n2 = warp_sum(t * t);
    if ((c & 31) == 0) red[c >> 5] = n2;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int total_nz = 0;
    for (int w = 0; w < 32; ++w) total_nz += zs[w];
    const double nn = ((double)red[0] + (double)red[1]) + ((double)red[2] + (double)red[3]);
    const double Ld = (double)L;
    mean[h] = L > 1 ? (float)((nn - (double)total_nz) / (Ld * (Ld - 1.0))) : 0.f;
  }
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace
}  // namespace mixkv

using namespace mixkv;

extern "C" {

int mixkv_similarity_workspace_size(int32_t heads, int32_t L, int32_t block, size_t* bytes) {
  if (!bytes || heads < 1 || L < 1 || block < 1) return MIXKV_ERR_INVALID_ARG;
  if (similarity_dense_block(block)) {
    *bytes = similarity_dense_workspace(heads, L);
    return MIXKV_OK;
  }
  const size_t T = ((size_t)L + block - 1) / block;
  const size_t S = ((size_t)block + kSimRows - 1) / kSimRows;   // slices per block
  *bytes = align256((size_t)heads * T * kHeadDim * 4) + align256((size_t)heads * T * 4);
  if (S > 1) *bytes += align256((size_t)heads * T * S * kHeadDim * 4) + align256((size_t)heads * T * S * 4);
  return MIXKV_OK;
}

int mixkv_similarity_map(const void* X, int32_t heads, int32_t L, int32_t head_dim, int32_t block,
                         void* workspace, size_t workspace_bytes, float* cells, float* mean_opt,
                         void* stream) {
  if (!X || !workspace || !cells || heads < 1 || L < 1 || block < 1) return MIXKV_ERR_INVALID_ARG;
  if (head_dim != kHeadDim) return MIXKV_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(X) & 15u) || (reinterpret_cast<uintptr_t>(workspace) & 15u))
    return MIXKV_ERR_INVALID_ARG;
  size_t need = 0;
  mixkv_similarity_workspace_size(heads, L, block, &need);
  if (workspace_bytes < need) return MIXKV_ERR_WORKSPACE_TOO_SMALL;
  const long long T = ((long long)L + block - 1) / block;
  const long long S = ((long long)block + kSimRows - 1) / kSimRows;
  if (T > 65535 || heads > 65535 || T * S > 0x7fffffffLL) return MIXKV_ERR_UNSUPPORTED;   // grid limits
  {
    const int rc = device_check(nullptr);
    if (rc != MIXKV_OK) return rc;
  }
  cudaStream_t s = (cudaStream_t)stream;
  if (similarity_dense_block(block)) {
    float* ud = nullptr;
    int* nzd = nullptr;
    int slices = 0;
    if (launch_similarity_dense(X, heads, L, block, workspace, cells, &ud, &nzd, &slices, s) !=
        cudaSuccess)
      return MIXKV_ERR_CUDA;
    if (mean_opt) k_head_mean<<<(unsigned)heads, 1024, 0, s>>>(ud, nzd, L, slices, mean_opt);
    return cudaGetLastError() == cudaSuccess ? MIXKV_OK : MIXKV_ERR_CUDA;
  }
  unsigned char* wsb = reinterpret_cast<unsigned char*>(workspace);
  float* u = reinterpret_cast<float*>(wsb);
  wsb += align256((size_t)heads * T * kHeadDim * 4);
  int* nz = reinterpret_cast<int*>(wsb);
  wsb += align256((size_t)heads * T * 4);
  if (S == 1) {
    k_block_unit_sums<<<dim3((unsigned)T, (unsigned)heads), kSimThreads, 0, s>>>(
        reinterpret_cast<const __nv_bfloat16*>(X), L, block, 1, u, nz);
  } else {
    float* us = reinterpret_cast<float*>(wsb);
    wsb += align256((size_t)heads * T * S * kHeadDim * 4);
    int* nzs = reinterpret_cast<int*>(wsb);
    k_block_unit_sums<<<dim3((unsigned)(T * S), (unsigned)heads), kSimThreads, 0, s>>>(
        reinterpret_cast<const __nv_bfloat16*>(X), L, block, (int)S, us, nzs);
    k_fold_slices<<<dim3((unsigned)T, (unsigned)heads), kHeadDim, 0, s>>>(us, nzs, (int)S, u, nz);
  }
  const unsigned g = (unsigned)((T + 15) / 16);
  k_block_map<<<dim3(g, g, (unsigned)heads), dim3(16, 16), 0, s>>>(u, nz, L, block, (int)T, cells);
  if (mean_opt) k_head_mean<<<(unsigned)heads, 1024, 0, s>>>(u, nz, L, (int)T, mean_opt);
  return cudaGetLastError() == cudaSuccess ? MIXKV_OK : MIXKV_ERR_CUDA;
}

}  // extern "C"
