// Shared declarations of the MixKV CUDA library (sm_100a): problem description handed to
// every kernel, the workspace carve-up, and small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mixkv.h"

namespace mixkv {

constexpr int kHeadDim = 128;        // d, fixed
constexpr int kMaxBatch = 64;        // sequences per call
constexpr int kMaxLayers = 1024;     // layers per call
constexpr int kMaxNQ = 240;          // G*W upper bound (16 spare rows carry the mean key)
constexpr int kTile = 128;           // keys per tensor-core tile
constexpr int kPChunk = 2048;        // candidate positions per CTA in pool / mix
constexpr int kExtraRows = 16;       // rows appended to the query tile in pass 2
constexpr float kLog2e = 1.4426950408889634f;

// Everything a kernel needs to find its slice of the ragged batch.
struct SeqTable {
  int layers;                        // layers handled by one call (an outer batch dimension)
  int batch, H, G, W, NQ;
  int Ltot, Ptot;
  int pchunks_total;                 // sum over sequences of ceil(P_b / kPChunk)
  int cu[kMaxBatch + 1];             // sequence offsets into Ltot
  int pchunk_start[kMaxBatch + 1];   // prefix sum of candidate chunks
  // persistent 128-key tile schedules of the two tensor-core passes, (b, h, t) order
  // Tiles of one layer: nt1 over all L keys (pass 1), nt2 over the P candidate keys (pass 2).
  // layers * nt tiles are split over g CTAs: layers * nt = q * g + r.
  int nt1, g1, q1, r1;
  int nt2, g2, q2, r2;
  int tile1_start[kMaxBatch + 1];    // prefix sum of H * ceil(L_b / 128)
  int tile2_start[kMaxBatch + 1];    // prefix sum of H * ceil(P_b / 128)
};

// nt tiles split contiguously over g CTAs (g <= nt): the first r CTAs take q + 1 tiles, the
// others q.
struct Split {
  int nt, g, q, r;
};

// Device workspace carve-up (all pointers into the caller's workspace).
struct Workspace {
  // every array below has a leading [layers] dimension
  float* kinv;        // [H, Ltot]   1 / |K_i|  (0 for a zero key)
  float* vnorm;       // [H, Ptot]   |V_i|
  float* s_ex_raw;    // [H, Ptot]   window attention score before pooling
  float* s_div;       // [H, Ptot]
  float* s_comp;      // [H, Ptot]
  // per-segment partial results; a segment is a run of tiles of one (b, h) inside one CTA's
  // range and its slot is the id of its first tile
  float2* rowstat;    // [nt1, NQ]  softmax (reference, sum) of each window row, log2 units
  float* ksum;        // [nt1, d]      sum of unit keys
  float4* vstat;      // [nt2]         (min, max, sum, -) of |V_i| over candidates
  float4* dstat;      // [nt2, 2]      per epilogue warpgroup: (min, max, sum) of s_div, window-count-weighted sum of s_ex_raw
  float* exsum;       // [H, pchunks_total]   per-chunk sum of pooled s_ex (max pooling only)
  float* rbar;        // [batch*H]   redundancy of Eq. 4, left by pass 2
  int* counts;        // [batch*H]
  int* idx_offsets;   // [batch*H + 1]
  int* idx;           // [batch*H*(B-W)]
  size_t bytes;
};

struct LaunchCtx {
  SeqTable st;
  Workspace ws;
  mixkv_params p;
  long long kv_layer_stride;   // elements between the K (V) tensors of consecutive layers
  long long q_layer_stride;    // elements between the window queries of consecutive layers
  int idx_cap;                 // selected rows one layer can produce (capacity of its index list)
  int out_rows_cap;            // output rows reserved per layer: batch * H * B
  float scale_log2e;   // softmax scale * log2(e)
  int max_seq_len;
  int max_prefix;
  cudaStream_t stream;
  void* const* trace_events;  // optional measurement hook: events recorded between kernels
  int n_trace_events;
  mutable int stage;

  // Records the event that marks the start of the next kernel (or the end of the last).
  void mark() const {
    if (trace_events && stage < n_trace_events && trace_events[stage])
      cudaEventRecord((cudaEvent_t)trace_events[stage], stream);
    ++stage;
  }
};

// ---- kernels (defined in the .cu files) ------------------------------------------
cudaError_t launch_pass1(const LaunchCtx& c, const void* K, const void* Q, int* status);
cudaError_t launch_pass2(const LaunchCtx& c, const void* K, const void* V, const void* Q,
                         float* s_div_out, float* rbar_out, int* status);
int device_sm_count();
// Fills a CUtensorMap (passed as void*) for a bf16 tensor of the given rank: dims innermost first,
// strides in bytes of dimensions 1 .. rank-1, box extents; 128-byte swizzle, zero fill outside.
bool encode_bf16_map(void* tm, const void* base, int rank, const unsigned long long* dims,
                     const unsigned long long* strides_bytes, const unsigned* box);
// MIXKV_OK on a compute-capability 10.x device, MIXKV_ERR_UNSUPPORTED on any other,
// MIXKV_ERR_CUDA when none can be queried; *major_out (optional) receives the major number.
int device_check(int* major_out);
cudaError_t launch_poolsum(const LaunchCtx& c);
cudaError_t launch_mixpool(const LaunchCtx& c, const float* s_div, const float* rbar_in,
                           float* s_ex_out, float* s_comp);
cudaError_t launch_budget(const LaunchCtx& c, const float* scores, int* counts);
// Selection (and optionally the mix before it and the gather after it) by one CTA cluster per
// (sequence, head).  scores != nullptr: select on them; else mix first (s_div, rbar_in) and
// write the mixed scores to s_comp_out.  counts_dev == nullptr: fixed budgets.
// Index of (layer, head h, sequence b, position i) in a [layers, H, Ltot] / [layers, H, Ptot]
// array.
__host__ __device__ __forceinline__ size_t kpos(const SeqTable& st, int layer, int h, int b,
                                                int i) {
  return ((size_t)layer * st.H + h) * st.Ltot + st.cu[b] + i;
}
__host__ __device__ __forceinline__ size_t ppos(const SeqTable& st, int layer, int h, int b,
                                                int i) {
  return ((size_t)layer * st.H + h) * st.Ptot + (st.cu[b] - b * st.W) + i;
}

// Dense (tensor-core) route of the similarity map for block = 1, 2, 4, 8, 16 (similarity_tc.cu).
bool similarity_dense_block(int block);
size_t similarity_dense_workspace(int heads, int L);
cudaError_t launch_similarity_dense(const void* X, int heads, int L, int block, void* workspace,
                                    float* cells, float** u_out, int** nz_out, int* slices_out,
                                    cudaStream_t s);

struct TailArgs {
  const float* scores;
  const float* s_div;
  const float* rbar_in;
  float* s_comp_out;
  const int* counts_dev;
  int* counts_out;
  int* idx;
  int* idx_offsets;
  int* out_row_offsets;
  const void* K;
  const void* V;
  void* K_out;
  void* V_out;
};
// counts [layers, batch*H] <- candidates to select for budgets [layers, batch*H] given by the caller
cudaError_t launch_given_budgets(const LaunchCtx& c, const int* budgets, int* counts);
cudaError_t launch_tail(const LaunchCtx& c, const TailArgs& a);
// Whether the longest sequence is short enough for the fused mix + select + gather kernel.
bool tail_can_fuse(const LaunchCtx& c);

// Launch with programmatic dependent launch (and an optional cluster size): the kernel may
// start while its predecessor in the stream drains; every kernel calls pdl_wait() before it
// touches global memory.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                       cudaStream_t stream, int cluster, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = (unsigned)n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- device helpers ----------------------------------------------------------------
__device__ __forceinline__ int find_seq(const int* start, int batch, int x) {
  int b = 0;
  while (b + 1 < batch && x >= start[b + 1]) ++b;
  return b;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Programmatic dependent launch: let the next kernel of the stream be scheduled, and wait
// until everything before this kernel in the stream has completed and is visible.
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

}  // namespace mixkv
