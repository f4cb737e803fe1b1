// C ABI of the MixKV library: argument checks, workspace carve-up, kernel sequencing.
#include <math.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "common.cuh"

namespace mixkv {

// MIXKV_OK when the current device has compute capability 10.x (tcgen05, tensor memory), else
// UNSUPPORTED; CUDA when the device cannot be queried.  Looked up once per device.
int classify_cc(int major) { return major == 10 ? MIXKV_OK : MIXKV_ERR_UNSUPPORTED; }
int device_check(int* major_out) {
  static std::atomic<int> cached[64];   // 0 = unknown, else major + 1
  int dev = 0;
  if (major_out) *major_out = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MIXKV_ERR_CUDA;
  int major = 0;
  if (dev >= 0 && dev < 64 && cached[dev].load(std::memory_order_relaxed) != 0) {
    major = cached[dev].load(std::memory_order_relaxed) - 1;
  } else {
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
      return MIXKV_ERR_CUDA;
    if (dev >= 0 && dev < 64) cached[dev].store(major + 1, std::memory_order_relaxed);
  }
  if (major_out) *major_out = major;
  return classify_cc(major);
}

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int check_params(const mixkv_params* p) {
  if (!p) return MIXKV_ERR_INVALID_ARG;
  if (p->kv_heads < 1 || p->gqa_ratio < 1 || p->window < 1) return MIXKV_ERR_INVALID_ARG;
  if (p->pool_kernel < 1 || (p->pool_kernel & 1) == 0) return MIXKV_ERR_INVALID_ARG;
  if (p->pool_mode != MIXKV_POOL_AVG && p->pool_mode != MIXKV_POOL_MAX) return MIXKV_ERR_INVALID_ARG;
  if (p->mix_mode < 0 || p->mix_mode > 3) return MIXKV_ERR_INVALID_ARG;
  if (p->use_vnorm < MIXKV_INTRINSIC_NONE || p->use_vnorm > MIXKV_INTRINSIC_KNORM)
    return MIXKV_ERR_INVALID_ARG;
  if (p->budget_mode != MIXKV_BUDGET_FIXED && p->budget_mode != MIXKV_BUDGET_ADAPTIVE)
    return MIXKV_ERR_INVALID_ARG;
  if (p->budget <= p->window) return MIXKV_ERR_INVALID_ARG;
  if (!(p->ada_floor >= 0.f && p->ada_floor <= 1.f)) return MIXKV_ERR_INVALID_ARG;
  if (!(p->eps >= 0.f) || !(p->softmax_scale >= 0.f)) return MIXKV_ERR_INVALID_ARG;
  if (p->head_dim != kHeadDim) return MIXKV_ERR_UNSUPPORTED;
  const long long nq = (long long)p->gqa_ratio * p->window;
  if (nq < 16 || nq > kMaxNQ || (nq % 16) != 0) return MIXKV_ERR_UNSUPPORTED;
  if (p->pool_kernel > 63) return MIXKV_ERR_UNSUPPORTED;
  if (p->kv_heads > 64) return MIXKV_ERR_UNSUPPORTED;
  return MIXKV_OK;
}

// Builds the sequence table from the host offsets (or a single length).
int build_table(const mixkv_params* p, const int32_t* cu, int batch, int L, int layers,
                SeqTable* st, int* max_len) {
  if (batch < 1 || layers < 1) return MIXKV_ERR_INVALID_ARG;
  if (batch > kMaxBatch || layers > kMaxLayers) return MIXKV_ERR_UNSUPPORTED;
  if (!cu && batch != 1) return MIXKV_ERR_INVALID_ARG;
  memset(st, 0, sizeof(*st));
  st->layers = layers;
  st->batch = batch;
  st->H = p->kv_heads;
  st->G = p->gqa_ratio;
  st->W = p->window;
  st->NQ = p->gqa_ratio * p->window;
  int mx = 0;
  for (int b = 0; b <= batch; ++b) st->cu[b] = cu ? cu[b] : (b == 0 ? 0 : L);
  if (st->cu[0] != 0) return MIXKV_ERR_INVALID_ARG;
  for (int b = 0; b < batch; ++b) {
    const long long len = (long long)st->cu[b + 1] - st->cu[b];
    if (len < p->window + 1 || len < 2) return MIXKV_ERR_INVALID_ARG;
    if (len > mx) mx = (int)len;
    st->pchunk_start[b + 1] =
        st->pchunk_start[b] + (int)((len - p->window + kPChunk - 1) / kPChunk);
    st->tile1_start[b + 1] = st->tile1_start[b] + st->H * (int)((len + kTile - 1) / kTile);
    st->tile2_start[b + 1] =
        st->tile2_start[b] + st->H * (int)((len - p->window + kTile - 1) / kTile);
  }
  st->Ltot = st->cu[batch];
  st->Ptot = st->Ltot - batch * p->window;
  st->pchunks_total = st->pchunk_start[batch];
  st->nt1 = st->tile1_start[batch];
  st->nt2 = st->tile2_start[batch];
  const long long t1 = (long long)layers * st->nt1, t2 = (long long)layers * st->nt2;
  if (t1 > 0x3fffffffLL) return MIXKV_ERR_UNSUPPORTED;
  const int sms = device_sm_count();
  st->g1 = t1 < sms ? (int)t1 : sms;
  st->g2 = t2 < sms ? (int)t2 : sms;
  st->q1 = (int)(t1 / st->g1), st->r1 = (int)(t1 % st->g1);
  st->q2 = (int)(t2 / st->g2), st->r2 = (int)(t2 % st->g2);
  *max_len = mx;
  return MIXKV_OK;
}

// Upper bound of selected (non-window) rows over the whole batch.
long long idx_capacity(const mixkv_params* p, const SeqTable& st) {
  long long cap = 0;
  for (int b = 0; b < st.batch; ++b) {
    const long long P = st.cu[b + 1] - st.cu[b] - st.W;
    long long per_seq = (long long)st.H * (p->budget - p->window);
    if (per_seq > st.H * P) per_seq = st.H * P;
    cap += per_seq;
  }
  return cap;
}

// Lays the workspace out; with base == nullptr only the size is computed.
void carve(const mixkv_params* p, const SeqTable& st, unsigned char* base, Workspace* ws) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    unsigned char* ptr = base ? base + off : nullptr;
    off = align_up(off + bytes, 256);
    return ptr;
  };
  const size_t NL = st.layers, H = st.H, BH = (size_t)st.batch * st.H;
  ws->kinv = (float*)take(NL * H * st.Ltot * 4);
  ws->vnorm = (float*)take(NL * H * st.Ptot * 4);
  ws->s_ex_raw = (float*)take(NL * H * st.Ptot * 4);
  ws->s_div = (float*)take(NL * H * st.Ptot * 4);
  ws->s_comp = (float*)take(NL * H * st.Ptot * 4);
  ws->rowstat = (float2*)take(NL * st.nt1 * st.NQ * 8);
  ws->ksum = (float*)take(NL * st.nt1 * kHeadDim * 4);
  ws->vstat = (float4*)take(NL * st.nt2 * 16);
  ws->dstat = (float4*)take(NL * st.nt2 * 2 * 16);
  ws->exsum = (float*)take(NL * H * st.pchunks_total * 4);
  ws->rbar = (float*)take(NL * BH * 4);
  ws->counts = (int*)take(NL * BH * 4);
  ws->idx_offsets = (int*)take(NL * (BH + 1) * 4);
  ws->idx = (int*)take(NL * (size_t)idx_capacity(p, st) * 4);
  ws->bytes = off;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int make_ctx(const mixkv_params* p, const int32_t* cu, int batch, int L, void* workspace,
             size_t workspace_bytes, void* stream, LaunchCtx* c, int layers = 1,
             long long kv_layer_stride = 0, long long q_layer_stride = 0) {
  int rc = check_params(p);
  if (rc != MIXKV_OK) return rc;
  int max_len = 0;
  rc = build_table(p, cu, batch, L, layers, &c->st, &max_len);
  if (rc != MIXKV_OK) return rc;
  // layer strides in elements; 0 = the layers are packed back to back
  const long long kv_dense = (long long)c->st.H * c->st.Ltot * kHeadDim;
  const long long q_dense = (long long)batch * c->st.H * c->st.NQ * kHeadDim;
  c->kv_layer_stride = kv_layer_stride ? kv_layer_stride : kv_dense;
  c->q_layer_stride = q_layer_stride ? q_layer_stride : q_dense;
  if (layers > 1 && (c->kv_layer_stride < kv_dense || c->q_layer_stride < q_dense ||
                     (c->kv_layer_stride & 7) || (c->q_layer_stride & 7)))
    return MIXKV_ERR_INVALID_ARG;   // layers must not overlap; TMA wants 16-byte strides
  c->idx_cap = (int)idx_capacity(p, c->st);
  c->out_rows_cap = batch * c->st.H * p->budget;
  if (!workspace || !aligned16(workspace)) return MIXKV_ERR_INVALID_ARG;
  carve(p, c->st, (unsigned char*)workspace, &c->ws);
  if (c->ws.bytes > workspace_bytes) return MIXKV_ERR_WORKSPACE_TOO_SMALL;
  c->p = *p;
  const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)kHeadDim);
  c->scale_log2e = scale * kLog2e;
  c->max_seq_len = max_len;
  c->max_prefix = max_len - p->window;
  c->stream = (cudaStream_t)stream;
  c->trace_events = nullptr;
  c->n_trace_events = 0;
  c->stage = 0;
  return MIXKV_OK;
}

// pass 1, pass 2 (and the pooled-score sums max pooling needs): everything the mix reads.
int enqueue_passes(const LaunchCtx& c, const void* K, const void* V, const void* Q, float* s_div,
                   float* rbar_out, int* status) {
  c.mark();
  if (launch_pass1(c, K, Q, status) != cudaSuccess) return MIXKV_ERR_CUDA;
  c.mark();
  if (launch_pass2(c, K, V, Q, s_div, rbar_out, status) != cudaSuccess) return MIXKV_ERR_CUDA;
  if (c.p.pool_mode == MIXKV_POOL_MAX) {
    c.mark();
    if (launch_poolsum(c) != cudaSuccess) return MIXKV_ERR_CUDA;
  }
  return MIXKV_OK;
}

int enqueue_scores(const LaunchCtx& c, const void* K, const void* V, const void* Q, float* s_comp,
                   float* s_ex_out, float* s_div_out, float* rbar_out, const float* rbar_in,
                   int* status) {
  float* s_div = s_div_out ? s_div_out : c.ws.s_div;
  int rc = enqueue_passes(c, K, V, Q, s_div, rbar_out, status);
  if (rc != MIXKV_OK) return rc;
  c.mark();
  if (launch_mixpool(c, s_div, rbar_in, s_ex_out, s_comp) != cudaSuccess) return MIXKV_ERR_CUDA;
  return MIXKV_OK;
}

// Budgets (adaptive only) and the selection on given scores; gathers when t.K_out is set.
int enqueue_select(const LaunchCtx& c, const float* scores, int* counts, TailArgs t) {
  t.scores = scores;
  t.counts_dev = nullptr;
  t.counts_out = counts;
  if (c.p.budget_mode == MIXKV_BUDGET_ADAPTIVE) {
    c.mark();
    if (launch_budget(c, scores, counts) != cudaSuccess) return MIXKV_ERR_CUDA;
    t.counts_dev = counts;
    t.counts_out = nullptr;
  }
  c.mark();
  if (launch_tail(c, t) != cudaSuccess) return MIXKV_ERR_CUDA;
  return MIXKV_OK;
}

// Names of the kernels a layer call enqueues, in order.
int layer_stages(const mixkv_params* p, bool fused_ok, const char** names) {
  int n = 0;
  names[n++] = "pass1";
  names[n++] = "pass2";
  if (p->pool_mode == MIXKV_POOL_MAX) names[n++] = "poolsum";
  if (p->budget_mode == MIXKV_BUDGET_ADAPTIVE || !fused_ok) names[n++] = "mixpool";
  if (p->budget_mode == MIXKV_BUDGET_ADAPTIVE) names[n++] = "budget";
  names[n++] = "tail";
  return n;
}

}  // namespace
}  // namespace mixkv

using namespace mixkv;

extern "C" {

void mixkv_default_params(mixkv_params* p, int32_t kv_heads, int32_t gqa_ratio, int32_t budget) {
  if (!p) return;
  memset(p, 0, sizeof(*p));
  p->kv_heads = kv_heads;
  p->gqa_ratio = gqa_ratio;
  p->head_dim = kHeadDim;
  p->window = 32;
  p->pool_kernel = 7;
  p->pool_mode = MIXKV_POOL_AVG;
  p->use_vnorm = 1;
  p->mix_mode = MIXKV_MIX_HEADWISE;
  p->budget_mode = MIXKV_BUDGET_FIXED;
  p->budget = budget;
  p->ada_floor = 0.2f;
  p->eps = 1e-6f;
  p->softmax_scale = 0.f;
}

int mixkv_workspace_size(const mixkv_params* p, int32_t batch, int64_t total_tokens,
                         int32_t max_seq_len, size_t* bytes) {
  return mixkv_workspace_size_layers(p, 1, batch, total_tokens, max_seq_len, bytes);
}

int mixkv_workspace_size_layers(const mixkv_params* p, int32_t n_layers, int32_t batch,
                                int64_t total_tokens, int32_t max_seq_len, size_t* bytes) {
  int rc = check_params(p);
  if (rc != MIXKV_OK) return rc;
  if (!bytes || batch < 1 || n_layers < 1 || total_tokens < batch || max_seq_len < 1)
    return MIXKV_ERR_INVALID_ARG;
  if (batch > kMaxBatch || n_layers > kMaxLayers) return MIXKV_ERR_UNSUPPORTED;
  if (total_tokens > 0x7fffffffLL / 2) return MIXKV_ERR_UNSUPPORTED;
  // a table with the worst-case chunk counts for these totals
  SeqTable st;
  memset(&st, 0, sizeof(st));
  st.layers = n_layers;
  st.batch = batch;
  st.H = p->kv_heads;
  st.G = p->gqa_ratio;
  st.W = p->window;
  st.NQ = p->gqa_ratio * p->window;
  st.Ltot = (int)total_tokens;
  st.Ptot = (int)total_tokens;  // >= the true candidate count
  st.pchunks_total = (int)(total_tokens / kPChunk) + batch;
  st.nt1 = st.nt2 = p->kv_heads * ((int)(total_tokens / kTile) + batch);
  // capacity of the index list: every sequence at its budget
  st.cu[0] = 0;
  for (int b = 1; b <= batch; ++b) st.cu[b] = 0;
  Workspace ws;
  carve(p, st, nullptr, &ws);
  // idx_capacity() saw empty sequences above; add the true bound
  const size_t idx_bytes =
      (size_t)n_layers * batch * p->kv_heads * (size_t)(p->budget - p->window) * 4;
  *bytes = ws.bytes + align_up(idx_bytes, 256) + 256;
  return MIXKV_OK;
}

int mixkv_scores(const void* K, const void* V, const void* Qwin, const int32_t* cu_seqlens_host,
                 int32_t batch, int32_t L, const mixkv_params* p, void* workspace,
                 size_t workspace_bytes, float* s_comp, float* s_ex_opt, float* s_div_opt,
                 float* rbar_opt, const float* rbar_in_opt, int32_t* status_dev, void* stream) {
  LaunchCtx c;
  int rc = make_ctx(p, cu_seqlens_host, batch, L, workspace, workspace_bytes, stream, &c);
  if (rc != MIXKV_OK) return rc;
  if (!K || !Qwin || !s_comp || (p->use_vnorm == MIXKV_INTRINSIC_VNORM && !V))
    return MIXKV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(Qwin) || (V && !aligned16(V))) return MIXKV_ERR_INVALID_ARG;
  rc = device_check(nullptr);   // last: every argument error is reported without a device
  if (rc != MIXKV_OK) return rc;
  return enqueue_scores(c, K, V, Qwin, s_comp, s_ex_opt, s_div_opt, rbar_opt, rbar_in_opt,
                        status_dev);
}

int mixkv_select(const float* scores, const int32_t* cu_seqlens_host, int32_t batch, int32_t L,
                 const mixkv_params* p, void* workspace, size_t workspace_bytes, int32_t* idx,
                 int32_t* counts, int32_t* idx_offsets, int32_t* status_dev, void* stream) {
  (void)status_dev;
  LaunchCtx c;
  int rc = make_ctx(p, cu_seqlens_host, batch, L, workspace, workspace_bytes, stream, &c);
  if (rc != MIXKV_OK) return rc;
  if (!scores || !idx || !counts || !idx_offsets) return MIXKV_ERR_INVALID_ARG;
  rc = device_check(nullptr);
  if (rc != MIXKV_OK) return rc;
  TailArgs t;
  memset(&t, 0, sizeof(t));
  t.idx = idx;
  t.idx_offsets = idx_offsets;
  return enqueue_select(c, scores, counts, t);
}

namespace {
// Body of the layer calls: n_layers layers of identical shape in one set of launches.
int compress_impl(const void* K, const void* V, const void* Qwin, int n_layers,
                  long long kv_layer_stride, long long q_layer_stride,
                  const int32_t* cu_seqlens_host, int32_t batch, int32_t L, const mixkv_params* p,
                  void* workspace, size_t workspace_bytes, const float* rbar_in_opt, void* K_out,
                  void* V_out, int32_t* out_row_offsets, int32_t* idx_opt, int32_t* counts_opt,
                  int32_t* idx_offsets_opt, float* s_comp_opt, int32_t* status_dev, void* stream,
                  void* const* events_host, int32_t n_events,
                  const int32_t* head_budgets = nullptr) {
  LaunchCtx c;
  int rc = make_ctx(p, cu_seqlens_host, batch, L, workspace, workspace_bytes, stream, &c, n_layers,
                    kv_layer_stride, q_layer_stride);
  if (rc != MIXKV_OK) return rc;
  if (events_host && n_events > 0) {
    c.trace_events = events_host;
    c.n_trace_events = n_events;
  }
  if (!K || !V || !Qwin || !K_out || !V_out || !out_row_offsets) return MIXKV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(Qwin) || !aligned16(K_out) || !aligned16(V_out))
    return MIXKV_ERR_INVALID_ARG;
  if (head_budgets && p->budget_mode != MIXKV_BUDGET_FIXED) return MIXKV_ERR_INVALID_ARG;
  rc = device_check(nullptr);
  if (rc != MIXKV_OK) return rc;
  float* s_comp = s_comp_opt ? s_comp_opt : c.ws.s_comp;
  int* counts = counts_opt ? counts_opt : c.ws.counts;
  TailArgs t;
  memset(&t, 0, sizeof(t));
  t.idx = idx_opt ? idx_opt : c.ws.idx;
  t.idx_offsets = idx_offsets_opt ? idx_offsets_opt : c.ws.idx_offsets;
  t.out_row_offsets = out_row_offsets;
  t.K = K;
  t.V = V;
  t.K_out = K_out;
  t.V_out = V_out;
  if (head_budgets) {
    // budgets given per (layer, sequence, head): no scores are needed to fix the counts
    if (p->budget_mode != MIXKV_BUDGET_FIXED) return MIXKV_ERR_INVALID_ARG;
    if (launch_given_budgets(c, head_budgets, counts) != cudaSuccess) return MIXKV_ERR_CUDA;
  }
  rc = enqueue_passes(c, K, V, Qwin, c.ws.s_div, nullptr, status_dev);
  if (rc != MIXKV_OK) return rc;
  if (p->budget_mode == MIXKV_BUDGET_FIXED && tail_can_fuse(c)) {
    // one kernel: mix, select, gather
    t.s_div = c.ws.s_div;
    t.rbar_in = rbar_in_opt;
    t.s_comp_out = s_comp;
    t.counts_dev = head_budgets ? counts : nullptr;
    t.counts_out = head_budgets ? nullptr : counts;
    c.mark();
    if (launch_tail(c, t) != cudaSuccess) return MIXKV_ERR_CUDA;
  } else if (head_budgets) {
    c.mark();
    if (launch_mixpool(c, c.ws.s_div, rbar_in_opt, nullptr, s_comp) != cudaSuccess)
      return MIXKV_ERR_CUDA;
    t.scores = s_comp;
    t.counts_dev = counts;
    t.counts_out = nullptr;
    c.mark();
    if (launch_tail(c, t) != cudaSuccess) return MIXKV_ERR_CUDA;
  } else {
    c.mark();
    if (launch_mixpool(c, c.ws.s_div, rbar_in_opt, nullptr, s_comp) != cudaSuccess)
      return MIXKV_ERR_CUDA;
    rc = enqueue_select(c, s_comp, counts, t);
    if (rc != MIXKV_OK) return rc;
  }
  c.mark();
  return MIXKV_OK;
}
}  // namespace

int mixkv_compress_layer_traced(const void* K, const void* V, const void* Qwin,
                                const int32_t* cu_seqlens_host, int32_t batch, int32_t L,
                                const mixkv_params* p, void* workspace, size_t workspace_bytes,
                                const float* rbar_in_opt, void* K_out, void* V_out,
                                int32_t* out_row_offsets, int32_t* idx_opt, int32_t* counts_opt,
                                int32_t* idx_offsets_opt, float* s_comp_opt, int32_t* status_dev,
                                void* stream, void* const* events_host, int32_t n_events) {
  return compress_impl(K, V, Qwin, 1, 0, 0, cu_seqlens_host, batch, L, p, workspace,
                       workspace_bytes, rbar_in_opt, K_out, V_out, out_row_offsets, idx_opt,
                       counts_opt, idx_offsets_opt, s_comp_opt, status_dev, stream, events_host,
                       n_events);
}

int mixkv_compress_layers(const void* K, const void* V, const void* Qwin, int32_t n_layers,
                          int64_t kv_layer_stride, int64_t q_layer_stride,
                          const int32_t* cu_seqlens_host, int32_t batch, int32_t L,
                          const mixkv_params* p, void* workspace, size_t workspace_bytes,
                          const float* rbar_in_opt, void* K_out, void* V_out,
                          int32_t* out_row_offsets, int32_t* idx_opt, int32_t* counts_opt,
                          int32_t* idx_offsets_opt, float* s_comp_opt, int32_t* status_dev,
                          void* stream, void* const* events_host, int32_t n_events) {
  if (kv_layer_stride < 0 || q_layer_stride < 0) return MIXKV_ERR_INVALID_ARG;
  return compress_impl(K, V, Qwin, n_layers, kv_layer_stride, q_layer_stride, cu_seqlens_host,
                       batch, L, p, workspace, workspace_bytes, rbar_in_opt, K_out, V_out,
                       out_row_offsets, idx_opt, counts_opt, idx_offsets_opt, s_comp_opt,
                       status_dev, stream, events_host, n_events);
}

int mixkv_compress_layers_budgeted(const void* K, const void* V, const void* Qwin,
                                   int32_t n_layers, int64_t kv_layer_stride,
                                   int64_t q_layer_stride, const int32_t* cu_seqlens_host,
                                   int32_t batch, int32_t L, const mixkv_params* p,
                                   void* workspace, size_t workspace_bytes,
                                   const float* rbar_in_opt, const int32_t* head_budgets,
                                   void* K_out, void* V_out, int32_t* out_row_offsets,
                                   int32_t* idx_opt, int32_t* counts_opt, int32_t* idx_offsets_opt,
                                   float* s_comp_opt, int32_t* status_dev, void* stream) {
  if (kv_layer_stride < 0 || q_layer_stride < 0 || !head_budgets) return MIXKV_ERR_INVALID_ARG;
  return compress_impl(K, V, Qwin, n_layers, kv_layer_stride, q_layer_stride, cu_seqlens_host,
                       batch, L, p, workspace, workspace_bytes, rbar_in_opt, K_out, V_out,
                       out_row_offsets, idx_opt, counts_opt, idx_offsets_opt, s_comp_opt,
                       status_dev, stream, nullptr, 0, head_budgets);
}

int mixkv_layer_budget_schedule(int32_t n_layers, int32_t budget, int32_t window,
                                int32_t taper_permille, int32_t* budgets_host) {
  if (n_layers < 1 || !budgets_host || window < 0 || budget <= window || taper_permille < 0 ||
      taper_permille > 999)
    return MIXKV_ERR_INVALID_ARG;
  const long long Bp = budget - window, n = n_layers;
  if (n == 1) {
    budgets_host[0] = budget;
    return MIXKV_OK;
  }
  // candidates of layer l: Bp * (1 + t * (1 - 2 l / (n - 1))), t = taper_permille / 1000, rounded
  // down; the rows lost to rounding go to the lowest layers, one each, so the total stays n * Bp
  const long long den = 1000 * (n - 1);
  long long given = 0;
  for (long long l = 0; l < n; ++l) {
    const long long num = Bp * (den + (long long)taper_permille * ((n - 1) - 2 * l));
    const long long c = num / den;
    budgets_host[l] = (int32_t)c;
    given += c;
  }
  long long rest = n * Bp - given;
  for (long long l = 0; l < n && rest > 0; ++l, --rest) budgets_host[l] += 1;
  for (long long l = 0; l < n; ++l) budgets_host[l] += window;
  return MIXKV_OK;
}

int mixkv_compress_layer(const void* K, const void* V, const void* Qwin,
                         const int32_t* cu_seqlens_host, int32_t batch, int32_t L,
                         const mixkv_params* p, void* workspace, size_t workspace_bytes,
                         const float* rbar_in_opt, void* K_out, void* V_out,
                         int32_t* out_row_offsets, int32_t* idx_opt, int32_t* counts_opt,
                         int32_t* idx_offsets_opt, float* s_comp_opt, int32_t* status_dev,
                         void* stream) {
  return mixkv_compress_layer_traced(K, V, Qwin, cu_seqlens_host, batch, L, p, workspace,
                                     workspace_bytes, rbar_in_opt, K_out, V_out, out_row_offsets,
                                     idx_opt, counts_opt, idx_offsets_opt, s_comp_opt, status_dev,
                                     stream, nullptr, 0);
}

// ---- the no-allocation variant of mixkv_scores -------------------------------------------
// Scratch for callers that cannot allocate: part of the library's device image, one copy per
// GPU that loads the library.  In host code the name g_static_scratch is only a handle for
// cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[MIXKV_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device; looked up once per device.
int static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MIXKV_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return MIXKV_ERR_CUDA;
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return MIXKV_OK;
}
}  // namespace

int mixkv_scores_static(const void* K, const void* V, const void* Qwin,
                        const int32_t* cu_seqlens_host, int32_t batch, int32_t L,
                        const mixkv_params* p, float* s_comp, float* s_ex_opt, float* s_div_opt,
                        float* rbar_opt, const float* rbar_in_opt, int32_t* status_dev,
                        void* stream) {
  // size the problem on the host first: too large a problem is refused before anything is
  // enqueued (only attribute queries have run by then)
  {
    int rc = check_params(p);
    if (rc != MIXKV_OK) return rc;
    SeqTable st;
    int max_len = 0;
    rc = build_table(p, cu_seqlens_host, batch, L, 1, &st, &max_len);
    if (rc != MIXKV_OK) return rc;
    Workspace ws;
    carve(p, st, nullptr, &ws);
    if (ws.bytes > (size_t)MIXKV_STATIC_SCRATCH_BYTES) return MIXKV_ERR_STATIC_SCRATCH_EXCEEDED;
  }
  void* scratch = nullptr;
  int rc = static_scratch(&scratch);
  if (rc != MIXKV_OK) return rc;
  return mixkv_scores(K, V, Qwin, cu_seqlens_host, batch, L, p, scratch,
                      (size_t)MIXKV_STATIC_SCRATCH_BYTES, s_comp, s_ex_opt, s_div_opt, rbar_opt,
                      rbar_in_opt, status_dev, stream);
}

namespace {
// Whether a call of this shape takes the fused tail (what tail_can_fuse decides at launch).
bool fused_route(const mixkv_params* p, int n_layers, int batch, int max_seq_len) {
  LaunchCtx c;
  memset(&c, 0, sizeof(c));
  c.st.layers = n_layers;
  c.st.batch = batch;
  c.st.H = p->kv_heads;
  c.max_prefix = max_seq_len - p->window;
  return p->budget_mode == MIXKV_BUDGET_FIXED && tail_can_fuse(c);
}
}  // namespace

int mixkv_launches_for(const mixkv_params* p, int32_t n_layers, int32_t batch,
                       int32_t max_seq_len) {
  if (!p || n_layers < 1 || batch < 1 || max_seq_len <= p->window) return 0;
  const char* names[8];
  return layer_stages(p, fused_route(p, n_layers, batch, max_seq_len), names);
}

const char* mixkv_stage_name_for(const mixkv_params* p, int32_t n_layers, int32_t batch,
                                 int32_t max_seq_len, int32_t i) {
  if (!p || n_layers < 1 || batch < 1 || max_seq_len <= p->window) return nullptr;
  const char* names[8];
  const int n = layer_stages(p, fused_route(p, n_layers, batch, max_seq_len), names);
  return (i >= 0 && i < n) ? names[i] : nullptr;
}

int mixkv_device_check(int32_t* cc_major_opt) {
  int major = 0;
  const int rc = device_check(&major);
  if (cc_major_opt) *cc_major_opt = major;
  return rc;
}

const char* mixkv_stage_name(const mixkv_params* p, int32_t i) {
  if (!p) return nullptr;
  const char* names[8];
  const int n = layer_stages(p, true, names);
  return (i >= 0 && i < n) ? names[i] : nullptr;
}

int mixkv_launches_per_layer(const mixkv_params* p) {
  if (!p) return 0;
  const char* names[8];
  return layer_stages(p, true, names);
}

const char* mixkv_status_string(int status) {
  switch (status) {
    case MIXKV_OK: return "ok";
    case MIXKV_ERR_INVALID_ARG: return "invalid argument";
    case MIXKV_ERR_UNSUPPORTED: return "unsupported configuration";
    case MIXKV_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MIXKV_ERR_CUDA: return "CUDA error";
    case MIXKV_ERR_TIMEOUT: return "device-side bounded wait expired";
    case MIXKV_ERR_STATIC_SCRATCH_EXCEEDED:
      return "problem needs more scratch than the built-in array of the no-allocation entry point";
    default: return "unknown status";
  }
}

}  // extern "C"
