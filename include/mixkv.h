/*
 * mixkv.h -- C ABI of the B200 (sm_100a) MixKV prefill KV-cache compression library.
 *
 * The library implements one step of LVLM / LLM inference: at the end of prefill, for
 * one transformer layer, score every cached key of every KV head, keep the best B per
 * head and copy the kept K/V rows into a compact cache (MixKV, arxiv 2510.20707,
 * Sec. 3.1 "KV Cache Compression", Sec. 3.2-3.3, Algorithm 1).
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 *  - All tensor pointers are DEVICE pointers unless the name ends in `_host`.
 *    bf16 tensors must be 16-byte aligned, fp32 / int32 tensors 4-byte aligned.
 *  - The caller owns every buffer, including the workspace.  The library allocates no
 *    device memory and never synchronises the stream: every call only enqueues kernels
 *    on `stream` (a cudaStream_t passed as void*; NULL is the default stream).  Host
 *    state kept between calls is limited to per-device caches of attributes (SM count,
 *    compute capability, shared-memory opt-in).  The workspace needs no initialisation
 *    and no clearing between calls (every word a kernel reads was written earlier in the
 *    same call; nothing is counted across CTAs), and may be reused for other shapes; two
 *    calls that may overlap in time need a workspace each.
 *  - Shapes.  H = kv_heads, G = gqa_ratio, d = head_dim (128), W = window.
 *      K, V      [H, Ltot, d] bf16, row-major.  Ltot = L for one sequence, else
 *                cu_seqlens_host[batch]; sequence b owns rows cu[b] .. cu[b+1]-1.
 *      Qwin      [batch, H*G, W, d] bf16: the last W prompt queries (post-RoPE) of every
 *                query head; query head q attends KV head q / G.  Window row j sits at
 *                sequence position P + j (P = L - W) and sees keys 0 .. P + j.
 *      scores    [H, Ptot] fp32, Ptot = Ltot - batch*W: the P_b = L_b - W candidate
 *                (non-window) positions of sequence b start at column cu[b] - b*W.
 *      rbar      [batch, H] fp32.
 *  - cu_seqlens_host: HOST pointer to batch+1 ascending int32 offsets, read during the
 *    call (not retained).  NULL means one sequence of length L (batch must be 1).
 *  - Return value: 0 on success, a negative mixkv_status otherwise.  Argument errors
 *    (INVALID_ARG, UNSUPPORTED, WORKSPACE_TOO_SMALL) enqueue nothing; MIXKV_ERR_CUDA means a
 *    launch failed, earlier kernels of the call may already be enqueued and the outputs are
 *    undefined.  A device whose compute capability is not 10.x gives MIXKV_ERR_UNSUPPORTED (the
 *    kernels use tcgen05 / tensor memory; see mixkv_device_check).  Conditions only the
 *    device can see (a bounded wait inside a kernel expired) are written to *status_dev
 *    (device int32, optional, must be zeroed by the caller) as MIXKV_ERR_TIMEOUT; kernels
 *    never trap.
 *  - CUDA graphs: a call may be recorded into a stream capture and replayed, provided the
 *    same entry point ran once on that device outside capture (its first use sets function
 *    attributes); the host arrays (cu_seqlens_host) are read at capture time only.
 *  - Limits: head_dim == 128; 16 <= G*W <= 240 and G*W % 16 == 0; batch <= 64;
 *    every sequence needs L_b >= W + 1; budget > W; odd pool_kernel <= 63.
 */
#ifndef MIXKV_H_
#define MIXKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MIXKV_OK = 0,
  MIXKV_ERR_INVALID_ARG = -1,
  MIXKV_ERR_UNSUPPORTED = -2,
  MIXKV_ERR_WORKSPACE_TOO_SMALL = -3,
  MIXKV_ERR_CUDA = -4,
  MIXKV_ERR_TIMEOUT = -5,
  MIXKV_ERR_STATIC_SCRATCH_EXCEEDED = -6
} mixkv_status;

enum { MIXKV_MIX_HEADWISE = 0, MIXKV_MIX_IMPORTANCE_ONLY = 1, MIXKV_MIX_DIVERSITY_ONLY = 2,
       MIXKV_MIX_PLAIN_SUM = 3 };
enum { MIXKV_POOL_AVG = 0, MIXKV_POOL_MAX = 1 };
enum { MIXKV_BUDGET_FIXED = 0, MIXKV_BUDGET_ADAPTIVE = 1 };
enum { MIXKV_INTRINSIC_NONE = 0, MIXKV_INTRINSIC_VNORM = 1, MIXKV_INTRINSIC_KNORM = 2 };

typedef struct mixkv_params {
  int32_t kv_heads;     /* H */
  int32_t gqa_ratio;    /* G: query heads per KV head */
  int32_t head_dim;     /* d: must be 128 */
  int32_t window;       /* W: observation window, paper default 32 (Sec. 3.2) */
  int32_t pool_kernel;  /* odd k >= 1; 1-D pooling of the attention score, 1 = none */
  int32_t pool_mode;    /* MIXKV_POOL_AVG (zero padded, divides by k) or MIXKV_POOL_MAX */
  int32_t use_vnorm;    /* intrinsic importance added in Eq. 2: MIXKV_INTRINSIC_VNORM (value norm,
                           the paper's default), _KNORM (minus the key norm: the KNorm variant of
                           Sec. 3.2 and of the ablation table), _NONE */
  int32_t mix_mode;     /* MIXKV_MIX_*: Eq. 5, or one of the ablation variants of Table 4 */
  int32_t budget_mode;  /* MIXKV_BUDGET_FIXED: B per head; _ADAPTIVE: B*H per sequence */
  int32_t budget;       /* B: rows kept per head INCLUDING the W window rows (Alg. 1) */
  float ada_floor;      /* adaptive: fraction of B - W guaranteed to every head (0..1) */
  float eps;            /* epsilon of the two min-max normalisations (Sec. 3.2, 3.3) */
  float softmax_scale;  /* 0 => 1/sqrt(d) */
} mixkv_params;

/* Fills *p with the paper's defaults: W 32, average pooling k 7, VNorm on, Eq. 5 mixing,
 * fixed budget, ada_floor 0.2, eps 1e-6, scale 1/sqrt(d).  Sets H, G and B as given. */
void mixkv_default_params(mixkv_params* p, int32_t kv_heads, int32_t gqa_ratio, int32_t budget);

/* Bytes of device workspace the three entry points below need for a batch whose sequence
 * lengths sum to total_tokens (max single length max_seq_len).  Host-only; no CUDA call. */
int mixkv_workspace_size(const mixkv_params* p, int32_t batch, int64_t total_tokens,
                         int32_t max_seq_len, size_t* bytes);

/* The same for a call that handles n_layers layers at once (mixkv_compress_layers). */
int mixkv_workspace_size_layers(const mixkv_params* p, int32_t n_layers, int32_t batch,
                                int64_t total_tokens, int32_t max_seq_len, size_t* bytes);

/* Scores of every candidate key (Sec. 3.2-3.3; Algorithm 1 step 1 and the mixing of step 2):
 *   s_ex   = pool_k( sum over the G query heads of the mean over the W window rows of the
 *            causal softmax attention weight on key i )             (extrinsic importance)
 *   s_imp  = s_ex + VNorm_i min-max normalised, rescaled to mean(s_ex)            (Eq. 2)
 *   s_div  = - cos(K_i, mean over all L keys of the unit keys)                  (diversity)
 *   rbar   = (L^2 |mean unit key|^2 - L) / (L (L-1))                            (Eq. 3-4)
 *   s_comp = (1 - rbar) s_imp + rbar * (s_div min-max normalised, rescaled to mean(s_imp))
 *                                                                                 (Eq. 5)
 * Key geometry (mean unit key, rbar) uses all L keys of the sequence; score vectors and
 * their min / max / mean use the P candidate positions.
 *   s_comp        out, required, [H, Ptot]
 *   s_ex_opt      out, optional (NULL to skip), pooled attention score [H, Ptot]
 *   s_div_opt     out, optional, raw diversity score [H, Ptot]
 *   rbar_opt      out, optional, [batch, H]
 *   rbar_in_opt   in, optional, [batch, H]: redundancy to mix with instead of the computed
 *                 one (head weights calibrated offline, Sec. 4.3)
 *   V may be NULL unless use_vnorm == MIXKV_INTRINSIC_VNORM. */
int mixkv_scores(const void* K, const void* V, const void* Qwin,
                 const int32_t* cu_seqlens_host, int32_t batch, int32_t L,
                 const mixkv_params* p, void* workspace, size_t workspace_bytes,
                 float* s_comp, float* s_ex_opt, float* s_div_opt, float* rbar_opt,
                 const float* rbar_in_opt, int32_t* status_dev, void* stream);

/* mixkv_scores for callers that cannot obtain device memory for a workspace (the paper has
 * no counterpart; this is a packaging variant of mixkv_scores, same kernels, same results).
 * Typical users: a serving engine that hands every free byte of HBM to its own paged KV pool
 * at start-up, so that a later cudaMalloc fails or fragments the pool; a plug-in running
 * inside somebody else's step loop, where cudaMalloc / cudaFree would stall the whole device
 * with their implicit synchronisation; a host language binding that can pass pointers it
 * was given but owns no allocator.  Such callers still pass their inputs and outputs; only
 * the scratch the kernels need between them comes from the library: a fixed array of
 * MIXKV_STATIC_SCRATCH_BYTES that lives in the library's device image, so every GPU that
 * loads the library sets that much memory aside until the process exits.
 *  - Problems whose workspace (mixkv_workspace_size) would exceed the array are refused with
 *    MIXKV_ERR_STATIC_SCRATCH_EXCEEDED before anything is enqueued (the size is worked out on
 *    the host; the only CUDA calls before the refusal are attribute queries).  As a guide the array covers
 *    about 128k (head, token) pairs, e.g. H = 4 at L = 32768 or H = 8 at L = 16384.
 *  - The call performs no cudaMalloc / cudaFree and calls no allocating library routine.
 *  - The first call on each device looks up the array's device address (once per device, with
 *    that device current) and keeps it for later calls; make that first call outside any
 *    stream capture.  The kept address does not survive cudaDeviceReset: a process that resets
 *    a device must not call this entry point on it afterwards.
 *  - All calls on one device share the one array, and it keeps whatever the previous call
 *    left in it.  Nothing in it needs to start from zero (every cell is written before it is
 *    read inside a call), but two calls whose kernels overlap on the GPU (different streams
 *    without an ordering between them) race on it: order such calls yourself.
 * Arguments are those of mixkv_scores without workspace / workspace_bytes. */
#define MIXKV_STATIC_SCRATCH_BYTES (12u << 20)
int mixkv_scores_static(const void* K, const void* V, const void* Qwin,
                        const int32_t* cu_seqlens_host, int32_t batch, int32_t L,
                        const mixkv_params* p, float* s_comp, float* s_ex_opt, float* s_div_opt,
                        float* rbar_opt, const float* rbar_in_opt, int32_t* status_dev,
                        void* stream);

/* TopB of Sec. 3.1 / Algorithm 1 on caller-supplied scores [H, Ptot]: per (sequence, head)
 * the b_h highest scores among the P_b candidates, ties to the lower position, written in
 * ascending position order.  b_h = min(B - W, P_b) for fixed budgets.  Adaptive budgets
 * (per sequence): every head is guaranteed f = floor(ada_floor * (B - W)); the remaining
 * H * (B - W - f) slots go to the highest scores of the H heads taken together (ties to the
 * lower (head, position)); b_h = min(f + share_h, P_b).
 *   idx          out, packed in (b, h) order; capacity batch * H * (B - W) int32 is always
 *                enough
 *   counts       out, [batch * H], b_h
 *   idx_offsets  out, [batch * H + 1], exclusive prefix sum of counts
 * status_dev is accepted for symmetry and never written: the kernels of this entry point
 * contain no bounded waits. */
int mixkv_select(const float* scores, const int32_t* cu_seqlens_host, int32_t batch, int32_t L,
                 const mixkv_params* p, void* workspace, size_t workspace_bytes,
                 int32_t* idx, int32_t* counts, int32_t* idx_offsets,
                 int32_t* status_dev, void* stream);

/* The whole per-layer step of Algorithm 1: mixkv_scores, mixkv_select, then the gather:
 * for every (b, h) the selected rows of K and V in ascending position order followed by the
 * W window rows, packed in (b, h) order.
 *   K_out, V_out      out, [rows, d] bf16; capacity batch * H * B rows is always enough
 *   out_row_offsets   out, [batch * H + 1]: first output row of each (b, h); last = rows
 *   idx_opt / counts_opt / idx_offsets_opt / s_comp_opt   optional outputs as above (NULL:
 *                     kept in the workspace) */
int mixkv_compress_layer(const void* K, const void* V, const void* Qwin,
                         const int32_t* cu_seqlens_host, int32_t batch, int32_t L,
                         const mixkv_params* p, void* workspace, size_t workspace_bytes,
                         const float* rbar_in_opt, void* K_out, void* V_out,
                         int32_t* out_row_offsets, int32_t* idx_opt, int32_t* counts_opt,
                         int32_t* idx_offsets_opt, float* s_comp_opt,
                         int32_t* status_dev, void* stream);

/* Measurement hook (no counterpart in the paper): mixkv_compress_layer with CUDA events
 * recorded on `stream` around its kernels.  events_host is a HOST array of n_events
 * cudaEvent_t handles created by the caller with timing enabled: events_host[i] is recorded
 * just before the i-th kernel and events_host[k] after the last of the k kernels
 * (k = mixkv_launches_per_layer); entries beyond n_events are skipped, so n_events = 2
 * brackets the first kernel only.  Everything else is as mixkv_compress_layer. */
int mixkv_compress_layer_traced(const void* K, const void* V, const void* Qwin,
                                const int32_t* cu_seqlens_host, int32_t batch, int32_t L,
                                const mixkv_params* p, void* workspace, size_t workspace_bytes,
                                const float* rbar_in_opt, void* K_out, void* V_out,
                                int32_t* out_row_offsets, int32_t* idx_opt, int32_t* counts_opt,
                                int32_t* idx_offsets_opt, float* s_comp_opt,
                                int32_t* status_dev, void* stream,
                                void* const* events_host, int32_t n_events);

/* mixkv_compress_layer for n_layers layers of identical shape in ONE set of kernel launches
 * (Algorithm 1's "for each layer l and head h" loop taken whole): a serving engine that keeps the
 * prefill KV of all layers resident can compress them together at the end of prefill, which
 * spreads the per-launch costs over all layers and keeps every SM busy in the selection and
 * gather step.  The layers are an outer batch dimension; each is processed exactly as
 * mixkv_compress_layer would.
 *   K, V              [n_layers, H, Ltot, d] bf16; kv_layer_stride = elements between the
 *                     tensors of consecutive layers (0: packed, H * Ltot * d; otherwise a
 *                     multiple of 8 and at least that)
 *   Qwin              [n_layers, batch, H*G, W, d] bf16; q_layer_stride likewise (0: packed)
 *   rbar_in_opt       optional, [n_layers, batch, H]
 *   K_out, V_out      [n_layers, batch * H * B, d]: layer l starts at row l * batch * H * B and
 *                     is packed inside its slice as mixkv_compress_layer packs it
 *   out_row_offsets   [n_layers, batch * H + 1], rows relative to the layer's slice
 *   idx_opt           [n_layers, cap], cap = sum over sequences of H * min(B - W, P_b)
 *   counts_opt        [n_layers, batch * H];  idx_offsets_opt [n_layers, batch * H + 1]
 *   s_comp_opt        [n_layers, H, Ptot]
 *   workspace         mixkv_workspace_size_layers bytes
 *   events_host       optional measurement hook as in mixkv_compress_layer_traced (NULL, 0: off)
 * n_layers <= 1024. */
int mixkv_compress_layers(const void* K, const void* V, const void* Qwin, int32_t n_layers,
                          int64_t kv_layer_stride, int64_t q_layer_stride,
                          const int32_t* cu_seqlens_host, int32_t batch, int32_t L,
                          const mixkv_params* p, void* workspace, size_t workspace_bytes,
                          const float* rbar_in_opt, void* K_out, void* V_out,
                          int32_t* out_row_offsets, int32_t* idx_opt, int32_t* counts_opt,
                          int32_t* idx_offsets_opt, float* s_comp_opt, int32_t* status_dev,
                          void* stream, void* const* events_host, int32_t n_events);

/* mixkv_compress_layers with the budgets chosen outside the library: the paper plugs its scores
 * into compressors that differ only in how many rows a layer or a head may keep (Section 4.1 and
 * the related-work appendix: PyramidKV gives lower layers more than higher ones, SparseMM / HeadKV
 * give every head its own static share).  Scores, selection and gather are exactly those of
 * mixkv_compress_layers; only the number of candidates taken per head comes from the caller.
 *   head_budgets   device, [n_layers, batch * H] int32: rows to keep for that (layer, sequence,
 *                  head), window included.  A value is used as min(max(v - W, 0), B - W, P_b)
 *                  selected candidates plus the W window rows; p->budget (B) is the largest
 *                  budget any head may get and sizes the outputs as in mixkv_compress_layers.
 *   p->budget_mode must be MIXKV_BUDGET_FIXED (else MIXKV_ERR_INVALID_ARG).
 * Outputs are ragged as with adaptive budgets: rows of (b, h) start at out_row_offsets[l][b*H+h]
 * of layer l's slice; counts_opt receives the candidates actually selected. */
int mixkv_compress_layers_budgeted(const void* K, const void* V, const void* Qwin,
                                   int32_t n_layers, int64_t kv_layer_stride,
                                   int64_t q_layer_stride, const int32_t* cu_seqlens_host,
                                   int32_t batch, int32_t L, const mixkv_params* p,
                                   void* workspace, size_t workspace_bytes,
                                   const float* rbar_in_opt, const int32_t* head_budgets,
                                   void* K_out, void* V_out, int32_t* out_row_offsets,
                                   int32_t* idx_opt, int32_t* counts_opt, int32_t* idx_offsets_opt,
                                   float* s_comp_opt, int32_t* status_dev, void* stream);

/* Host-side layer schedule in the manner of PyramidKV (named in the paper's related work; the
 * paper gives no formula, this is the build's reading): budgets fall linearly with depth and
 * their sum stays n_layers * budget.  With B' = budget - window candidates per head and
 * t = taper_permille / 1000 (0 <= taper_permille <= 999), layer l of n gets
 * floor(B' * (1 + t * (1 - 2 l / (n - 1)))) candidates; the candidates lost to rounding go to
 * the lowest layers, one each; window is added back.  budgets_host [n_layers] (host memory)
 * receives the rows to keep per head of each layer: layer 0 gets the most.  Fill a
 * [n_layers, batch * H] array with them for mixkv_compress_layers_budgeted and pass
 * budgets_host[0] as p->budget.  No device work. */
int mixkv_layer_budget_schedule(int32_t n_layers, int32_t budget, int32_t window,
                                int32_t taper_permille, int32_t* budgets_host);

/* Redundancy analysis: the pairwise cosine similarity of the keys (or values) of a head, which
 * the paper plots as heat maps and summarises per head (Sec. 1, Sec. 3.1, the redundancy
 * figures), at block resolution.
 *   X          device, [heads, L, head_dim] bf16, 16-byte aligned (head_dim must be 128)
 *   block      rows per map cell (>= 1); T = ceil(L / block) cells per side (T <= 65535)
 *   cells      device, [heads, T, T] fp32: mean of cos(x_i, x_j) over i in block I, j in block J,
 *              pairs i == j left out (a diagonal cell averages n (n - 1) pairs, 0 if n == 1)
 *   mean_opt   device, [heads] fp32 or NULL: mean over all ordered pairs i != j of the head,
 *              the redundancy of Eq. 4
 *   workspace  device, mixkv_similarity_workspace_size bytes, 16-byte aligned, caller-owned
 * A zero row has cosine 0 with every row.  Two routes: for block = 1, 2, 4, 8 or 16 the dense
 * matrix X^ X^T of Eq. 3 is formed on the tensor cores (rows normalised once into two bf16
 * halves, upper triangle of 128 x 128 tiles, cells reduced in the epilogue); for every other
 * block size the cells come from the Gram matrix of the per-block sums of unit rows (one
 * streaming pass over X).  The workspace size depends on the route.  Errors as for the other
 * entry points. */
int mixkv_similarity_workspace_size(int32_t heads, int32_t L, int32_t block, size_t* bytes);
int mixkv_similarity_map(const void* X, int32_t heads, int32_t L, int32_t head_dim, int32_t block,
                         void* workspace, size_t workspace_bytes, float* cells, float* mean_opt,
                         void* stream);

/* The step after compression: one new query token per sequence attends over the compact cache
 * that mixkv_compress_layers wrote (paper Sec. 3.1: decoding continues on the compressed K, V),
 * all layers in one launch.  softmax(q . K^T * scale) V per query head over the rows kept for
 * its KV head, fp32 accumulation.
 *   K_cache, V_cache   device, [n_layers, rows_cap, d] bf16: K_out / V_out of the compression
 *   out_row_offsets    device, [n_layers, batch * H + 1]: rows of (b, h) inside a layer's slice
 *   rows_cap           rows between the slices of consecutive layers (batch * H * B)
 *   q                  device, [n_layers, batch, H * G, d] bf16: the token's query per layer
 *   max_rows           upper bound on the rows of one (layer, b, h), e.g. B, or L for a cache
 *                      that was not compressed; rows beyond it are not read.  It only steers
 *                      how many CTAs share one head (the warps of a cluster of 1, 2, 4 or 8
 *                      CTAs take the rows 16 at a time, each with a running softmax), so any
 *                      length is accepted
 *   out                device, [n_layers, batch, H * G, d] fp32; a head without rows gets zeros
 * softmax_scale 0 means 1 / sqrt(d).  d must be 128, G <= 16 (else MIXKV_ERR_UNSUPPORTED). */
int mixkv_decode_attention(const void* K_cache, const void* V_cache,
                           const int32_t* out_row_offsets, int64_t rows_cap, const void* q,
                           int32_t n_layers, int32_t batch, int32_t kv_heads, int32_t gqa_ratio,
                           int32_t head_dim, float softmax_scale, int32_t max_rows, float* out,
                           void* stream);

/* Number of kernels one mixkv_compress_layer[s] call enqueues, and the name of the i-th of
 * them (NULL when i is out of range), for the measurement hook.  The route depends on the
 * shape: fixed budgets take three kernels (pass1, pass2, tail; max pooling adds poolsum) while
 * the candidates of the longest sequence fit the tail kernel's shared memory (P_b <= 131072)
 * and add the unfused mix kernel beyond that; adaptive budgets always take the unfused route
 * with the budget kernel.  The _for variants take the shape and follow the route the call
 * takes; the short forms assume the fused route where it exists. */
int mixkv_launches_per_layer(const mixkv_params* p);
const char* mixkv_stage_name(const mixkv_params* p, int32_t i);
int mixkv_launches_for(const mixkv_params* p, int32_t n_layers, int32_t batch,
                       int32_t max_seq_len);
const char* mixkv_stage_name_for(const mixkv_params* p, int32_t n_layers, int32_t batch,
                                 int32_t max_seq_len, int32_t i);

/* Whether the current device can run the library (no counterpart in the paper): MIXKV_OK for
 * compute capability 10.x, MIXKV_ERR_UNSUPPORTED for any other device, MIXKV_ERR_CUDA when no
 * device can be queried.  *cc_major_opt receives the major compute capability (0 when unknown).
 * Every enqueueing entry point performs the same check (cached per device). */
int mixkv_device_check(int32_t* cc_major_opt);

/* Diagnostic (no counterpart in the paper): enqueues a one-CTA kernel that waits, through the
 * same bounded-wait helper as the pass kernels, on a barrier nothing arrives on.  After the
 * wait limit (2 s) the kernel writes MIXKV_ERR_TIMEOUT to *status_dev and, if waited_ns_dev is
 * not NULL, the time it waited; it never traps and the context stays usable.  For tests of the
 * error path. */
int mixkv_selftest_bounded_wait(int32_t* status_dev, unsigned long long* waited_ns_dev,
                                void* stream);

/* Static, human-readable name of a status code. */
const char* mixkv_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MIXKV_H_ */
