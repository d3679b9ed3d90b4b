/*
 * lava.h -- C ABI of the LAVa prefill-time KV-cache eviction hot path for NVIDIA B200 (sm_100a).
 *
 * The library scores every cached (KV head, position) entry of a layer with the LAVa metric,
 * turns per-layer score entropies into integer layer budgets, selects the layer-wide top-k
 * (which yields per-head budgets) and gathers the retained K/V rows into a packed cache.
 *
 * Conventions that hold for every function unless its comment says otherwise:
 *   - Every data pointer is a caller-owned DEVICE pointer.  The library never allocates or
 *     frees device memory and never synchronises the device; all work is enqueued on `stream`
 *     (a cudaStream_t passed as void*, NULL = the legacy default stream).
 *   - Pointers must be 16-byte aligned, token rows contiguous (`head_dim` elements), strides
 *     are in elements and multiples of 8.
 *   - Functions return a lava_status.  Arguments are validated on the host before any launch;
 *     on error nothing is enqueued and lava_last_error() describes the problem.  No C++
 *     exception crosses this boundary.
 *   - Failures that only the device can see (a sequence shorter than the window, an
 *     infeasible budget, an expired bounded wait) set bits in the status word at the start
 *     of the workspace; read it with lava_poll_status().
 *
 * Positions are 0-based.  For a sequence of n tokens and window w, P = n - w is the number of
 * prefix candidates; the window is positions P..n-1 and is always retained (constraints of
 * Eq. 1).  "Head" in budgets and offsets means KV head.
 *
 * Score layout (one layer):  sequence b, KV head g, prefix position i lives at
 *      H_kv * (cu_seqlens[b] - b*w)  +  g * P_b  +  i
 * so one sequence's scores form one contiguous flat array of H_kv*P_b floats, heads in order.
 * A layer has  total_scores = H_kv * (total_tokens - batch*w)  entries.
 */
#ifndef LAVA_H_
#define LAVA_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define LAVA_API __attribute__((visibility("default")))
#else
#define LAVA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lava_status {
  LAVA_OK = 0,
  LAVA_ERR_INVALID_ARG = 1,  /* null / misaligned pointer, bad geometry */
  LAVA_ERR_UNSUPPORTED = 2,  /* valid request outside what the kernels cover */
  LAVA_ERR_WORKSPACE = 3,    /* workspace missing or smaller than lava_workspace_bytes() */
  LAVA_ERR_CUDA = 4,         /* a CUDA runtime call or launch failed */
  LAVA_ERR_TIMEOUT = 5       /* a bounded device-side wait expired (reported by poll) */
} lava_status;

typedef enum lava_dtype { LAVA_F32 = 0, LAVA_BF16 = 1 } lava_dtype;
typedef enum lava_pool { LAVA_POOL_NONE = 0, LAVA_POOL_MAX = 1, LAVA_POOL_AVG = 2 } lava_pool;
typedef enum lava_budget_mode {
  LAVA_BUDGET_DYNAMIC = 0,  /* Algorithm 2: shares e_l / sum e                                   */
  LAVA_BUDGET_UNIFORM = 1,  /* "- layer dynamic" / LAVa-Uniform of the ablation (Sec. 5.4): B / L   */
  LAVA_BUDGET_PYRAMID = 2   /* LAVa-Pyramid of the layer-allocation comparison: the PyramidKV line
                               B_{L-1} = B / (beta L), B_0 = 2B/L - B_{L-1}, descending with depth;
                               beta = mode >> 8 (0 means 20): pass LAVA_BUDGET_PYRAMID | beta << 8   */
} lava_budget_mode;

/* Bits of the device status word. */
#define LAVA_DEV_SHORT_SEQUENCE 1u    /* some sequence has fewer than `window` tokens: the score
                                         layout has no room for it, so the score, select and
                                         compact kernels of such a batch do nothing at all (the
                                         host can only check total_tokens >= batch*window)      */
#define LAVA_DEV_BUDGET_INFEASIBLE 2u /* total budget outside [L*floor, L*cap]; was clamped  */
#define LAVA_DEV_WAIT_EXPIRED 4u      /* a bounded wait inside a kernel gave up              */
#define LAVA_DEV_BAD_SEQLEN 8u        /* some sequence is longer than desc->max_seqlen       */

/* Variants of the method (the ablation of Sec. 5.4 and the score functions of the methods the
 * paper compares with).  0 is LAVa as published. */
#define LAVA_FLAG_PER_HEAD_TOPK 1u    /* "- head dynamic": every KV head keeps its even share of the
                                         layer budget, no comparison across heads (lava_select_topk) */
#define LAVA_FLAG_UNIT_VALUE_NORM 2u  /* SnapKV / AdaKV score: value term 1 instead of Vbar; V is not
                                         read and may be NULL (lava_score_layer)                     */
#define LAVA_FLAG_TOKEN_VALUE_NORM 4u /* VATP score: ||V_g[i]||_1 of every position instead of Vbar
                                         (lava_score_layer; vbar_in must be NULL)                    */

/* Geometry of one layer (all layers of a model share it).  Plain data, caller-owned (host). */
typedef struct lava_layer_desc {
  int32_t n_q_heads;   /* H_q, a multiple of n_kv_heads                                     */
  int32_t n_kv_heads;  /* H_kv                                                              */
  int32_t head_dim;    /* d_h: 64 or 128                                                    */
  int32_t window;      /* w >= 1: observation window = last w tokens of each sequence       */
  int32_t pool_kind;   /* lava_pool                                                         */
  int32_t pool_kernel; /* odd, 1..63; ignored for LAVA_POOL_NONE                            */
  int32_t dtype;       /* lava_dtype of Q, K, V and of the compacted output                 */
  int32_t batch;       /* number of sequences (>= 1)                                        */
  int32_t max_seqlen;  /* upper bound on any sequence length (0 => total_tokens)            */
  int32_t flags;       /* LAVA_FLAG_* bits, 0 for the paper's method                        */
  const int32_t* cu_seqlens; /* device int32 [batch+1] token offsets; NULL => batch == 1    */
  int64_t total_tokens;      /* sum of sequence lengths                                     */
  int64_t k_stride_head, k_stride_tok; /* K[g][tok][c] = k[g*k_stride_head + tok*k_stride_tok + c] */
  int64_t v_stride_head, v_stride_tok;
  float sm_scale;      /* logit scale; 0 => 1/sqrt(head_dim)                                */
  float c_hat;         /* optional ||W_O^T||_1 factor of Theorem 1; 0 => 1.  Multiplies every
                          score of the layer, so it changes no budget and no selection.     */
} lava_layer_desc;

/* Library / error plumbing ------------------------------------------------------------- */
LAVA_API int32_t lava_version(void);            /* major*10000 + minor*100 + patch                  */
LAVA_API const char* lava_last_error(void);     /* thread-local text of the last failure, never NULL */

/* Bytes of device scratch that the score and select calls need for `n_layers` layers of this
 * geometry processed in one call.  The first 256 bytes hold the status word; the caller
 * should zero the workspace once after allocating it. */
LAVA_API size_t lava_workspace_bytes(const lava_layer_desc* desc, int32_t n_layers);

/* Synchronises `stream`, copies the status word to *device_status_out (host) and clears it.
 * Returns LAVA_ERR_TIMEOUT if LAVA_DEV_WAIT_EXPIRED is set, LAVA_OK otherwise. */
LAVA_API lava_status lava_poll_status(void* workspace, void* stream, uint32_t* device_status_out);

/* C-hat of Theorem 1: the largest absolute row sum of W_O ([rows, cols], row-major, device,
 * LAVA_F32 or LAVA_BF16) written to *c_hat_out (device float). */
LAVA_API lava_status lava_wo_norm(const void* w_o, int32_t dtype, int64_t rows, int64_t cols,
                         float* c_hat_out, void* stream);

/* Step 1 -- LAVa score of one layer (Definition 1 with pooling and the GQA group maximum).
 *   For each query head h (KV head g = h / G), window query t at position P+t:
 *     A_{h,t} = softmax over keys i <= P+t of sm_scale * q_{h,t} . k_{g,i}        (Sec. 2)
 *     a_h[i]  = (1/w) sum_t A_{h,t}[i],  i < P                                   (Definition 1)
 *     pooled_h = pool(a_h), stride 1, centred, over the prefix only               (Sec. 5.1)
 *     Vbar_g  = max over all n rows of the row L1 norm of V_g                     (Theorem 1)
 *     s_g[i]  = c_hat * Vbar_g * max_{h in g} pooled_h[i]                         (Sec. 4.3)
 *   and the layer uncertainty  e = -sum(s_hat ln s_hat) / (H_kv * n),  s_hat = s / sum(s)
 *   over the sequence's flat score array (normalised score and entropy equations, Sec. 4.2).
 *
 *   q_win    [batch, H_q, w, d]  the last w queries of every sequence (post-RoPE), contiguous
 *   k, v     per the strides in desc; v may be NULL iff vbar_in != NULL
 *   vbar_in  [batch, H_kv] value norms supplied by the caller, or NULL to compute them from v
 *   scores   out, float [total_scores] in the layout described at the top of this file
 *   vbar_out out, float [batch, H_kv], may be NULL
 *   entropy  out, double [batch]
 * Outputs are fully overwritten; bytes beyond the stated sizes are never touched. */
LAVA_API lava_status lava_score_layer(const lava_layer_desc* desc, const void* q_win, const void* k,
                             const void* v, const float* vbar_in, float* scores,
                             float* vbar_out, double* entropy, void* workspace,
                             size_t workspace_bytes, void* stream);

/* The same for n_layers layers in one call.  Layer l reads q_win + l*q_layer_stride,
 * k + l*k_layer_stride, v + l*v_layer_stride (strides in elements) and writes
 * scores + l*total_scores, vbar_out + l*batch*H_kv, entropy + l*batch.  vbar_in, when given,
 * is [n_layers, batch, H_kv]. */
LAVA_API lava_status lava_score_layers(const lava_layer_desc* desc, int32_t n_layers, const void* q_win,
                              const void* k, const void* v, int64_t q_layer_stride,
                              int64_t k_layer_stride, int64_t v_layer_stride,
                              const float* vbar_in, float* scores, float* vbar_out,
                              double* entropy, void* workspace, size_t workspace_bytes,
                              void* stream);

/* The score step of one layer for callers that cannot allocate device memory (no counterpart
 * in the paper: it exists for the callers, not for the method).
 *
 * Who needs it: code that runs inside another framework's memory pool without access to its
 * allocator, plugins whose host forbids device allocations after start-up, and serving loops
 * that must not risk the stall an allocation can cause.  Such a caller has inputs and outputs
 * but no spare buffer to pass as `workspace`.  Here the scratch is a fixed 8 MiB array inside
 * the library image; every GPU that loads the library holds it until the process exits.
 *
 * Same computation, same arguments and same results as lava_score_layer, minus the workspace:
 *   device_status_out  DEVICE uint32, may be NULL: receives the status word of this call
 *                      (LAVA_DEV_* bits) once `stream` has run past the call
 * Limits and rules:
 *   - A layer whose lava_workspace_bytes(desc, 1) exceeds 8 MiB is rejected with
 *     LAVA_ERR_WORKSPACE before anything is enqueued (about 128K tokens at 32/8 heads, d 128).
 *   - The first call on a device looks up the array's device address (a host-side set-up step,
 *     once per device, with that device current); make that first call before any stream
 *     capture begins.
 *   - All calls share the one array, and it keeps the contents of the previous call; the entry
 *     point clears what must start at zero itself.  Two calls whose kernels overlap on the GPU
 *     (different streams, or different host threads on the same device) race on it: keep calls
 *     on one device ordered on one stream.
 *   - It calls no allocator: no cudaMalloc/cudaFree, no allocating library routine. */
LAVA_API lava_status lava_score_layer_static(const lava_layer_desc* desc, const void* q_win,
                                    const void* k, const void* v, const float* vbar_in,
                                    float* scores, float* vbar_out, double* entropy,
                                    uint32_t* device_status_out, void* stream);

/* Step 2 -- layer budgets (Algorithm 2: B_l = e_l / sum_l e_l * B), made integral.
 *   entropy          double [n_layers, batch]
 *   total_budget     int64 [batch]: model-wide budget of each sequence in KV-head rows,
 *                    window rows included
 *   floor_per_layer  int64 [batch]: H_kv * w      cap_per_layer  int64 [batch]: H_kv * n_b
 *   mode             lava_budget_mode (uniform and pyramid ignore the entropies)
 *   layer_budget     out int64 [n_layers, batch], sums to total_budget[b] over layers
 *   layer_row_offset out int64 [n_layers*batch + 1]: exclusive prefix sums of layer_budget in
 *                    (layer, sequence) order = first row of each (layer, sequence) in the
 *                    packed cache
 *   status_word      device uint32 that receives LAVA_DEV_BUDGET_INFEASIBLE (may be NULL;
 *                    normally the workspace pointer)
 * Rule: shares proportional to e_l are rounded by largest remainder (ties to the lower layer);
 * layers outside [floor, cap] are clamped one side at a time (the side with the larger total
 * violation, the floor side on a tie) and the rest is re-shared among the remaining layers.
 * n_layers <= 256, batch <= 1024. */
LAVA_API lava_status lava_layer_budgets(int32_t n_layers, int32_t batch, const double* entropy,
                               const int64_t* total_budget, const int64_t* floor_per_layer,
                               const int64_t* cap_per_layer, int32_t mode,
                               int64_t* layer_budget, int64_t* layer_row_offset,
                               uint32_t* status_word, void* stream);

/* Step 3 -- layer-wide top-k (Algorithm 1, Evict): of a sequence's H_kv*P_b prefix scores keep
 * the  layer_budget[b] - H_kv*w  largest; equal scores are taken in ascending flat index.
 *   scores        float [total_scores]
 *   layer_budget  int64 [batch] (this layer's row of lava_layer_budgets' output)
 *   keep_idx      out int32 [total_scores]: sequence b's kept prefix positions start at the
 *                 sequence's score offset, head after head, ascending within a head; only the
 *                 first (layer_budget[b] - H_kv*w) entries of the segment are written
 *   head_offsets  out int32 [batch, H_kv+1]: exclusive scan of rows per head (kept prefix
 *                 rows + w window rows); head_offsets[b][H_kv] == min(layer_budget[b], H_kv*n_b)
 * The per-head differences of head_offsets are the dynamic head budgets. */
LAVA_API lava_status lava_select_topk(const lava_layer_desc* desc, const float* scores,
                             const int64_t* layer_budget, int32_t* keep_idx,
                             int32_t* head_offsets, void* workspace, size_t workspace_bytes,
                             void* stream);

/* n_layers layers in one launch: scores/keep_idx advance by total_scores per layer,
 * layer_budget by batch, head_offsets by batch*(H_kv+1). */
LAVA_API lava_status lava_select_topk_layers(const lava_layer_desc* desc, int32_t n_layers,
                                    const float* scores, const int64_t* layer_budget,
                                    int32_t* keep_idx, int32_t* head_offsets, void* workspace,
                                    size_t workspace_bytes, void* stream);

/* Step 4 -- gather and compact (Algorithm 1: K-hat = K (.) I, V-hat = V (.) I as a gather).
 * For sequence b and head g the rows  layer_row_offset[b] + head_offsets[b][g] ...  of k_out /
 * v_out receive, bit for bit, the kept prefix rows in ascending position followed by the w
 * window rows.
 *   layer_row_offset  int64 [batch]: this layer's entries of lava_layer_budgets' output
 *   k_out, v_out      packed caches [rows, head_dim] of the input dtype
 * Rows outside the ranges above are not written. */
LAVA_API lava_status lava_compact_kv(const lava_layer_desc* desc, const void* k, const void* v,
                            const int32_t* keep_idx, const int32_t* head_offsets,
                            const int64_t* layer_row_offset, void* k_out, void* v_out,
                            void* stream);

/* n_layers layers in one launch (k, v advance by the layer strides; keep_idx by total_scores;
 * head_offsets by batch*(H_kv+1); layer_row_offset by batch). */
LAVA_API lava_status lava_compact_kv_layers(const lava_layer_desc* desc, int32_t n_layers, const void* k,
                                   const void* v, int64_t k_layer_stride, int64_t v_layer_stride,
                                   const int32_t* keep_idx, const int32_t* head_offsets,
                                   const int64_t* layer_row_offset, void* k_out, void* v_out,
                                   void* stream);

/* Host-buffer path -- one full-model eviction (steps 1-4 over all layers) for callers whose
 * Q window, K and V live in HOST memory (pinned memory gives asynchronous copies).
 * Layer l is copied to the device on an internal copy stream while layer l-1 is being scored
 * on `stream`; budgets, selection and compaction follow, and the results are copied back.
 * Everything is asynchronous with respect to the host: the host buffers must stay valid, and
 * the outputs are complete, once `stream` has been synchronised by the caller.
 *   desc              geometry; desc->cu_seqlens is ignored (sequence lengths come from
 *                     seq_lens), strides are ignored (host arrays are dense)
 *   q_win, k, v       HOST, dense [L, batch, H_q, w, d] and [L, H_kv, total_tokens, d]
 *   seq_lens          HOST int32 [batch]
 *   total_budget      HOST int64 [batch]
 *   layer_budget      HOST out int64 [L, batch]
 *   head_offsets      HOST out int32 [L, batch, H_kv+1]
 *   k_out, v_out      HOST out packed caches [sum(total_budget), d]
 *   arena             DEVICE scratch of at least lava_host_arena_bytes() bytes, 256-byte
 *                     aligned; holds the staged inputs, all intermediates and the packed cache
 * The first call on a device creates one internal stream and a few events (host resources). */
LAVA_API size_t lava_host_arena_bytes(const lava_layer_desc* desc, int32_t n_layers,
                                      int64_t total_budget_rows);
LAVA_API lava_status lava_evict_model_host(const lava_layer_desc* desc, int32_t n_layers,
                                           const void* q_win, const void* k, const void* v,
                                           const int32_t* seq_lens, const int64_t* total_budget,
                                           int32_t mode, int64_t* layer_budget,
                                           int32_t* head_offsets, void* k_out, void* v_out,
                                           void* arena, size_t arena_bytes, void* stream);

/* Layer-by-layer form of the method (Algorithm 2 and the paragraph after it): prefill and evict
 * one layer at a time, so that only one layer's full K/V is ever alive.  After layer l has been
 * scored, the budgets of layers 0..l are recomputed from e_0..e_l out of the total in force
 * (the model's total, held inside [(l+1)*floor, (l+1)*cap] while few layers are live), layer l
 * is evicted from its full K/V, and every lower layer is evicted again from what it still holds
 * with the scores stored at its first eviction; only the retained scores are stored.  A second
 * eviction can only drop entries, so the final cache equals the one-shot result of
 * lava_layer_budgets / lava_select_topk / lava_compact_kv whenever no layer's budget ever grows
 * from one step to the next.
 *
 *   lava_cascade_state_bytes  bytes of DEVICE memory the caller must provide as `state` for
 *                     n_layers layers and an arena of total_rows packed rows (>= the sum of the
 *                     sequences' total budgets).  Holds the packed K and V rows twice (each step
 *                     writes the shrunken layout into the other copy), the held scores and
 *                     positions twice, and one layer's full score and index arrays.
 *   lava_cascade_create   validates and makes the HOST-side handle (owned by the caller, freed
 *                     with lava_cascade_destroy; it owns no device memory).  `desc` is copied;
 *                     desc->cu_seqlens and `state` must stay valid while the handle is used.
 *                     mode is LAVA_BUDGET_DYNAMIC or LAVA_BUDGET_UNIFORM; LAVA_FLAG_PER_HEAD_TOPK
 *                     is not supported here.  At most 524288 candidates per (layer, sequence).
 *   lava_cascade_begin    total_budget: DEVICE int64 [batch], the model-wide budgets in rows.
 *                     A total outside [L*floor, L*cap], or totals that exceed total_rows, are
 *                     replaced by feasible ones and LAVA_DEV_BUDGET_INFEASIBLE is set in the
 *                     status word of `workspace`.  Restarts the handle at layer 0.
 *   lava_cascade_step     takes the next layer: q_win, k, v (and optional vbar_in) exactly as
 *                     lava_score_layer, workspace of lava_workspace_bytes(desc, 1) bytes.  K and V
 *                     of this layer may be released once the work enqueued here has finished.
 *                     A step that returns an error leaves the handle unusable until the next
 *                     lava_cascade_begin.
 *   lava_cascade_get      device pointers into `state` for the layers taken so far (valid until
 *                     the next step): rows and list entries of (layer l, sequence b) start at
 *                     layer_row_offset[l*batch + b]; inside, head g's rows start at
 *                     head_offsets[l][b][g] (kept prefix rows in ascending position, then the w
 *                     window rows) and its kept positions / scores are list entries
 *                     head_offsets[l][b][g] - g*w ... of that segment. */
typedef struct lava_cascade lava_cascade;
typedef struct lava_cascade_view {
  int32_t layers_done;
  void* k_out;                     /* packed rows [total_rows, d]                               */
  void* v_out;
  const int32_t* kept_pos;         /* [total_rows] positions of the kept prefix entries          */
  const float* kept_scores;        /* [total_rows] their scores                                  */
  const int32_t* head_offsets;     /* [layers_done, batch, H_kv+1]                               */
  const int64_t* layer_budget;     /* [layers_done, batch]                                       */
  const int64_t* layer_row_offset; /* [layers_done*batch + 1]                                    */
  const double* entropy;           /* [layers_done, batch]                                       */
} lava_cascade_view;
LAVA_API size_t lava_cascade_state_bytes(const lava_layer_desc* desc, int32_t n_layers,
                                         int64_t total_rows);
LAVA_API lava_status lava_cascade_create(const lava_layer_desc* desc, int32_t n_layers,
                                         int64_t total_rows, int32_t mode, void* state,
                                         size_t state_bytes, lava_cascade** out);
LAVA_API void lava_cascade_destroy(lava_cascade* h);
LAVA_API lava_status lava_cascade_begin(lava_cascade* h, const int64_t* total_budget,
                                        void* workspace, void* stream);
LAVA_API lava_status lava_cascade_step(lava_cascade* h, const void* q_win, const void* k,
                                       const void* v, const float* vbar_in, void* workspace,
                                       size_t workspace_bytes, void* stream);
LAVA_API lava_status lava_cascade_get(const lava_cascade* h, lava_cascade_view* out);

/* Consumer of the packed cache: the attention of one new token per sequence over the retained
 * rows (Sec. 2 attention restricted to K-hat, V-hat of Algorithm 1).  After the layer-wide
 * selection every KV head holds its own number of rows; query head h reads KV head
 * g = h / (H_q / H_kv):   out[h] = softmax_i(sm_scale * q[h] . K-hat_g[i]) V-hat_g.
 *   q                 [n_layers, batch, H_q, d] queries of the new token, dtype desc->dtype
 *   k_packed, v_packed   the packed caches written by lava_compact_kv (or a cascade's k_out, v_out)
 *   head_offsets      [n_layers, batch, H_kv+1] as written by lava_select_topk
 *   layer_row_offset  [n_layers*batch (+1)]
 *   out               float [n_layers, batch, H_q, d]; a head without rows gives zeros
 *   workspace         lava_decode_workspace_bytes(desc, n_layers) bytes (partial results of the
 *                     warps that share a head; unused outside bf16 / d = 128 / group <= 8)
 * bf16 with d = 128 runs on the tensor path with the probabilities rounded to bf16 before they
 * multiply V (error <= 2^-8 * sum_i p_i |V[i][c]| per output); other geometries run a plain
 * fp32 kernel.  lava_decode_attention is the one-layer form (pointers of that layer). */
LAVA_API size_t lava_decode_workspace_bytes(const lava_layer_desc* desc, int32_t n_layers);
LAVA_API lava_status lava_decode_attention_layers(const lava_layer_desc* desc, int32_t n_layers,
                                                  const void* q, const void* k_packed,
                                                  const void* v_packed, const int32_t* head_offsets,
                                                  const int64_t* layer_row_offset, float* out,
                                                  void* workspace, size_t workspace_bytes,
                                                  void* stream);
LAVA_API lava_status lava_decode_attention(const lava_layer_desc* desc, const void* q,
                                           const void* k_packed, const void* v_packed,
                                           const int32_t* head_offsets,
                                           const int64_t* layer_row_offset, float* out,
                                           void* workspace, size_t workspace_bytes, void* stream);

/* Layer-wide selection (Algorithm 1, Evict) with the KV heads of a layer split over several GPUs.
 * Every rank describes its own heads (desc->n_kv_heads = local heads, scores of the local heads in
 * the usual layout) and the ranks agree on one threshold per (layer, sequence).  The library
 * provides the local steps; the caller runs the two small collectives between them:
 *
 *   lava_select_shard_begin(desc, L, total_kv_heads, layer_budget, state)
 *   for pass in 0, 1, 2:
 *       lava_select_shard_hist(desc, L, scores, pass, state)     -- fills the histogram block
 *       all-reduce (sum, uint32) of the histogram block over the ranks
 *       lava_select_shard_step(desc, L, pass, state)             -- same result on every rank
 *   lava_select_shard_count(desc, L, scores, state)              -- fills the tie block
 *   ties_before_rank[p] = sum of the tie blocks of the lower ranks (all-gather + prefix);
 *                         a separate DEVICE int64 [L*batch] array, zeros on rank 0
 *   lava_select_shard_emit(desc, L, scores, ties_before_rank, keep_idx, head_offsets,
 *                          layer_row_offset, state)
 *
 * Heads are ordered by rank, then by local index: equal scores go to the lower rank first, so the
 * union of the ranks' outputs equals lava_select_topk on the unsplit layer.  keep_idx and
 * head_offsets are local (same layout as lava_select_topk for the local desc); layer_row_offset
 * (may be NULL) receives the prefix sums of the LOCAL row counts, ready for lava_compact_kv on the
 * rank's own K/V.  layer_budget is the budget of the whole layer (all ranks pass the same).
 * `state` is DEVICE memory of lava_select_shard_bytes(desc, L) bytes; lava_select_shard_layout
 * gives the byte ranges of the histogram block (uint32 [L*batch][2048]) and of the tie block
 * (int64 [L*batch]) inside it.  No kernel here reads another GPU's memory. */
LAVA_API size_t lava_select_shard_bytes(const lava_layer_desc* desc, int32_t n_layers);
LAVA_API lava_status lava_select_shard_layout(const lava_layer_desc* desc, int32_t n_layers,
                                              size_t* hist_offset, size_t* hist_bytes,
                                              size_t* ties_offset, size_t* ties_bytes);
LAVA_API lava_status lava_select_shard_begin(const lava_layer_desc* desc, int32_t n_layers,
                                             int32_t total_kv_heads, const int64_t* layer_budget,
                                             void* state, size_t state_bytes, void* stream);
LAVA_API lava_status lava_select_shard_hist(const lava_layer_desc* desc, int32_t n_layers,
                                            const float* scores, int32_t pass, void* state,
                                            size_t state_bytes, void* stream);
LAVA_API lava_status lava_select_shard_step(const lava_layer_desc* desc, int32_t n_layers,
                                            int32_t pass, void* state, size_t state_bytes,
                                            void* stream);
LAVA_API lava_status lava_select_shard_count(const lava_layer_desc* desc, int32_t n_layers,
                                             const float* scores, void* state, size_t state_bytes,
                                             void* stream);
LAVA_API lava_status lava_select_shard_emit(const lava_layer_desc* desc, int32_t n_layers,
                                            const float* scores, const int64_t* ties_before_rank,
                                            int32_t* keep_idx, int32_t* head_offsets,
                                            int64_t* layer_row_offset, void* state,
                                            size_t state_bytes, void* stream);

/* Evaluator (not on the eviction path): layer attention output loss of a selection, Lemma 1 with
 * p = 1 for the last token of every sequence, and the upper bound of Theorem 1:
 *     loss[b]  = || Cat_h[ (A_h - A^_h) V_g(h) ] W_O ||_1 ,  A^_h = (A_h (.) I) / ||A_h (.) I||_1
 *     bound[b] = 2 ||W_O^T||_1 sum_h Vbar_g(h) sum_i A_h[i] (1 - I_g(h)[i])
 * where A_h is the softmax attention row of the last token over all keys of its sequence and I
 * marks the retained entries of KV head g(h) (kept prefix positions and the window).
 *   q_win, k, v        one layer, as in lava_score_layer (the last row of the window is the query)
 *   keep_idx, head_offsets   the layer's selection, as written by lava_select_topk
 *   vbar               [batch, H_kv] value norms of the layer (vbar_out of lava_score_layer)
 *   w_o                DEVICE row-major [H_q*d, d_model], dtype w_o_dtype (lava_dtype)
 *   loss_out, bound_out   DEVICE double [batch]
 *   workspace          at least lava_loss_workspace_bytes(desc, d_model) bytes (holds the attention
 *                      rows as doubles: 8*H_q*total_tokens bytes, plus small arrays)
 * Sums are taken in double in a fixed order. */
LAVA_API size_t lava_loss_workspace_bytes(const lava_layer_desc* desc, int64_t d_model);
LAVA_API lava_status lava_layer_output_loss(const lava_layer_desc* desc, const void* q_win,
                                            const void* k, const void* v, const int32_t* keep_idx,
                                            const int32_t* head_offsets, const float* vbar,
                                            const void* w_o, int32_t w_o_dtype, int64_t d_model,
                                            double* loss_out, double* bound_out, void* workspace,
                                            size_t workspace_bytes, void* stream);

/* Tuning and test knobs (no counterpart in the paper).  Process-wide; the defaults come from the
 * environment variables named below, read once when the library first needs an option, so no
 * call on the hot path reads the environment.  Set them while no call of this library is running.
 *   "select_cluster"     0 = choose by size (default), 8 or 16 CTAs per selection cluster
 *                        (LAVA_SELECT_CLUSTER)
 *   "score_kernel"       0 or 1 = two-pass tensor-core kernel (default), 2 = single-pass kernel
 *                        that keeps the exponentials in tensor memory, where the geometry allows
 *                        it (bf16, d 128, pooling kernel <= 9, about 54K tokens; slower today,
 *                        and its stored exponentials are fp16: scores within 3e-4 relative)
 *                        (LAVA_SCORE_KERNEL)
 *   "score_chunk_tiles"  0 = choose per launch, else 1..64 key tiles per chunk of the two-pass
 *                        kernel (LAVA_SM100_CHUNK_TILES)
 *   "score_lead_tiles"   -1 = choose, else extra tiles pass 1 leads pass 2 by (LAVA_SM100_LEAD_TILES)
 *   "force_generic"      1 = score on the CUDA-core path whatever the geometry (LAVA_FORCE_GENERIC)
 *   "wait_limit_cycles"  SM cycles after which a device-side wait on another warp role or CTA
 *                        gives up and sets LAVA_DEV_WAIT_EXPIRED (default 2^32, about two seconds;
 *                        LAVA_WAIT_LIMIT_CYCLES).  Waits for copies already in flight keep the
 *                        default so that a kernel never exits under a running copy.
 * lava_set_option returns LAVA_ERR_INVALID_ARG for an unknown name or a value out of range;
 * lava_get_option returns INT64_MIN for an unknown name. */
LAVA_API lava_status lava_set_option(const char* name, int64_t value);
LAVA_API int64_t lava_get_option(const char* name);

/* Number of kernel launches this library has enqueued from the calling process so far. */
LAVA_API int64_t lava_launch_count(void);

/* Which kernels lava_score_layer(s) will use for this geometry (host-side decision, no device
 * work; honours the "force_generic" option): 0 = CUDA-core path (fp32 inputs, head_dim 64, other
 * windows), 1 = tensor-core path with one 128-row unit per KV head (Definition 1 with the GQA
 * group maximum of Sec. 4.3 taken inside the kernel), 2 = tensor-core path with the query group
 * of a KV head split into two units of at most 128 window-query rows whose maxima are merged
 * in memory.  Returns -1 and sets lava_last_error() for an invalid descriptor. */
LAVA_API int32_t lava_score_path(const lava_layer_desc* desc);

#ifdef __cplusplus
}
#endif
#endif /* LAVA_H_ */
