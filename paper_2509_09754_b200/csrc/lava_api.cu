// C ABI of liblava: argument validation, workspace layout, dispatch to the kernel launchers.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>

#include "lava_internal.cuh"

namespace lava {

static thread_local char g_error[512] = "";
static std::atomic<long long> g_launches{0};

void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

lava_status fail(lava_status st, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_error, sizeof(g_error), fmt, ap);
  va_end(ap);
  return st;
}

lava_status check_cuda(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return LAVA_OK;
  return fail(LAVA_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

static long long env_ll(const char* name, long long lo, long long hi, long long dflt) {
  const char* e = getenv(name);
  if (!e || !*e) return dflt;
  const long long v = atoll(e);
  return (v < lo || v > hi) ? dflt : v;
}

Options& options() {
  static Options opt = [] {
    Options o;
    o.select_cluster = (int)env_ll("LAVA_SELECT_CLUSTER", 8, 16, 0);
    if (o.select_cluster != 8 && o.select_cluster != 16) o.select_cluster = 0;
    o.score_chunk_tiles = (int)env_ll("LAVA_SM100_CHUNK_TILES", 1, 64, 0);
    o.score_lead_tiles = (int)env_ll("LAVA_SM100_LEAD_TILES", 0, 4096, -1);
    o.force_generic = (int)env_ll("LAVA_FORCE_GENERIC", 0, 1, 0);
    o.score_kernel = (int)env_ll("LAVA_SCORE_KERNEL", 0, 2, 0);
    o.wait_limit_cycles = env_ll("LAVA_WAIT_LIMIT_CYCLES", 1, 1ll << 40, 1ll << 32);
    return o;
  }();
  return opt;
}

int sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  cached[dev].store(n, std::memory_order_relaxed);
  return n;
}


static size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

lava_status make_geom(const lava_layer_desc* d, Geom* out) {
  if (!d) return fail(LAVA_ERR_INVALID_ARG, "desc is NULL");
  if (d->n_kv_heads < 1 || d->n_q_heads < 1 || d->n_q_heads % d->n_kv_heads != 0)
    return fail(LAVA_ERR_INVALID_ARG, "n_q_heads (%d) must be a positive multiple of n_kv_heads (%d)",
                d->n_q_heads, d->n_kv_heads);
  if (d->n_kv_heads > 128) return fail(LAVA_ERR_UNSUPPORTED, "n_kv_heads > 128");
  if (d->head_dim != 64 && d->head_dim != 128)
    return fail(LAVA_ERR_UNSUPPORTED, "head_dim must be 64 or 128 (got %d)", d->head_dim);
  if (d->window < 1) return fail(LAVA_ERR_INVALID_ARG, "window must be >= 1");
  if (d->window > 128) return fail(LAVA_ERR_UNSUPPORTED, "window > 128");
  if (d->pool_kind < LAVA_POOL_NONE || d->pool_kind > LAVA_POOL_AVG)
    return fail(LAVA_ERR_INVALID_ARG, "unknown pool_kind %d", d->pool_kind);
  if (d->pool_kind != LAVA_POOL_NONE &&
      (d->pool_kernel < 1 || d->pool_kernel > 63 || d->pool_kernel % 2 == 0))
    return fail(LAVA_ERR_INVALID_ARG, "pool_kernel must be odd and in 1..63 (got %d)",
                d->pool_kernel);
  if (d->dtype != LAVA_F32 && d->dtype != LAVA_BF16)
    return fail(LAVA_ERR_INVALID_ARG, "unknown dtype %d", d->dtype);
  if (d->batch < 1) return fail(LAVA_ERR_INVALID_ARG, "batch must be >= 1");
  if (d->batch > 1 && !d->cu_seqlens)
    return fail(LAVA_ERR_INVALID_ARG, "cu_seqlens is required when batch > 1");
  if (d->flags < 0 || d->flags > 7) return fail(LAVA_ERR_INVALID_ARG, "unknown bits in flags");
  if ((d->flags & LAVA_FLAG_UNIT_VALUE_NORM) && (d->flags & LAVA_FLAG_TOKEN_VALUE_NORM))
    return fail(LAVA_ERR_INVALID_ARG, "the unit and the per-token value term exclude each other");
  if (d->total_tokens < (int64_t)d->batch * d->window)
    return fail(LAVA_ERR_INVALID_ARG, "total_tokens (%lld) < batch*window: every sequence needs "
                "at least `window` tokens", (long long)d->total_tokens);
  if (d->total_tokens > 0x7fffffffLL / d->n_kv_heads)
    return fail(LAVA_ERR_UNSUPPORTED, "H_kv * total_tokens must fit in 31 bits");
  if (d->max_seqlen < 0 || d->max_seqlen > d->total_tokens)
    return fail(LAVA_ERR_INVALID_ARG, "max_seqlen out of range");
  const int64_t strides[4] = {d->k_stride_head, d->k_stride_tok, d->v_stride_head, d->v_stride_tok};
  for (int i = 0; i < 4; ++i)
    if (strides[i] < d->head_dim && (i % 2 == 1))
      return fail(LAVA_ERR_INVALID_ARG, "token stride smaller than head_dim");
  for (int i = 0; i < 4; ++i)
    if (strides[i] < 0 || strides[i] % 8 != 0)
      return fail(LAVA_ERR_INVALID_ARG, "strides must be non-negative multiples of 8 elements");
  if (!(d->sm_scale >= 0.f) || !(d->c_hat >= 0.f) || isinf(d->sm_scale) || isinf(d->c_hat))
    return fail(LAVA_ERR_INVALID_ARG, "sm_scale and c_hat must be finite and >= 0");

  Geom g;
  g.n_q_heads = d->n_q_heads;
  g.n_kv_heads = d->n_kv_heads;
  g.group = d->n_q_heads / d->n_kv_heads;
  g.head_dim = d->head_dim;
  g.window = d->window;
  g.w_pad = (d->window + 15) / 16 * 16;
  g.pool_kind = (d->pool_kind != LAVA_POOL_NONE && d->pool_kernel <= 1) ? LAVA_POOL_NONE
                                                                       : d->pool_kind;
  g.pool_kernel = d->pool_kernel;
  g.pool_radius = g.pool_kind == LAVA_POOL_NONE ? 0 : d->pool_kernel / 2;
  g.dtype = d->dtype;
  g.batch = d->batch;
  g.max_seqlen = d->max_seqlen > 0 ? d->max_seqlen : (int)d->total_tokens;
  g.flags = d->flags;
  g.cu_seqlens = d->cu_seqlens;
  g.total_tokens = d->total_tokens;
  g.total_scores = (long long)d->n_kv_heads * (d->total_tokens - (long long)d->batch * d->window);
  g.k_sh = d->k_stride_head;
  g.k_st = d->k_stride_tok;
  g.v_sh = d->v_stride_head;
  g.v_st = d->v_stride_tok;
  const double scale = d->sm_scale > 0.f ? (double)d->sm_scale : 1.0 / sqrt((double)d->head_dim);
  g.scale_log2 = (float)(scale * 1.4426950408889634);
  g.c_hat = d->c_hat > 0.f ? d->c_hat : 1.0f;
  *out = g;
  return LAVA_OK;
}

Workspace workspace_layout(const lava_layer_desc* d, int n_layers) {
  Workspace w;
  const int max_seqlen = d->max_seqlen > 0 ? d->max_seqlen : (int)d->total_tokens;
  const size_t problems = (size_t)n_layers * d->batch;
  w.n_slices = ceil_div(max_seqlen, Workspace::kSlice);
  w.n_vslices = ceil_div(max_seqlen, Workspace::kVSlice);
  size_t off = Workspace::kStatusBytes;
  w.off_vpart = off;
  off = round_up(off + problems * d->n_kv_heads * w.n_vslices * sizeof(float), 256);
  w.off_stats = off;
  off = round_up(off + problems * d->n_q_heads * w.n_slices * d->window * sizeof(float2), 256);
  w.off_lse = off;
  off = round_up(off + problems * d->n_q_heads * d->window * sizeof(float), 256);
  w.off_vbar = off;
  off = round_up(off + problems * d->n_kv_heads * sizeof(float), 256);
  w.off_ones = off;
  off = round_up(off + problems * d->n_kv_heads * sizeof(float), 256);
  w.off_ent = off;
  off = round_up(off + problems * d->n_kv_heads * w.n_slices * sizeof(double2), 256);
  w.off_sm100 = off;
  Geom g;
  const bool tensor_path = make_geom(d, &g) == LAVA_OK && sm100_supported(g);
  if (tensor_path) off += sm100_layout(g, n_layers).total;
  w.off_tmem = off;
  if (tensor_path && tmem_supported(g)) off += tmem_layout(g, n_layers).total;
  w.total = off;
  return w;
}

}  // namespace lava

using namespace lava;

extern "C" {

int32_t lava_version(void) { return 100; }

int64_t lava_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int32_t lava_score_path(const lava_layer_desc* desc) {
  Geom g;
  if (make_geom(desc, &g) != LAVA_OK) return -1;
  if (!sm100_supported(g) || options().force_generic) return 0;
  return g.group * g.window > 128 ? 2 : 1;
}

const char* lava_last_error(void) { return g_error; }

static long long* option_slot(const char* name, long long* lo, long long* hi, int** as_int) {
  Options& o = options();
  *as_int = nullptr;
  if (!name) return nullptr;
  if (!strcmp(name, "select_cluster")) { *lo = 0; *hi = 16; *as_int = &o.select_cluster; }
  else if (!strcmp(name, "score_chunk_tiles")) { *lo = 0; *hi = 64; *as_int = &o.score_chunk_tiles; }
  else if (!strcmp(name, "score_lead_tiles")) { *lo = -1; *hi = 4096; *as_int = &o.score_lead_tiles; }
  else if (!strcmp(name, "force_generic")) { *lo = 0; *hi = 1; *as_int = &o.force_generic; }
  else if (!strcmp(name, "score_kernel")) { *lo = 0; *hi = 2; *as_int = &o.score_kernel; }
  else if (!strcmp(name, "wait_limit_cycles")) { *lo = 1; *hi = 1ll << 40; return &o.wait_limit_cycles; }
  return nullptr;
}

lava_status lava_set_option(const char* name, int64_t value) {
  long long lo = 0, hi = 0;
  int* as_int = nullptr;
  long long* slot = option_slot(name, &lo, &hi, &as_int);
  if (!slot && !as_int) return fail(LAVA_ERR_INVALID_ARG, "unknown option '%s'", name ? name : "(null)");
  if (value < lo || value > hi || (as_int == &options().select_cluster && value != 0 && value != 8 && value != 16))
    return fail(LAVA_ERR_INVALID_ARG, "option %s: value %lld out of range", name, (long long)value);
  if (as_int) *as_int = (int)value; else *slot = value;
  return LAVA_OK;
}

int64_t lava_get_option(const char* name) {
  long long lo = 0, hi = 0;
  int* as_int = nullptr;
  long long* slot = option_slot(name, &lo, &hi, &as_int);
  if (as_int) return *as_int;
  if (slot) return *slot;
  fail(LAVA_ERR_INVALID_ARG, "unknown option '%s'", name ? name : "(null)");
  return INT64_MIN;
}

size_t lava_workspace_bytes(const lava_layer_desc* desc, int32_t n_layers) {
  Geom g;
  if (n_layers < 1 || make_geom(desc, &g) != LAVA_OK) return 0;
  return workspace_layout(desc, n_layers).total;
}

lava_status lava_poll_status(void* workspace, void* stream, uint32_t* device_status_out) {
  if (!workspace || !device_status_out) return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  cudaStream_t st = (cudaStream_t)stream;
  uint32_t word = 0;
  lava_status rc = check_cuda(cudaMemcpyAsync(&word, workspace, sizeof(word),
                                              cudaMemcpyDeviceToHost, st), "status copy");
  if (rc != LAVA_OK) return rc;
  rc = check_cuda(cudaMemsetAsync(workspace, 0, sizeof(word), st), "status clear");
  if (rc != LAVA_OK) return rc;
  rc = check_cuda(cudaStreamSynchronize(st), "stream synchronize");
  if (rc != LAVA_OK) return rc;
  *device_status_out = word;
  if (word & LAVA_DEV_WAIT_EXPIRED) return fail(LAVA_ERR_TIMEOUT, "a bounded device wait expired");
  return LAVA_OK;
}

lava_status lava_wo_norm(const void* w_o, int32_t dtype, int64_t rows, int64_t cols,
                         float* c_hat_out, void* stream) {
  if (!w_o || !c_hat_out) return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  if (dtype != LAVA_F32 && dtype != LAVA_BF16) return fail(LAVA_ERR_INVALID_ARG, "unknown dtype");
  if (rows < 1 || cols < 1) return fail(LAVA_ERR_INVALID_ARG, "rows and cols must be positive");
  return launch_wo_norm(w_o, dtype, rows, cols, c_hat_out, (cudaStream_t)stream);
}

lava_status lava_score_layers(const lava_layer_desc* desc, int32_t n_layers, const void* q_win,
                              const void* k, const void* v, int64_t q_layer_stride,
                              int64_t k_layer_stride, int64_t v_layer_stride,
                              const float* vbar_in, float* scores, float* vbar_out,
                              double* entropy, void* workspace, size_t workspace_bytes,
                              void* stream) {
  Geom g;
  lava_status rc = make_geom(desc, &g);
  if (rc != LAVA_OK) return rc;
  if (n_layers < 1) return fail(LAVA_ERR_INVALID_ARG, "n_layers must be >= 1");
  if (!q_win || !k || !entropy || (!scores && g.total_scores > 0))
    return fail(LAVA_ERR_INVALID_ARG, "q_win, k, scores and entropy are required");
  const bool unit_term = (g.flags & (LAVA_FLAG_UNIT_VALUE_NORM | LAVA_FLAG_TOKEN_VALUE_NORM)) != 0;
  const bool token_term = (g.flags & LAVA_FLAG_TOKEN_VALUE_NORM) != 0;
  if (!v && !vbar_in && !(unit_term && !token_term))
    return fail(LAVA_ERR_INVALID_ARG, "v may be NULL only if vbar_in is given");
  if (unit_term && vbar_in)
    return fail(LAVA_ERR_INVALID_ARG, "vbar_in must be NULL with a value-term flag");
  if (token_term && !v) return fail(LAVA_ERR_INVALID_ARG, "the per-token value term needs v");
  if (!aligned16(q_win) || !aligned16(k) || (v && !aligned16(v)) || !aligned16(scores))
    return fail(LAVA_ERR_INVALID_ARG, "q_win, k, v and scores must be 16-byte aligned");
  if (n_layers > 1 && (q_layer_stride % 8 || k_layer_stride % 8 || v_layer_stride % 8 ||
                       q_layer_stride < 0 || k_layer_stride < 0 || v_layer_stride < 0))
    return fail(LAVA_ERR_INVALID_ARG, "layer strides must be non-negative multiples of 8");
  const Workspace lay = workspace_layout(desc, n_layers);
  if (!workspace) return fail(LAVA_ERR_WORKSPACE, "workspace is NULL");
  if (workspace_bytes < lay.total)
    return fail(LAVA_ERR_WORKSPACE, "workspace too small: %zu < %zu bytes", workspace_bytes,
                lay.total);
  if (!aligned16(workspace)) return fail(LAVA_ERR_INVALID_ARG, "workspace must be 16-byte aligned");
  cudaStream_t st = (cudaStream_t)stream;
  const void* v_used = v;
  if (unit_term) {
    // the score kernels run with a value-norm array of ones and never touch V
    float* ones = reinterpret_cast<float*>((char*)workspace + lay.off_ones);
    rc = launch_fill_ones(ones, (long long)n_layers * g.batch * g.n_kv_heads, st);
    if (rc != LAVA_OK) return rc;
    vbar_in = ones;
    v_used = nullptr;
  }
  if (sm100_supported(g) && !options().force_generic) {
    // the single-pass kernel (exponentials kept in tensor memory) is opt-in: the exchange of row
    // statistics between the CTAs outlasts what six exponent buffers can cover, so it is the
    // slower of the two today
    if (options().score_kernel == 2 && tmem_supported(g) && tmem_fits(g, tmem_grid(g, n_layers)))
      rc = launch_score_tmem(g, n_layers, q_win, k, v_used, q_layer_stride, k_layer_stride,
                             v_layer_stride, vbar_in, scores, vbar_out, entropy,
                             (char*)workspace, lay.off_tmem, st);
    else
      rc = launch_score_sm100(g, n_layers, q_win, k, v_used, q_layer_stride, k_layer_stride,
                              v_layer_stride, vbar_in, scores, vbar_out, entropy,
                              (char*)workspace, lay.off_sm100, st);
  } else {
    rc = launch_score_generic(g, n_layers, q_win, k, v_used, q_layer_stride, k_layer_stride,
                              v_layer_stride, vbar_in, scores, vbar_out, entropy,
                              (char*)workspace, lay, st);
  }
  if (rc != LAVA_OK || !token_term) return rc;
  // VATP: every position's own value-row norm, then the entropy of the final scores
  rc = launch_token_norm_scale(g, n_layers, v, v_layer_stride, scores, st);
  if (rc != LAVA_OK) return rc;
  return launch_entropy_from_scores(g, n_layers, scores, entropy, st);
}

lava_status lava_score_layer(const lava_layer_desc* desc, const void* q_win, const void* k,
                             const void* v, const float* vbar_in, float* scores,
                             float* vbar_out, double* entropy, void* workspace,
                             size_t workspace_bytes, void* stream) {
  return lava_score_layers(desc, 1, q_win, k, v, 0, 0, 0, vbar_in, scores, vbar_out, entropy,
                           workspace, workspace_bytes, stream);
}

lava_status lava_layer_budgets(int32_t n_layers, int32_t batch, const double* entropy,
                               const int64_t* total_budget, const int64_t* floor_per_layer,
                               const int64_t* cap_per_layer, int32_t mode,
                               int64_t* layer_budget, int64_t* layer_row_offset,
                               uint32_t* status_word, void* stream) {
  if (n_layers < 1 || n_layers > 256) return fail(LAVA_ERR_UNSUPPORTED, "n_layers must be in 1..256");
  if (batch < 1 || batch > 1024) return fail(LAVA_ERR_UNSUPPORTED, "batch must be in 1..1024");
  if (!entropy || !total_budget || !floor_per_layer || !cap_per_layer || !layer_budget ||
      !layer_row_offset)
    return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  if (mode < 0 || (mode & 0xff) > LAVA_BUDGET_PYRAMID || (mode >> 8) > 1000 ||
      ((mode >> 8) != 0 && (mode & 0xff) != LAVA_BUDGET_PYRAMID))
    return fail(LAVA_ERR_INVALID_ARG, "unknown budget mode %d", mode);
  return launch_budgets(n_layers, batch, entropy, (const long long*)total_budget,
                        (const long long*)floor_per_layer, (const long long*)cap_per_layer, mode,
                        (long long*)layer_budget, (long long*)layer_row_offset, status_word,
                        (cudaStream_t)stream);
}

lava_status lava_select_topk_layers(const lava_layer_desc* desc, int32_t n_layers,
                                    const float* scores, const int64_t* layer_budget,
                                    int32_t* keep_idx, int32_t* head_offsets, void* workspace,
                                    size_t workspace_bytes, void* stream) {
  Geom g;
  lava_status rc = make_geom(desc, &g);
  if (rc != LAVA_OK) return rc;
  if (n_layers < 1) return fail(LAVA_ERR_INVALID_ARG, "n_layers must be >= 1");
  if (!layer_budget || !head_offsets || ((!scores || !keep_idx) && g.total_scores > 0))
    return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  if ((long long)n_layers * g.batch > 65535)
    return fail(LAVA_ERR_UNSUPPORTED, "n_layers*batch must be <= 65535");
  (void)workspace_bytes;
  return launch_select(g, n_layers, scores, (const long long*)layer_budget, keep_idx, head_offsets,
                       (unsigned*)workspace, (cudaStream_t)stream);
}

lava_status lava_select_topk(const lava_layer_desc* desc, const float* scores,
                             const int64_t* layer_budget, int32_t* keep_idx,
                             int32_t* head_offsets, void* workspace, size_t workspace_bytes,
                             void* stream) {
  return lava_select_topk_layers(desc, 1, scores, layer_budget, keep_idx, head_offsets, workspace,
                                 workspace_bytes, stream);
}

lava_status lava_compact_kv_layers(const lava_layer_desc* desc, int32_t n_layers, const void* k,
                                   const void* v, int64_t k_layer_stride, int64_t v_layer_stride,
                                   const int32_t* keep_idx, const int32_t* head_offsets,
                                   const int64_t* layer_row_offset, void* k_out, void* v_out,
                                   void* stream) {
  Geom g;
  lava_status rc = make_geom(desc, &g);
  if (rc != LAVA_OK) return rc;
  if (n_layers < 1) return fail(LAVA_ERR_INVALID_ARG, "n_layers must be >= 1");
  if (!k || !v || !head_offsets || !layer_row_offset || !k_out || !v_out ||
      (!keep_idx && g.total_scores > 0))
    return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  if (!aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out))
    return fail(LAVA_ERR_INVALID_ARG, "k, v, k_out and v_out must be 16-byte aligned");
  if ((long long)n_layers * g.batch > 65535)
    return fail(LAVA_ERR_UNSUPPORTED, "n_layers*batch must be <= 65535");
  return launch_compact(g, n_layers, k, v, k_layer_stride, v_layer_stride, keep_idx, head_offsets,
                        (const long long*)layer_row_offset, k_out, v_out, (cudaStream_t)stream);
}

lava_status lava_compact_kv(const lava_layer_desc* desc, const void* k, const void* v,
                            const int32_t* keep_idx, const int32_t* head_offsets,
                            const int64_t* layer_row_offset, void* k_out, void* v_out,
                            void* stream) {
  return lava_compact_kv_layers(desc, 1, k, v, 0, 0, keep_idx, head_offsets, layer_row_offset,
                                k_out, v_out, stream);
}

}  // extern "C"
