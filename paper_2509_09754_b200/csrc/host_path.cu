// Host-buffer path: stages a model's Q window / K / V from host memory layer by layer on a copy
// stream while earlier layers are scored, then runs budgets, selection and compaction and
// copies the results back.  Only copies and calls into the device-pointer entry points happen
// here; all arithmetic stays in the kernels.
#include <mutex>
#include <vector>

#include "lava_internal.cuh"

namespace lava {
namespace {

struct HostPathState {
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t start = nullptr;
  std::vector<cudaEvent_t> layer_ready;
};

HostPathState g_state[64];
std::mutex g_state_mutex;  // guards the creation of a device's stream and events

// The host arrays are dense whatever strides the caller's descriptor carries.
void set_dense_layout(lava_layer_desc* d) {
  d->k_stride_tok = d->v_stride_tok = d->head_dim;
  d->k_stride_head = d->v_stride_head = d->total_tokens * d->head_dim;
}

size_t up256(size_t x) { return (x + 255) / 256 * 256; }

struct Arena {
  size_t ws, cu, tb, lo, hi, q, k, v, scores, vbar, ent, budget, rowoff, keep, hoff, k_out, v_out,
      total;
  size_t ws_bytes, q_layer, kv_layer;  // bytes
};

Arena arena_layout(const lava_layer_desc* d, int n_layers, long long rows) {
  Arena a;
  const size_t es = d->dtype == LAVA_BF16 ? 2 : 4;
  const size_t problems = (size_t)n_layers * d->batch;
  const size_t total_scores =
      (size_t)d->n_kv_heads * (size_t)(d->total_tokens - (long long)d->batch * d->window);
  lava_layer_desc one = *d;
  // sizes do not read the offsets; batches need a non-null pointer to pass validation
  one.cu_seqlens = d->batch > 1 ? reinterpret_cast<const int32_t*>(16) : nullptr;
  a.ws_bytes = workspace_layout(&one, 1).total;
  a.q_layer = (size_t)d->batch * d->n_q_heads * d->window * d->head_dim * es;
  a.kv_layer = (size_t)d->n_kv_heads * d->total_tokens * d->head_dim * es;
  size_t off = 0;
  a.ws = off;      off = up256(off + a.ws_bytes);
  a.cu = off;      off = up256(off + sizeof(int) * (d->batch + 1));
  a.tb = off;      off = up256(off + sizeof(long long) * d->batch);
  a.lo = off;      off = up256(off + sizeof(long long) * d->batch);
  a.hi = off;      off = up256(off + sizeof(long long) * d->batch);
  a.q = off;       off = up256(off + a.q_layer * n_layers);
  a.k = off;       off = up256(off + a.kv_layer * n_layers);
  a.v = off;       off = up256(off + a.kv_layer * n_layers);
  a.scores = off;  off = up256(off + sizeof(float) * total_scores * n_layers);
  a.vbar = off;    off = up256(off + sizeof(float) * problems * d->n_kv_heads);
  a.ent = off;     off = up256(off + sizeof(double) * problems);
  a.budget = off;  off = up256(off + sizeof(long long) * problems);
  a.rowoff = off;  off = up256(off + sizeof(long long) * (problems + 1));
  a.keep = off;    off = up256(off + sizeof(int) * total_scores * n_layers);
  a.hoff = off;    off = up256(off + sizeof(int) * problems * (d->n_kv_heads + 1));
  a.k_out = off;   off = up256(off + (size_t)rows * d->head_dim * es);
  a.v_out = off;   off = up256(off + (size_t)rows * d->head_dim * es);
  a.total = off;
  return a;
}

}  // namespace
}  // namespace lava

using namespace lava;

extern "C" {

size_t lava_host_arena_bytes(const lava_layer_desc* desc, int32_t n_layers,
                             int64_t total_budget_rows) {
  Geom g;
  if (n_layers < 1 || total_budget_rows < 0) return 0;
  if (!desc) return 0;
  lava_layer_desc d = *desc;
  d.cu_seqlens = d.batch > 1 ? reinterpret_cast<const int32_t*>(16) : nullptr;
  set_dense_layout(&d);
  if (make_geom(&d, &g) != LAVA_OK) return 0;
  return arena_layout(&d, n_layers, total_budget_rows).total;
}

lava_status lava_evict_model_host(const lava_layer_desc* desc, int32_t n_layers,
                                  const void* q_win, const void* k, const void* v,
                                  const int32_t* seq_lens, const int64_t* total_budget,
                                  int32_t mode, int64_t* layer_budget, int32_t* head_offsets,
                                  void* k_out, void* v_out, void* arena, size_t arena_bytes,
                                  void* stream) {
  if (!desc) return fail(LAVA_ERR_INVALID_ARG, "desc is NULL");
  if (n_layers < 1 || n_layers > 256) return fail(LAVA_ERR_UNSUPPORTED, "n_layers must be in 1..256");
  if (!q_win || !k || !v || !seq_lens || !total_budget || !layer_budget || !head_offsets ||
      !k_out || !v_out || !arena)
    return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  if (reinterpret_cast<uintptr_t>(arena) & 255u)
    return fail(LAVA_ERR_INVALID_ARG, "arena must be 256-byte aligned");
  if (desc->batch < 1 || desc->batch > 1024) return fail(LAVA_ERR_UNSUPPORTED, "batch must be in 1..1024");

  char* base = static_cast<char*>(arena);
  long long rows = 0, tokens = 0;
  int max_len = 0;
  std::vector<int> cu(desc->batch + 1, 0);
  std::vector<long long> lo(desc->batch), hi(desc->batch);
  for (int b = 0; b < desc->batch; ++b) {
    if (seq_lens[b] < desc->window)
      return fail(LAVA_ERR_INVALID_ARG, "sequence %d is shorter than the window", b);
    if (total_budget[b] < 0) return fail(LAVA_ERR_INVALID_ARG, "negative budget");
    rows += total_budget[b];
    tokens += seq_lens[b];
    cu[b + 1] = cu[b] + seq_lens[b];
    max_len = seq_lens[b] > max_len ? seq_lens[b] : max_len;
    lo[b] = (long long)desc->n_kv_heads * desc->window;
    hi[b] = (long long)desc->n_kv_heads * seq_lens[b];
    if (total_budget[b] < n_layers * lo[b] || total_budget[b] > n_layers * hi[b])
      return fail(LAVA_ERR_INVALID_ARG, "total_budget[%d] outside [L*H_kv*w, L*H_kv*n]", b);
  }
  if (tokens != desc->total_tokens)
    return fail(LAVA_ERR_INVALID_ARG, "seq_lens do not sum to total_tokens");

  lava_layer_desc d = *desc;
  set_dense_layout(&d);
  d.max_seqlen = max_len;
  const Arena a = arena_layout(&d, n_layers, rows);
  d.cu_seqlens = d.batch > 1 ? reinterpret_cast<const int32_t*>(base + a.cu) : nullptr;
  Geom g;
  lava_status rc = make_geom(&d, &g);
  if (rc != LAVA_OK) return rc;
  if (arena_bytes < a.total)
    return fail(LAVA_ERR_WORKSPACE, "arena too small: %zu < %zu bytes", arena_bytes, a.total);

  int dev = 0;
  rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (rc != LAVA_OK) return rc;
  if (dev < 0 || dev >= 64) return fail(LAVA_ERR_UNSUPPORTED, "device index out of range");
  HostPathState& st = g_state[dev];
  {
    std::lock_guard<std::mutex> lock(g_state_mutex);
    if (!st.copy_stream) {
      rc = check_cuda(cudaStreamCreateWithFlags(&st.copy_stream, cudaStreamNonBlocking), "stream create");
      if (rc != LAVA_OK) return rc;
      rc = check_cuda(cudaEventCreateWithFlags(&st.start, cudaEventDisableTiming), "event create");
      if (rc != LAVA_OK) return rc;
    }
    while ((int)st.layer_ready.size() < n_layers) {
      cudaEvent_t e;
      rc = check_cuda(cudaEventCreateWithFlags(&e, cudaEventDisableTiming), "event create");
      if (rc != LAVA_OK) return rc;
      st.layer_ready.push_back(e);
    }
  }

  cudaStream_t main_s = (cudaStream_t)stream, copy_s = st.copy_stream;
  const size_t es = d.dtype == LAVA_BF16 ? 2 : 4;
  const size_t total_scores = (size_t)g.total_scores;
#define LAVA_TRY(expr, what)                       \
  do {                                             \
    rc = check_cuda((expr), what);                 \
    if (rc != LAVA_OK) return rc;                  \
  } while (0)
  // the arena may still be in use by earlier work on `stream`
  LAVA_TRY(cudaEventRecord(st.start, main_s), "event record");
  LAVA_TRY(cudaStreamWaitEvent(copy_s, st.start, 0), "stream wait");
  LAVA_TRY(cudaMemsetAsync(base + a.ws, 0, Workspace::kStatusBytes, main_s), "status clear");
  LAVA_TRY(cudaMemcpyAsync(base + a.cu, cu.data(), sizeof(int) * cu.size(), cudaMemcpyHostToDevice, main_s), "H2D cu_seqlens");
  LAVA_TRY(cudaMemcpyAsync(base + a.tb, total_budget, sizeof(long long) * d.batch, cudaMemcpyHostToDevice, main_s), "H2D budgets");
  LAVA_TRY(cudaMemcpyAsync(base + a.lo, lo.data(), sizeof(long long) * d.batch, cudaMemcpyHostToDevice, main_s), "H2D floors");
  LAVA_TRY(cudaMemcpyAsync(base + a.hi, hi.data(), sizeof(long long) * d.batch, cudaMemcpyHostToDevice, main_s), "H2D caps");
  for (int l = 0; l < n_layers; ++l) {
    LAVA_TRY(cudaMemcpyAsync(base + a.q + l * a.q_layer, (const char*)q_win + l * a.q_layer, a.q_layer, cudaMemcpyHostToDevice, copy_s), "H2D q");
    LAVA_TRY(cudaMemcpyAsync(base + a.k + l * a.kv_layer, (const char*)k + l * a.kv_layer, a.kv_layer, cudaMemcpyHostToDevice, copy_s), "H2D k");
    LAVA_TRY(cudaMemcpyAsync(base + a.v + l * a.kv_layer, (const char*)v + l * a.kv_layer, a.kv_layer, cudaMemcpyHostToDevice, copy_s), "H2D v");
    LAVA_TRY(cudaEventRecord(st.layer_ready[l], copy_s), "event record");
    LAVA_TRY(cudaStreamWaitEvent(main_s, st.layer_ready[l], 0), "stream wait");
    rc = lava_score_layer(&d, base + a.q + l * a.q_layer, base + a.k + l * a.kv_layer,
                          base + a.v + l * a.kv_layer, nullptr,
                          reinterpret_cast<float*>(base + a.scores) + l * total_scores,
                          reinterpret_cast<float*>(base + a.vbar) + (size_t)l * d.batch * d.n_kv_heads,
                          reinterpret_cast<double*>(base + a.ent) + (size_t)l * d.batch,
                          base + a.ws, a.ws_bytes, main_s);
    if (rc != LAVA_OK) return rc;
  }
  rc = lava_layer_budgets(n_layers, d.batch, reinterpret_cast<double*>(base + a.ent),
                          reinterpret_cast<int64_t*>(base + a.tb), reinterpret_cast<int64_t*>(base + a.lo),
                          reinterpret_cast<int64_t*>(base + a.hi), mode,
                          reinterpret_cast<int64_t*>(base + a.budget),
                          reinterpret_cast<int64_t*>(base + a.rowoff),
                          reinterpret_cast<uint32_t*>(base + a.ws), main_s);
  if (rc != LAVA_OK) return rc;
  rc = lava_select_topk_layers(&d, n_layers, reinterpret_cast<float*>(base + a.scores),
                               reinterpret_cast<int64_t*>(base + a.budget),
                               reinterpret_cast<int32_t*>(base + a.keep),
                               reinterpret_cast<int32_t*>(base + a.hoff), base + a.ws, a.ws_bytes, main_s);
  if (rc != LAVA_OK) return rc;
  const long long kv_ls = (long long)(a.kv_layer / es);
  rc = lava_compact_kv_layers(&d, n_layers, base + a.k, base + a.v, kv_ls, kv_ls,
                              reinterpret_cast<int32_t*>(base + a.keep),
                              reinterpret_cast<int32_t*>(base + a.hoff),
                              reinterpret_cast<int64_t*>(base + a.rowoff), base + a.k_out,
                              base + a.v_out, main_s);
  if (rc != LAVA_OK) return rc;
  const size_t problems = (size_t)n_layers * d.batch;
  LAVA_TRY(cudaMemcpyAsync(layer_budget, base + a.budget, sizeof(long long) * problems, cudaMemcpyDeviceToHost, main_s), "D2H budgets");
  LAVA_TRY(cudaMemcpyAsync(head_offsets, base + a.hoff, sizeof(int) * problems * (d.n_kv_heads + 1), cudaMemcpyDeviceToHost, main_s), "D2H head offsets");
  LAVA_TRY(cudaMemcpyAsync(k_out, base + a.k_out, (size_t)rows * d.head_dim * es, cudaMemcpyDeviceToHost, main_s), "D2H k_out");
  LAVA_TRY(cudaMemcpyAsync(v_out, base + a.v_out, (size_t)rows * d.head_dim * es, cudaMemcpyDeviceToHost, main_s), "D2H v_out");
#undef LAVA_TRY
  return LAVA_OK;
}

}  // extern "C"
