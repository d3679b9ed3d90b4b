// Algorithm 2 as it is deployed: prefill and evict layer by layer.  After layer l is scored,
// the budgets of layers 0..l are recomputed from e_0..e_l, layer l is evicted from its full
// K/V, and every lower layer is evicted again from what it still holds, with the scores stored
// when it was first evicted (only the retained scores are kept, as the paper's memory analysis
// says).  The retained rows of all live layers stay packed in one arena of `total_rows` rows;
// each step writes the shrunken layout into the arena's second copy and the two swap roles, so
// every row is read once and written once per step and no copy depends on another.
//
// The state block (caller-owned device memory) holds, twice where marked (*):
//   per-step totals, floors, caps, entropies, layer budgets (*), row offsets (*), head offsets (*),
//   held scores (*), held positions (*), the source map of the last re-selection, the new
//   layer's full score and keep arrays, and the packed K and V rows (*).
#include <new>

#include "lava_internal.cuh"

namespace lava {
namespace {

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct CascadeLayout {
  size_t off_total, off_floor, off_cap, off_entropy, off_vbar;
  size_t off_budget[2], off_roff[2], off_hoff[2], off_score[2], off_pos[2], off_src;
  size_t off_scores_full, off_keep_full, off_k[2], off_v[2], total;
};

CascadeLayout cascade_layout(const Geom& g, int n_layers, long long rows) {
  CascadeLayout c;
  const size_t lb = (size_t)n_layers * g.batch;
  const size_t row_bytes = (size_t)g.head_dim * (g.dtype == LAVA_BF16 ? 2 : 4);
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t at = off; off = round_up(off + bytes, 256); return at; };
  c.off_total = take(lb * sizeof(long long));
  c.off_floor = take(g.batch * sizeof(long long));
  c.off_cap = take(g.batch * sizeof(long long));
  c.off_entropy = take(lb * sizeof(double));
  c.off_vbar = take((size_t)g.batch * g.n_kv_heads * sizeof(float));
  for (int i = 0; i < 2; ++i) {
    c.off_budget[i] = take(lb * sizeof(long long));
    c.off_roff[i] = take((lb + 1) * sizeof(long long));
    c.off_hoff[i] = take(lb * (g.n_kv_heads + 1) * sizeof(int));
    c.off_score[i] = take((size_t)rows * sizeof(float));
    c.off_pos[i] = take((size_t)rows * sizeof(int));
  }
  c.off_src = take((size_t)rows * sizeof(int));
  c.off_scores_full = take((size_t)g.total_scores * sizeof(float));
  c.off_keep_full = take((size_t)g.total_scores * sizeof(int));
  for (int i = 0; i < 2; ++i) {
    c.off_k[i] = take((size_t)rows * row_bytes);
    c.off_v[i] = take((size_t)rows * row_bytes);
  }
  c.total = off;
  return c;
}

// Per-step totals of Algorithm 2: with `live` layers prefilled the budget in force is the
// model's total, held inside what those layers can take (live*floor .. live*cap).  A total
// that the arena cannot hold, or that the whole model cannot honour, is replaced by the
// smallest feasible one and reported.
__global__ void cascade_init_kernel(Geom g, int n_layers, long long rows, const long long* total_in,
                                    long long* total_now, long long* floor_out, long long* cap_out,
                                    unsigned* status) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  long long need = 0;
  bool bad = false;
  for (int b = 0; b < g.batch; ++b) {
    const SeqInfo s = seq_info(g, b);
    const long long lo = (long long)g.n_kv_heads * min(g.window, s.n);
    const long long hi = (long long)g.n_kv_heads * s.n;
    floor_out[b] = lo;
    cap_out[b] = hi;
    long long t = total_in[b];
    if (t < n_layers * lo || t > n_layers * hi) bad = true;
    t = max(n_layers * lo, min(t, n_layers * hi));
    need += t;
  }
  const bool shrink = need > rows;  // the arena is too small for the totals asked for
  if ((bad || shrink) && status) atomicOr(status, LAVA_DEV_BUDGET_INFEASIBLE);
  for (int b = 0; b < g.batch; ++b) {
    const long long lo = floor_out[b], hi = cap_out[b];
    const long long t = shrink ? n_layers * lo : total_in[b];
    for (int l = 0; l < n_layers; ++l) {
      const long long live = l + 1;
      total_now[(size_t)l * g.batch + b] = max(live * lo, min(t, live * hi));
    }
  }
}

// Scores and positions of the entries the new layer keeps, taken from its full arrays into its
// list (the list of sequence b starts at row_off[b]).
__global__ void __launch_bounds__(256)
cascade_adopt_kernel(Geom g, const float* scores_full, const int* keep_full, const int* head_offsets,
                     const long long* row_off, float* score_list, int* pos_list) {
  if (batch_has_short_sequence(g)) return;  // the score layout has no room for such a batch
  const int b = blockIdx.y;
  const SeqInfo s = seq_info(g, b);
  const int win = min(g.window, s.n);
  const int* hoff = head_offsets + (size_t)b * (g.n_kv_heads + 1);
  const int kept = hoff[g.n_kv_heads] - g.n_kv_heads * win;
  const long long base = row_off[b];
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < kept; j += gridDim.x * blockDim.x) {
    int head = 0;
    while (head + 1 < g.n_kv_heads && hoff[head + 1] - (head + 1) * win <= j) ++head;
    const int pos = keep_full[s.score_off + j];
    pos_list[base + j] = pos;
    score_list[base + j] = scores_full[s.score_off + (long long)head * s.prefix + pos];
  }
}

// Rows of the lower layers move from the old arena to their place in the new one: for
// (layer, sequence, head) the kept rows named by the source map, then the w window rows.
__global__ void __launch_bounds__(256)
cascade_move_kernel(Geom g, const int* src_pos, const int* hoff_old_all, const int* hoff_new_all,
                    const long long* roff_old, const long long* roff_new, const char* k_old,
                    const char* v_old, char* k_new, char* v_new, int blocks_per_head) {
  if (batch_has_short_sequence(g)) return;  // the score layout has no room for such a batch
  const int prob = blockIdx.z, b = prob % g.batch, kvh = blockIdx.y;
  const SeqInfo s = seq_info(g, b);
  const int win = min(g.window, s.n);
  const int row_bytes = g.head_dim * (g.dtype == LAVA_BF16 ? 2 : 4);
  const int lanes = row_bytes / 16;
  const int* ho = hoff_old_all + (size_t)prob * (g.n_kv_heads + 1);
  const int* hn = hoff_new_all + (size_t)prob * (g.n_kv_heads + 1);
  const int h0 = hn[kvh], rows = hn[kvh + 1] - h0, kept = rows - win;
  const long long new0 = roff_new[prob], old0 = roff_old[prob];
  const int* src = src_pos + new0 + (h0 - kvh * win);  // this head's entries of the new list
  const long long old_window0 = old0 + ho[kvh + 1] - win;
  const int rows_per_iter = blockDim.x / lanes;
  const int sub = threadIdx.x / lanes, c = threadIdx.x - sub * lanes;
  for (int r = blockIdx.x * rows_per_iter + sub; r < rows; r += blocks_per_head * rows_per_iter) {
    // entry p of the old list sits in old row p + kvh*win of the sequence's segment
    const long long from = r < kept ? old0 + src[r] + (long long)kvh * win : old_window0 + (r - kept);
    const uint4 kk = *reinterpret_cast<const uint4*>(k_old + from * row_bytes + c * 16);
    const uint4 vv = *reinterpret_cast<const uint4*>(v_old + from * row_bytes + c * 16);
    const long long dst = (new0 + h0 + r) * row_bytes + c * 16;
    *reinterpret_cast<uint4*>(k_new + dst) = kk;
    *reinterpret_cast<uint4*>(v_new + dst) = vv;
  }
}

}  // namespace
}  // namespace lava

using namespace lava;

struct lava_cascade {
  lava_layer_desc desc;
  Geom g;
  int n_layers, mode, layers_done;
  long long rows;
  bool begun;
  char* state;
  CascadeLayout lay;
};

extern "C" {

size_t lava_cascade_state_bytes(const lava_layer_desc* desc, int32_t n_layers, int64_t total_rows) {
  Geom g;
  if (n_layers < 1 || total_rows < 0 || make_geom(desc, &g) != LAVA_OK) return 0;
  return cascade_layout(g, n_layers, total_rows).total;
}

lava_status lava_cascade_create(const lava_layer_desc* desc, int32_t n_layers, int64_t total_rows,
                                int32_t mode, void* state, size_t state_bytes,
                                lava_cascade** out) {
  Geom g;
  lava_status rc = make_geom(desc, &g);
  if (rc != LAVA_OK) return rc;
  if (!out) return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  *out = nullptr;
  if (n_layers < 1 || n_layers > 256) return fail(LAVA_ERR_UNSUPPORTED, "n_layers must be in 1..256");
  if (g.batch > 1024) return fail(LAVA_ERR_UNSUPPORTED, "batch must be in 1..1024");
  if (mode != LAVA_BUDGET_DYNAMIC && mode != LAVA_BUDGET_UNIFORM)
    return fail(LAVA_ERR_UNSUPPORTED, "the cascade takes the dynamic or the uniform budget rule");
  if (g.flags & LAVA_FLAG_PER_HEAD_TOPK)
    return fail(LAVA_ERR_UNSUPPORTED, "the cascade selects layer-wide");
  // the windows of every layer must fit whatever the budgets turn out to be
  const long long window_rows = (long long)n_layers * g.batch * g.n_kv_heads * g.window;
  if (total_rows < window_rows || total_rows > (1ll << 31) - 1)
    return fail(LAVA_ERR_INVALID_ARG, "total_rows must be in [%lld, 2^31)", window_rows);
  if (!state || !aligned16(state)) return fail(LAVA_ERR_INVALID_ARG, "state must be 16-byte aligned");
  const CascadeLayout lay = cascade_layout(g, n_layers, total_rows);
  if (state_bytes < lay.total)
    return fail(LAVA_ERR_WORKSPACE, "state too small: %zu < %zu bytes", state_bytes, lay.total);
  lava_cascade* h = new (std::nothrow) lava_cascade;
  if (!h) return fail(LAVA_ERR_INVALID_ARG, "out of host memory");
  h->desc = *desc;
  h->g = g;
  h->n_layers = n_layers;
  h->mode = mode;
  h->layers_done = 0;
  h->rows = total_rows;
  h->begun = false;
  h->state = (char*)state;
  h->lay = lay;
  *out = h;
  return LAVA_OK;
}

void lava_cascade_destroy(lava_cascade* h) { delete h; }

lava_status lava_cascade_begin(lava_cascade* h, const int64_t* total_budget, void* workspace,
                               void* stream) {
  if (!h || !total_budget || !workspace) return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  const CascadeLayout& c = h->lay;
  cascade_init_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(
      h->g, h->n_layers, h->rows, (const long long*)total_budget,
      (long long*)(h->state + c.off_total), (long long*)(h->state + c.off_floor),
      (long long*)(h->state + c.off_cap), (unsigned*)workspace);
  count_launches(1);
  lava_status rc = check_cuda(cudaGetLastError(), "cascade init launch");
  h->begun = rc == LAVA_OK;
  h->layers_done = 0;
  return rc;
}

lava_status lava_cascade_step(lava_cascade* h, const void* q_win, const void* k, const void* v,
                              const float* vbar_in, void* workspace, size_t workspace_bytes,
                              void* stream) {
  if (!h) return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  if (!h->begun) return fail(LAVA_ERR_INVALID_ARG, "lava_cascade_begin has not run");
  if (h->layers_done >= h->n_layers) return fail(LAVA_ERR_INVALID_ARG, "all layers have been taken");
  if (!k || !v) return fail(LAVA_ERR_INVALID_ARG, "k and v are required");
  if (!aligned16(k) || !aligned16(v)) return fail(LAVA_ERR_INVALID_ARG, "k and v must be 16-byte aligned");
  const Geom& g = h->g;
  const CascadeLayout& c = h->lay;
  const int t = h->layers_done, from = t & 1, to = from ^ 1;
  cudaStream_t st = (cudaStream_t)stream;
  char* base = h->state;
  const size_t lb_t = (size_t)t * g.batch;  // first (layer, sequence) index of the new layer
  double* entropy = (double*)(base + c.off_entropy);
  float* scores_full = (float*)(base + c.off_scores_full);
  int* keep_full = (int*)(base + c.off_keep_full);
  long long* budget_new = (long long*)(base + c.off_budget[to]);
  long long* roff_new = (long long*)(base + c.off_roff[to]);
  int* hoff_new = (int*)(base + c.off_hoff[to]);
  h->begun = false;  // a step that fails half way leaves no usable state behind

  // s_l and e_l of the new layer
  lava_status rc = lava_score_layers(&h->desc, 1, q_win, k, v, 0, 0, 0, vbar_in, scores_full,
                                     (float*)(base + c.off_vbar), entropy + lb_t, workspace,
                                     workspace_bytes, stream);
  if (rc != LAVA_OK) return rc;
  // budgets of layers 0..t from e_0..e_t, out of the total in force with t+1 layers prefilled
  rc = launch_budgets(t + 1, g.batch, entropy, (const long long*)(base + c.off_total) + lb_t,
                      (const long long*)(base + c.off_floor), (const long long*)(base + c.off_cap),
                      h->mode, budget_new, roff_new, (unsigned*)workspace, st);
  if (rc != LAVA_OK) return rc;
  // Evict(B_t, s_t, K_t, V_t): layer-wide top-k of the full layer, rows and list entries
  rc = launch_select(g, 1, scores_full, budget_new + lb_t, keep_full,
                     hoff_new + lb_t * (g.n_kv_heads + 1), (unsigned*)workspace, st);
  if (rc != LAVA_OK) return rc;
  rc = launch_compact(g, 1, k, v, 0, 0, keep_full, hoff_new + lb_t * (g.n_kv_heads + 1),
                      roff_new + lb_t, base + c.off_k[to], base + c.off_v[to], st);
  if (rc != LAVA_OK) return rc;
  if (g.total_scores > 0) {
    dim3 grid(std::max(1, std::min(64, sm_count() * 4 / std::max(1, g.batch))), g.batch);
    cascade_adopt_kernel<<<grid, 256, 0, st>>>(g, scores_full, keep_full,
                                               hoff_new + lb_t * (g.n_kv_heads + 1),
                                               roff_new + lb_t, (float*)(base + c.off_score[to]),
                                               (int*)(base + c.off_pos[to]));
    count_launches(1);
    rc = check_cuda(cudaGetLastError(), "cascade adopt launch");
    if (rc != LAVA_OK) return rc;
  }
  // Evict(B_l, s_l, K_l, V_l) for every lower layer, from what it still holds
  if (t > 0) {
    HeldLists io;
    io.score_old = (const float*)(base + c.off_score[from]);
    io.pos_old = (const int*)(base + c.off_pos[from]);
    io.row_off_old = (const long long*)(base + c.off_roff[from]);
    io.hoff_old = (const int*)(base + c.off_hoff[from]);
    io.score_new = (float*)(base + c.off_score[to]);
    io.pos_new = (int*)(base + c.off_pos[to]);
    io.src_pos = (int*)(base + c.off_src);
    io.row_off_new = roff_new;
    const long long prefix_max = g.max_seqlen > g.window ? g.max_seqlen - g.window : 0;
    const long long max_held = std::min<long long>((long long)g.n_kv_heads * prefix_max, h->rows);
    rc = launch_reselect(g, t * g.batch, max_held, budget_new, hoff_new, io, st);
    if (rc != LAVA_OK) return rc;
    const int heads_total = t * g.batch * g.n_kv_heads;
    const int sms = sm_count() > 0 ? sm_count() : 1;
    int bph = std::max(1, (sms * 8 + heads_total - 1) / heads_total);
    bph = std::min(bph, std::max(1, (g.max_seqlen + 15) / 16));
    dim3 grid(bph, g.n_kv_heads, t * g.batch);
    cascade_move_kernel<<<grid, 256, 0, st>>>(g, io.src_pos, io.hoff_old, hoff_new, io.row_off_old,
                                              roff_new, base + c.off_k[from], base + c.off_v[from],
                                              base + c.off_k[to], base + c.off_v[to], bph);
    count_launches(1);
    rc = check_cuda(cudaGetLastError(), "cascade move launch");
    if (rc != LAVA_OK) return rc;
  }
  h->layers_done = t + 1;
  h->begun = true;
  return LAVA_OK;
}

lava_status lava_cascade_get(const lava_cascade* h, lava_cascade_view* out) {
  if (!h || !out) return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  const CascadeLayout& c = h->lay;
  const int cur = h->layers_done & 1;
  char* base = h->state;
  out->layers_done = h->layers_done;
  out->k_out = base + c.off_k[cur];
  out->v_out = base + c.off_v[cur];
  out->kept_pos = (const int32_t*)(base + c.off_pos[cur]);
  out->kept_scores = (const float*)(base + c.off_score[cur]);
  out->head_offsets = (const int32_t*)(base + c.off_hoff[cur]);
  out->layer_budget = (const int64_t*)(base + c.off_budget[cur]);
  out->layer_row_offset = (const int64_t*)(base + c.off_roff[cur]);
  out->entropy = (const double*)(base + c.off_entropy);
  return LAVA_OK;
}

}  // extern "C"
