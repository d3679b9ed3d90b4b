// Layer-wide top-k (Algorithm 1, Evict) when the KV heads of a layer are split over several
// GPUs: every rank holds the scores of its own heads and the ranks must agree on one threshold
// for the whole layer.  The exact radix select of select.cu is cut at the points where the
// ranks have to meet:
//
//   begin                      k_rem = B_l - H_kv(all ranks) * w, clamped
//   for pass in 0, 1, 2:
//     hist   (local)           digit histogram of the local keys that still match the prefix
//     -- all-reduce(sum) of the 2048-bin histograms over the ranks (a few KB per problem) --
//     step   (same on all)     walk the global histogram from the top, fix the next digit
//   count  (local)             per local head: entries above tau, entries equal to tau
//   -- all-gather of the ranks' tie counts; ties go to the lower flat index, that is, to the
//      lower rank first --
//   emit   (local)             kept positions of the local heads in ascending order, offsets
//
// The collective itself is the caller's (NCCL through torch.distributed in the Python layer);
// these kernels never touch another GPU's memory.  Plain kernels: the data is the rank's share
// of one layer's scores, the latency is the collectives'.
#include "lava_internal.cuh"

namespace lava {
namespace {

constexpr int kBins = 2048;
__host__ __device__ inline int digit_shift(int pass) { return pass == 0 ? 21 : pass == 1 ? 10 : 0; }
__host__ __device__ inline int digit_width(int pass) { return pass == 2 ? 10 : 11; }

struct ShardState {  // per (layer, sequence); identical on every rank after each step
  long long prefix_val, prefix_mask, k_rem, k_sel;
};

__global__ void shard_begin_kernel(Geom g, int n_layers, int total_kv_heads,
                                   const long long* layer_budget, ShardState* state) {
  const int prob = blockIdx.x * blockDim.x + threadIdx.x;
  if (prob >= n_layers * g.batch) return;
  const SeqInfo s = seq_info(g, prob % g.batch);
  const long long m_total = (long long)total_kv_heads * s.prefix;
  long long k = layer_budget[prob] - (long long)total_kv_heads * min(g.window, s.n);
  k = max(0ll, min(k, m_total));
  state[prob] = ShardState{0, 0, k, k};
}

__global__ void __launch_bounds__(512)
shard_hist_kernel(Geom g, const float* scores, const ShardState* state, int pass, unsigned* hist) {
  if (batch_has_short_sequence(g)) return;  // the score layout has no room for such a batch
  __shared__ unsigned sh[kBins];
  const int prob = blockIdx.y, layer = prob / g.batch;
  const SeqInfo s = seq_info(g, prob - layer * g.batch);
  const ShardState st = state[prob];
  if (st.k_sel == 0) return;
  for (int i = threadIdx.x; i < kBins; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  const unsigned* keys =
      reinterpret_cast<const unsigned*>(scores + (size_t)layer * g.total_scores + s.score_off);
  const long long m = (long long)g.n_kv_heads * s.prefix;
  const unsigned pv = (unsigned)st.prefix_val, pm = (unsigned)st.prefix_mask;
  const int shift = digit_shift(pass);
  const unsigned dmask = (1u << digit_width(pass)) - 1u;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < m;
       i += (long long)gridDim.x * blockDim.x) {
    const unsigned key = keys[i];
    if ((key & pm) == pv) atomicAdd(&sh[(key >> shift) & dmask], 1u);
  }
  __syncthreads();
  unsigned* out = hist + (size_t)prob * kBins;
  for (int i = threadIdx.x; i < kBins; i += blockDim.x)
    if (sh[i]) atomicAdd(&out[i], sh[i]);
}

// One block per problem: the digit whose bucket holds the k_rem-th largest matching key.
__global__ void __launch_bounds__(256)
shard_step_kernel(int pass, const unsigned* hist, ShardState* state) {
  __shared__ unsigned long long wsum[8];
  __shared__ int found;
  __shared__ unsigned long long found_before;
  const int prob = blockIdx.x;
  ShardState st = state[prob];
  if (st.k_sel == 0) return;
  const unsigned* h = hist + (size_t)prob * kBins;
  // thread t owns digits [kBins-1-8t-7, kBins-1-8t], walked from the top
  unsigned mine[8];
  unsigned long long local = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    mine[j] = h[kBins - 1 - (threadIdx.x * 8 + j)];
    local += mine[j];
  }
  unsigned long long incl = local;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) wsum[warp] = incl;
  if (threadIdx.x == 0) found = -1;
  __syncthreads();
  unsigned long long before = incl - local;
  for (int wdx = 0; wdx < warp; ++wdx) before += wsum[wdx];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if ((long long)before < st.k_rem && st.k_rem <= (long long)(before + mine[j])) {
      found = kBins - 1 - (threadIdx.x * 8 + j);
      found_before = before;
    }
    before += mine[j];
  }
  __syncthreads();
  if (threadIdx.x == 0 && found >= 0) {
    const long long dmask = (1ll << digit_width(pass)) - 1;
    st.prefix_val |= (long long)found << digit_shift(pass);
    st.prefix_mask |= dmask << digit_shift(pass);
    st.k_rem -= (long long)found_before;
    state[prob] = st;
  }
}

// counts[prob][head] = (entries above tau, entries equal to tau) of every local head.
__global__ void __launch_bounds__(512)
shard_count_kernel(Geom g, const float* scores, const ShardState* state, uint2* counts) {
  if (batch_has_short_sequence(g)) return;  // the score layout has no room for such a batch
  __shared__ unsigned wg[16], we[16];
  const int prob = blockIdx.y, layer = prob / g.batch, head = blockIdx.x;
  const SeqInfo s = seq_info(g, prob - layer * g.batch);
  const ShardState st = state[prob];
  const unsigned tau = st.k_sel > 0 ? (unsigned)st.prefix_val : 0xffffffffu;
  const unsigned* keys = reinterpret_cast<const unsigned*>(
      scores + (size_t)layer * g.total_scores + s.score_off + (long long)head * s.prefix);
  unsigned n_gt = 0, n_eq = 0;
  for (int i = threadIdx.x; i < s.prefix; i += blockDim.x) {
    const unsigned key = keys[i];
    n_gt += key > tau;
    n_eq += key == tau;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    n_gt += __shfl_down_sync(0xffffffffu, n_gt, o);
    n_eq += __shfl_down_sync(0xffffffffu, n_eq, o);
  }
  if ((threadIdx.x & 31) == 0) {
    wg[threadIdx.x >> 5] = n_gt;
    we[threadIdx.x >> 5] = n_eq;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned a = 0, b = 0;
    for (int i = 0; i < 16; ++i) {
      a += wg[i];
      b += we[i];
    }
    counts[(size_t)prob * g.n_kv_heads + head] = make_uint2(a, b);
  }
}

// Sum of the local tie counts per problem (what the ranks exchange).
__global__ void shard_ties_kernel(int problems, int heads, const uint2* counts, long long* ties) {
  const int prob = blockIdx.x * blockDim.x + threadIdx.x;
  if (prob >= problems) return;
  long long t = 0;
  for (int h = 0; h < heads; ++h) t += counts[(size_t)prob * heads + h].y;
  ties[prob] = t;
}

// One block per (local head, problem): ordered emit.  Ties are taken in flat-index order over
// the whole layer: `ties_before_rank` of them belong to lower ranks.
__global__ void __launch_bounds__(1024)
shard_emit_kernel(Geom g, const float* scores, const ShardState* state, const uint2* counts,
                  const long long* ties_before_rank, int* keep_idx, int* head_offsets,
                  long long* rows_out) {
  if (batch_has_short_sequence(g)) return;  // the score layout has no room for such a batch
  __shared__ unsigned wsum[32];
  __shared__ unsigned run_keep, run_eq;
  const int prob = blockIdx.y, layer = prob / g.batch, head = blockIdx.x;
  const SeqInfo s = seq_info(g, prob - layer * g.batch);
  const int win = min(g.window, s.n);
  const ShardState st = state[prob];
  const unsigned tau = st.k_sel > 0 ? (unsigned)st.prefix_val : 0xffffffffu;
  const long long ties_wanted = st.k_sel > 0 ? st.k_rem : 0;
  // what the heads before this one (lower ranks first, then lower local heads) take
  long long ties_before = ties_before_rank[prob];
  long long kept_before = 0;
  const uint2* cnt = counts + (size_t)prob * g.n_kv_heads;
  for (int h = 0; h < head; ++h) {
    const long long take = max(0ll, min((long long)cnt[h].y, ties_wanted - ties_before));
    kept_before += cnt[h].x + take;
    ties_before += cnt[h].y;
  }
  const long long my_ties = max(0ll, min((long long)cnt[head].y, ties_wanted - ties_before));
  const unsigned* keys = reinterpret_cast<const unsigned*>(
      scores + (size_t)layer * g.total_scores + s.score_off + (long long)head * s.prefix);
  int* out = keep_idx + (size_t)layer * g.total_scores + s.score_off + kept_before;
  if (threadIdx.x == 0) {
    run_keep = 0;
    run_eq = 0;
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int base = 0; base < s.prefix; base += 1024) {
    const int i = base + threadIdx.x;
    const unsigned key = i < s.prefix ? keys[i] : 0u;
    const unsigned eq = i < s.prefix && key == tau;
    // exclusive scan of the tie flags, then of the keep flags (two rounds over one buffer)
    unsigned incl = eq;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    unsigned eq_before = run_eq + incl - eq;
    for (int wdx = 0; wdx < warp; ++wdx) eq_before += wsum[wdx];
    unsigned eq_total = 0;
    for (int wdx = 0; wdx < 32; ++wdx) eq_total += wsum[wdx];
    __syncthreads();
    const unsigned keep = i < s.prefix && (key > tau || (eq && (long long)eq_before < my_ties));
    incl = keep;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    unsigned slot = run_keep + incl - keep;
    for (int wdx = 0; wdx < warp; ++wdx) slot += wsum[wdx];
    unsigned keep_total = 0;
    for (int wdx = 0; wdx < 32; ++wdx) keep_total += wsum[wdx];
    if (keep) out[slot] = i;
    __syncthreads();
    if (threadIdx.x == 0) {
      run_keep += keep_total;
      run_eq += eq_total;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    int* hoff = head_offsets + (size_t)prob * (g.n_kv_heads + 1);
    hoff[head] = (int)kept_before + head * win;
    if (head == g.n_kv_heads - 1) {
      const long long rows = kept_before + cnt[head].x + my_ties + (long long)g.n_kv_heads * win;
      hoff[g.n_kv_heads] = (int)rows;
      if (rows_out) rows_out[prob] = rows;
    }
  }
}

// Exclusive prefix sum of `count` row counts (one block).
__global__ void __launch_bounds__(256)
shard_row_offsets_kernel(int count, const long long* rows, long long* row_off) {
  __shared__ long long warp_tot[8];
  __shared__ long long carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int base = 0; base < count; base += 256) {
    const int i = base + threadIdx.x;
    const long long x = i < count ? rows[i] : 0;
    long long incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    long long before = carry;
    for (int wdx = 0; wdx < warp; ++wdx) before += warp_tot[wdx];
    if (i < count) row_off[i] = before + incl - x;
    __syncthreads();
    if (threadIdx.x == 255) carry = before + incl;
    __syncthreads();
  }
  if (threadIdx.x == 0) row_off[count] = carry;
}

struct ShardLayout {
  size_t off_state, off_hist, off_counts, off_ties, total;
};
inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }
ShardLayout shard_layout(const Geom& g, int n_layers) {
  ShardLayout l;
  const size_t problems = (size_t)n_layers * g.batch;
  size_t off = 0;
  l.off_state = off;
  off = up256(off + problems * sizeof(ShardState));
  l.off_hist = off;
  off = up256(off + problems * kBins * sizeof(unsigned));
  l.off_counts = off;
  off = up256(off + problems * g.n_kv_heads * sizeof(uint2));
  l.off_ties = off;
  off = up256(off + problems * sizeof(long long));
  l.total = off;
  return l;
}

}  // namespace
}  // namespace lava

using namespace lava;

extern "C" {

size_t lava_select_shard_bytes(const lava_layer_desc* desc, int32_t n_layers) {
  Geom g;
  if (n_layers < 1 || make_geom(desc, &g) != LAVA_OK) return 0;
  return shard_layout(g, n_layers).total;
}

lava_status lava_select_shard_layout(const lava_layer_desc* desc, int32_t n_layers,
                                     size_t* hist_offset, size_t* hist_bytes, size_t* ties_offset,
                                     size_t* ties_bytes) {
  Geom g;
  lava_status rc = make_geom(desc, &g);
  if (rc != LAVA_OK) return rc;
  if (n_layers < 1 || !hist_offset || !hist_bytes || !ties_offset || !ties_bytes)
    return fail(LAVA_ERR_INVALID_ARG, "bad argument");
  const ShardLayout l = shard_layout(g, n_layers);
  *hist_offset = l.off_hist;
  *hist_bytes = (size_t)n_layers * g.batch * kBins * sizeof(unsigned);
  *ties_offset = l.off_ties;
  *ties_bytes = (size_t)n_layers * g.batch * sizeof(long long);
  return LAVA_OK;
}

static lava_status shard_args(const lava_layer_desc* desc, int32_t n_layers, void* state,
                              size_t state_bytes, Geom* g, ShardLayout* l) {
  lava_status rc = make_geom(desc, g);
  if (rc != LAVA_OK) return rc;
  if (n_layers < 1) return fail(LAVA_ERR_INVALID_ARG, "n_layers must be >= 1");
  if ((long long)n_layers * g->batch > 65535)
    return fail(LAVA_ERR_UNSUPPORTED, "n_layers*batch must be <= 65535");
  *l = shard_layout(*g, n_layers);
  if (!state || !aligned16(state)) return fail(LAVA_ERR_INVALID_ARG, "state must be 16-byte aligned");
  if (state_bytes < l->total)
    return fail(LAVA_ERR_WORKSPACE, "state too small: %zu < %zu bytes", state_bytes, l->total);
  return LAVA_OK;
}

lava_status lava_select_shard_begin(const lava_layer_desc* desc, int32_t n_layers,
                                    int32_t total_kv_heads, const int64_t* layer_budget,
                                    void* state, size_t state_bytes, void* stream) {
  Geom g;
  ShardLayout l;
  lava_status rc = shard_args(desc, n_layers, state, state_bytes, &g, &l);
  if (rc != LAVA_OK) return rc;
  if (!layer_budget || total_kv_heads < g.n_kv_heads)
    return fail(LAVA_ERR_INVALID_ARG, "layer_budget is required and total_kv_heads >= local heads");
  const int problems = n_layers * g.batch;
  shard_begin_kernel<<<(problems + 127) / 128, 128, 0, (cudaStream_t)stream>>>(
      g, n_layers, total_kv_heads, (const long long*)layer_budget,
      (ShardState*)((char*)state + l.off_state));
  count_launches(1);
  return check_cuda(cudaGetLastError(), "shard begin launch");
}

lava_status lava_select_shard_hist(const lava_layer_desc* desc, int32_t n_layers,
                                   const float* scores, int32_t pass, void* state,
                                   size_t state_bytes, void* stream) {
  Geom g;
  ShardLayout l;
  lava_status rc = shard_args(desc, n_layers, state, state_bytes, &g, &l);
  if (rc != LAVA_OK) return rc;
  if (pass < 0 || pass > 2) return fail(LAVA_ERR_INVALID_ARG, "pass must be 0, 1 or 2");
  if (!scores && g.total_scores > 0) return fail(LAVA_ERR_INVALID_ARG, "scores is required");
  cudaStream_t st = (cudaStream_t)stream;
  const int problems = n_layers * g.batch;
  unsigned* hist = (unsigned*)((char*)state + l.off_hist);
  rc = check_cuda(cudaMemsetAsync(hist, 0, (size_t)problems * kBins * sizeof(unsigned), st),
                  "histogram clear");
  if (rc != LAVA_OK) return rc;
  const long long m_max = (long long)g.n_kv_heads * (g.max_seqlen > g.window ? g.max_seqlen - g.window : 0);
  const int blocks = (int)std::max(1ll, std::min(64ll, (m_max + 8191) / 8192));
  shard_hist_kernel<<<dim3(blocks, problems), 512, 0, st>>>(
      g, scores, (const ShardState*)((char*)state + l.off_state), pass, hist);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "shard histogram launch");
}

lava_status lava_select_shard_step(const lava_layer_desc* desc, int32_t n_layers, int32_t pass,
                                   void* state, size_t state_bytes, void* stream) {
  Geom g;
  ShardLayout l;
  lava_status rc = shard_args(desc, n_layers, state, state_bytes, &g, &l);
  if (rc != LAVA_OK) return rc;
  if (pass < 0 || pass > 2) return fail(LAVA_ERR_INVALID_ARG, "pass must be 0, 1 or 2");
  shard_step_kernel<<<n_layers * g.batch, 256, 0, (cudaStream_t)stream>>>(
      pass, (const unsigned*)((char*)state + l.off_hist), (ShardState*)((char*)state + l.off_state));
  count_launches(1);
  return check_cuda(cudaGetLastError(), "shard step launch");
}

lava_status lava_select_shard_count(const lava_layer_desc* desc, int32_t n_layers,
                                    const float* scores, void* state, size_t state_bytes,
                                    void* stream) {
  Geom g;
  ShardLayout l;
  lava_status rc = shard_args(desc, n_layers, state, state_bytes, &g, &l);
  if (rc != LAVA_OK) return rc;
  if (!scores && g.total_scores > 0) return fail(LAVA_ERR_INVALID_ARG, "scores is required");
  cudaStream_t st = (cudaStream_t)stream;
  const int problems = n_layers * g.batch;
  uint2* counts = (uint2*)((char*)state + l.off_counts);
  shard_count_kernel<<<dim3(g.n_kv_heads, problems), 512, 0, st>>>(
      g, scores, (const ShardState*)((char*)state + l.off_state), counts);
  shard_ties_kernel<<<(problems + 127) / 128, 128, 0, st>>>(problems, g.n_kv_heads, counts,
                                                            (long long*)((char*)state + l.off_ties));
  count_launches(2);
  return check_cuda(cudaGetLastError(), "shard count launch");
}

lava_status lava_select_shard_emit(const lava_layer_desc* desc, int32_t n_layers,
                                   const float* scores, const int64_t* ties_before_rank,
                                   int32_t* keep_idx, int32_t* head_offsets,
                                   int64_t* layer_row_offset, void* state, size_t state_bytes,
                                   void* stream) {
  Geom g;
  ShardLayout l;
  lava_status rc = shard_args(desc, n_layers, state, state_bytes, &g, &l);
  if (rc != LAVA_OK) return rc;
  if (!ties_before_rank || !head_offsets || ((!scores || !keep_idx) && g.total_scores > 0))
    return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  cudaStream_t st = (cudaStream_t)stream;
  const int problems = n_layers * g.batch;
  // the local row counts reuse the tie array once the ranks have exchanged it
  long long* rows = layer_row_offset ? (long long*)((char*)state + l.off_ties) : nullptr;
  shard_emit_kernel<<<dim3(g.n_kv_heads, problems), 1024, 0, st>>>(
      g, scores, (const ShardState*)((char*)state + l.off_state),
      (const uint2*)((char*)state + l.off_counts), (const long long*)ties_before_rank, keep_idx,
      head_offsets, rows);
  count_launches(1);
  if (layer_row_offset) {
    shard_row_offsets_kernel<<<1, 256, 0, st>>>(problems, rows, (long long*)layer_row_offset);
    count_launches(1);
  }
  return check_cuda(cudaGetLastError(), "shard emit launch");
}

}  // extern "C"
