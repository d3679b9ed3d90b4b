// Layer attention output loss of an eviction (Lemma 1 with p = 1, the last query of the
// sequence) and its upper bound (Theorem 1), the quality measure of the paper's analysis of layer
// attention output loss:
//     loss  = || Cat_h[ (A_h - A^_h) V_g(h) ] W_O ||_1 ,   A^_h = (A_h (.) I_g(h)) / ||A_h (.) I_g(h)||_1
//     bound = 2 C^ sum_h Vbar_g(h) sum_i A_h[i] (1 - I_g(h)[i]) ,   C^ = ||W_O^T||_1
// A_h is the attention row of the sequence's last token over all its keys; I_g marks what the
// selection kept of KV head g (its window included).  This is an evaluator, not part of the
// eviction path: plain kernels, sums in double.
#include "lava_internal.cuh"

namespace lava {
namespace {

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct LossLayout {
  size_t off_att, off_mask, off_mass, off_cat, off_part, off_chat, total;
  int col_blocks;
};

LossLayout loss_layout(const Geom& g, long long d_model) {
  LossLayout l;
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t at = off; off = round_up(off + bytes, 256); return at; };
  l.off_att = take((size_t)g.n_q_heads * g.total_tokens * sizeof(double));
  l.off_mask = take((size_t)g.n_kv_heads * g.total_tokens);
  l.off_mass = take((size_t)g.batch * g.n_q_heads * sizeof(double));
  l.off_cat = take((size_t)g.batch * g.n_q_heads * g.head_dim * sizeof(double));
  l.col_blocks = (int)((d_model + 255) / 256);
  l.off_part = take((size_t)g.batch * l.col_blocks * sizeof(double));
  l.off_chat = take(sizeof(float));
  l.total = off;
  return l;
}

__device__ inline float load_elem(const void* p, int dtype, long long i) {
  return dtype == LAVA_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i])
                            : reinterpret_cast<const float*>(p)[i];
}

__device__ inline double block_sum(double x, double* sh) {
  for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (lane == 0) sh[warp] = x;
  __syncthreads();
  double t = 0.0;
  for (int wdx = 0; wdx < nw; ++wdx) t += sh[wdx];  // warp order: the same bits for every thread
  return t;
}

__device__ inline double block_max(double x, double* sh) {
  for (int o = 16; o > 0; o >>= 1) x = fmax(x, __shfl_down_sync(0xffffffffu, x, o));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (lane == 0) sh[warp] = x;
  __syncthreads();
  double t = sh[0];
  for (int wdx = 1; wdx < nw; ++wdx) t = fmax(t, sh[wdx]);
  return t;
}

// A_h of the last token: softmax over all keys of the sequence (Sec. 2).  One block per
// (query head, sequence); the row is left in `att` as doubles.
__global__ void __launch_bounds__(256)
loss_attention_kernel(Geom g, const void* q_win, const void* k, double* att) {
  __shared__ float q[128];
  __shared__ double red[8];
  const int h = blockIdx.x, b = blockIdx.y, kvh = h / g.group;
  const SeqInfo s = seq_info(g, b);
  if (s.n < 1) return;
  // the last row of the window: q_win [batch, H_q, w, d]
  const long long qoff = (((long long)b * g.n_q_heads + h) * g.window + (g.window - 1)) * g.head_dim;
  for (int c = threadIdx.x; c < g.head_dim; c += blockDim.x) q[c] = load_elem(q_win, g.dtype, qoff + c);
  __syncthreads();
  double* row = att + (size_t)h * g.total_tokens + s.tok0;
  const double scale = (double)g.scale_log2 * 0.6931471805599453;  // back to natural units
  double mx = -1e300;
  for (int i = threadIdx.x; i < s.n; i += blockDim.x) {
    const long long koff = (long long)kvh * g.k_sh + (s.tok0 + i) * g.k_st;
    double z = 0.0;
    for (int c = 0; c < g.head_dim; ++c) z += (double)q[c] * (double)load_elem(k, g.dtype, koff + c);
    z *= scale;
    row[i] = z;
    mx = fmax(mx, z);
  }
  mx = block_max(mx, red);
  double sum = 0.0;
  for (int i = threadIdx.x; i < s.n; i += blockDim.x) {
    const double e = exp(row[i] - mx);
    row[i] = e;
    sum += e;
  }
  sum = block_sum(sum, red);
  for (int i = threadIdx.x; i < s.n; i += blockDim.x) row[i] = row[i] / sum;
}

// I_g: kept prefix positions and the window.  One block per (KV head, sequence).
__global__ void __launch_bounds__(256)
loss_mask_kernel(Geom g, const int* keep_idx, const int* head_offsets, unsigned char* mask) {
  if (batch_has_short_sequence(g)) return;  // the score layout has no room for such a batch
  const int kvh = blockIdx.x, b = blockIdx.y;
  const SeqInfo s = seq_info(g, b);
  const int win = min(g.window, s.n);
  unsigned char* row = mask + (size_t)kvh * g.total_tokens + s.tok0;
  for (int i = threadIdx.x; i < s.n; i += blockDim.x) row[i] = i >= s.prefix ? 1 : 0;
  __syncthreads();
  const int* hoff = head_offsets + (size_t)b * (g.n_kv_heads + 1);
  const int first = hoff[kvh] - kvh * win, kept = hoff[kvh + 1] - hoff[kvh] - win;
  const int* keep = keep_idx + s.score_off + first;
  for (int j = threadIdx.x; j < kept; j += blockDim.x) {
    const int pos = keep[j];
    if (pos >= 0 && pos < s.prefix) row[pos] = 1;
  }
}

// (A_h - A^_h) V_g(h): one block per (query head, sequence), thread = (slice of keys, column).
__global__ void __launch_bounds__(512)
loss_diff_value_kernel(Geom g, const void* v, const double* att, const unsigned char* mask,
                       double* mass, double* cat) {
  __shared__ double red[16];
  __shared__ double part[4][128];
  const int h = blockIdx.x, b = blockIdx.y, kvh = h / g.group;
  const SeqInfo s = seq_info(g, b);
  const double* row = att + (size_t)h * g.total_tokens + s.tok0;
  const unsigned char* keep = mask + (size_t)kvh * g.total_tokens + s.tok0;
  double kept_mass = 0.0;
  for (int i = threadIdx.x; i < s.n; i += blockDim.x) kept_mass += keep[i] ? row[i] : 0.0;
  kept_mass = block_sum(kept_mass, red);
  if (threadIdx.x == 0) mass[(size_t)b * g.n_q_heads + h] = kept_mass;
  const int c = threadIdx.x % 128, slice = threadIdx.x / 128;  // head_dim <= 128
  double acc = 0.0;
  if (c < g.head_dim) {
    for (int i = slice; i < s.n; i += 4) {
      const double a = row[i];
      const double diff = keep[i] ? a - a / kept_mass : a;
      acc += diff * (double)load_elem(v, g.dtype, (long long)kvh * g.v_sh + (s.tok0 + i) * g.v_st + c);
    }
  }
  part[slice][c] = acc;
  __syncthreads();
  if (slice == 0 && c < g.head_dim)
    cat[((size_t)b * g.n_q_heads + h) * g.head_dim + c] =
        ((part[0][c] + part[1][c]) + part[2][c]) + part[3][c];
}

// | Cat W_O |: thread = output column, block partial sums of the absolute values.
__global__ void __launch_bounds__(256)
loss_project_kernel(Geom g, const double* cat, const void* w_o, int w_dtype, long long d_model,
                    double* part) {
  __shared__ double red[8];
  const int b = blockIdx.y;
  const long long j = (long long)blockIdx.x * 256 + threadIdx.x;
  const int rows = g.n_q_heads * g.head_dim;
  const double* x = cat + (size_t)b * rows;
  double acc = 0.0;
  if (j < d_model)
    for (int r = 0; r < rows; ++r) acc += x[r] * (double)load_elem(w_o, w_dtype, (long long)r * d_model + j);
  const double total = block_sum(fabs(acc), red);
  if (threadIdx.x == 0) part[(size_t)b * gridDim.x + blockIdx.x] = total;
}

__global__ void loss_final_kernel(Geom g, const double* part, int col_blocks, const double* mass,
                                  const float* vbar, const float* c_hat, double* loss, double* bound) {
  const int b = blockIdx.x;
  if (threadIdx.x != 0) return;
  double l = 0.0;
  for (int i = 0; i < col_blocks; ++i) l += part[(size_t)b * col_blocks + i];
  loss[b] = l;
  double evicted = 0.0;
  for (int h = 0; h < g.n_q_heads; ++h)
    evicted += (double)vbar[(size_t)b * g.n_kv_heads + h / g.group] *
               (1.0 - mass[(size_t)b * g.n_q_heads + h]);
  bound[b] = 2.0 * (double)c_hat[0] * evicted;
}

}  // namespace
}  // namespace lava

using namespace lava;

extern "C" {

size_t lava_loss_workspace_bytes(const lava_layer_desc* desc, int64_t d_model) {
  Geom g;
  if (d_model < 1 || make_geom(desc, &g) != LAVA_OK) return 0;
  return loss_layout(g, d_model).total;
}

lava_status lava_layer_output_loss(const lava_layer_desc* desc, const void* q_win, const void* k,
                                   const void* v, const int32_t* keep_idx,
                                   const int32_t* head_offsets, const float* vbar,
                                   const void* w_o, int32_t w_o_dtype, int64_t d_model,
                                   double* loss_out, double* bound_out, void* workspace,
                                   size_t workspace_bytes, void* stream) {
  Geom g;
  lava_status rc = make_geom(desc, &g);
  if (rc != LAVA_OK) return rc;
  if (!q_win || !k || !v || !head_offsets || !vbar || !w_o || !loss_out || !bound_out ||
      (!keep_idx && g.total_scores > 0))
    return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  if (w_o_dtype != LAVA_F32 && w_o_dtype != LAVA_BF16) return fail(LAVA_ERR_INVALID_ARG, "unknown dtype");
  if (d_model < 1) return fail(LAVA_ERR_INVALID_ARG, "d_model must be positive");
  if (g.head_dim > 128) return fail(LAVA_ERR_UNSUPPORTED, "head_dim must be <= 128");
  const LossLayout l = loss_layout(g, d_model);
  if (!workspace || workspace_bytes < l.total)
    return fail(LAVA_ERR_WORKSPACE, "workspace too small: %zu < %zu bytes", workspace_bytes, l.total);
  if (!aligned16(workspace)) return fail(LAVA_ERR_INVALID_ARG, "workspace must be 16-byte aligned");
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  double* att = (double*)(ws + l.off_att);
  unsigned char* mask = (unsigned char*)(ws + l.off_mask);
  double* mass = (double*)(ws + l.off_mass);
  double* cat = (double*)(ws + l.off_cat);
  double* part = (double*)(ws + l.off_part);
  float* c_hat = (float*)(ws + l.off_chat);
  rc = launch_wo_norm(w_o, w_o_dtype, (long long)g.n_q_heads * g.head_dim, d_model, c_hat, st);
  if (rc != LAVA_OK) return rc;
  loss_attention_kernel<<<dim3(g.n_q_heads, g.batch), 256, 0, st>>>(g, q_win, k, att);
  loss_mask_kernel<<<dim3(g.n_kv_heads, g.batch), 256, 0, st>>>(g, keep_idx, head_offsets, mask);
  loss_diff_value_kernel<<<dim3(g.n_q_heads, g.batch), 512, 0, st>>>(g, v, att, mask, mass, cat);
  loss_project_kernel<<<dim3(l.col_blocks, g.batch), 256, 0, st>>>(g, cat, w_o, w_o_dtype, d_model, part);
  loss_final_kernel<<<g.batch, 32, 0, st>>>(g, part, l.col_blocks, mass, vbar, c_hat, loss_out, bound_out);
  count_launches(5);
  return check_cuda(cudaGetLastError(), "layer output loss launch");
}

}  // extern "C"
