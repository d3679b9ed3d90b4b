// Gather of the retained K/V rows into the packed cache (Algorithm 1: K-hat = K (.) I,
// V-hat = V (.) I, realised as a gather so evicted rows cost no memory).
//
// For (layer, sequence, KV head) the output rows are the kept prefix rows in ascending position
// followed by the w window rows.  Rows are copied bit for bit with 16-byte accesses: a group of
// (row bytes / 16) threads moves one K row and the matching V row.
#include "lava_internal.cuh"

namespace lava {
namespace {

__global__ void __launch_bounds__(256)
compact_kernel(Geom g, const char* k, const char* v, long long k_ls, long long v_ls,
               const int* keep_idx, const int* head_offsets, const long long* row_off,
               char* k_out, char* v_out, int blocks_per_head) {
  if (batch_has_short_sequence(g)) return;  // the score layout has no room for such a batch
  const int prob = blockIdx.z, layer = prob / g.batch, b = prob - layer * g.batch;
  const int kvh = blockIdx.y;
  const SeqInfo s = seq_info(g, b);
  const int es = g.dtype == LAVA_BF16 ? 2 : 4;
  const int row_bytes = g.head_dim * es;
  const int lanes = row_bytes / 16;  // threads per row: 16 (bf16 d128, f32 d64), 8, or 32
  const int* hoff = head_offsets + (size_t)prob * (g.n_kv_heads + 1);
  const int h0 = hoff[kvh], h1 = hoff[kvh + 1];
  const int rows = h1 - h0;
  const int win = min(g.window, s.n);
  const int kept = rows - win;  // kept prefix rows of this head
  // this head's kept positions: entries [h0 - kvh*win, ...) of the sequence's keep list
  const int* keep = keep_idx + (size_t)layer * g.total_scores + s.score_off + (h0 - kvh * win);
  const long long out_row0 = row_off[prob] + h0;
  const char* kl = k + ((size_t)layer * k_ls + (long long)kvh * g.k_sh) * es;
  const char* vl = v + ((size_t)layer * v_ls + (long long)kvh * g.v_sh) * es;

  const int rows_per_iter = blockDim.x / lanes;
  const int sub = threadIdx.x / lanes, c = threadIdx.x - sub * lanes;
  for (int r = blockIdx.x * rows_per_iter + sub; r < rows; r += blocks_per_head * rows_per_iter) {
    const int pos = r < kept ? keep[r] : s.prefix + (r - kept);
    const long long tok = s.tok0 + pos;
    const uint4 kk = *reinterpret_cast<const uint4*>(kl + tok * g.k_st * es + c * 16);
    const uint4 vv = *reinterpret_cast<const uint4*>(vl + tok * g.v_st * es + c * 16);
    const long long dst = (out_row0 + r) * row_bytes + c * 16;
    *reinterpret_cast<uint4*>(k_out + dst) = kk;
    *reinterpret_cast<uint4*>(v_out + dst) = vv;
  }
}

}  // namespace

lava_status launch_compact(const Geom& g, int n_layers, const void* k, const void* v,
                           long long k_ls, long long v_ls, const int* keep_idx,
                           const int* head_offsets, const long long* row_off, void* k_out,
                           void* v_out, cudaStream_t stream) {
  // Row counts live on the device, so the grid is sized for the bandwidth, not the data: enough
  // blocks per (layer, sequence, head) to fill the GPU, each striding over the head's rows.
  const int heads_total = n_layers * g.batch * g.n_kv_heads;
  const int sms = sm_count() > 0 ? sm_count() : 1;
  int blocks_per_head = (sms * 8 + heads_total - 1) / heads_total;
  if (blocks_per_head < 1) blocks_per_head = 1;
  const int max_useful = (g.max_seqlen + 15) / 16;
  if (blocks_per_head > max_useful) blocks_per_head = max_useful;
  dim3 grid(blocks_per_head, g.n_kv_heads, n_layers * g.batch);
  compact_kernel<<<grid, 256, 0, stream>>>(g, (const char*)k, (const char*)v, k_ls, v_ls, keep_idx,
                                           head_offsets, row_off, (char*)k_out, (char*)v_out,
                                           blocks_per_head);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "compact_kv launch");
}

}  // namespace lava
