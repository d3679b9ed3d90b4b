// Internal declarations shared by the translation units of liblava (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lava.h"

namespace lava {

// Geometry handed to kernels by value.
struct Geom {
  int n_q_heads, n_kv_heads, group, head_dim, window, w_pad;
  int pool_kind, pool_kernel, pool_radius, dtype, batch, max_seqlen, flags;
  const int* cu_seqlens;
  long long total_tokens, total_scores;
  long long k_sh, k_st, v_sh, v_st;  // strides in elements
  float scale_log2;                  // sm_scale * log2(e): logits are kept in the base-2 domain
  float c_hat;
};

struct SeqInfo {
  long long tok0;       // first token of the sequence in the concatenated token axis
  int n;                // sequence length
  int prefix;           // P = n - w (0 if the sequence is not longer than the window)
  long long score_off;  // offset of the sequence's flat score array inside a layer
};

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

__device__ inline SeqInfo seq_info(const Geom& g, int b) {
  SeqInfo s;
  if (g.cu_seqlens) {
    s.tok0 = g.cu_seqlens[b];
    s.n = g.cu_seqlens[b + 1] - g.cu_seqlens[b];
  } else {
    s.tok0 = 0;
    s.n = (int)g.total_tokens;
  }
  s.prefix = s.n > g.window ? s.n - g.window : 0;
  s.score_off = (long long)g.n_kv_heads * (s.tok0 - (long long)b * g.window);
  return s;
}

// The score layout gives sequence b the offset H_kv * (tok0 - b*w): it has no room for a sequence
// shorter than the window (the host can only check the total, the lengths live on the device).
// Every kernel that addresses scores or kept positions through that layout asks this first and
// does nothing if it holds, so that such a batch cannot write outside its arrays; the score
// kernels also report LAVA_DEV_SHORT_SEQUENCE.  Block-wide: every thread of a one-dimensional
// block must call it.
__device__ inline bool batch_has_short_sequence(const Geom& g) {
  int bad = 0;
  if (g.cu_seqlens) {
    for (int b = threadIdx.x; b < g.batch; b += blockDim.x)
      bad |= (g.cu_seqlens[b + 1] - g.cu_seqlens[b]) < g.window;
  } else {
    bad = g.total_tokens < g.window;
  }
  return __syncthreads_or(bad) != 0;
}

// Workspace layout (byte offsets from the workspace base), identical for every caller.
struct Workspace {
  static constexpr size_t kStatusBytes = 256;
  static constexpr int kSlice = 512;    // keys per block in the generic score kernels
  static constexpr int kVSlice = 1024;  // V rows per block in the value-norm kernel
  size_t off_vpart, off_stats, off_lse, off_vbar, off_ones, off_ent, off_sm100, off_tmem, total;
  int n_slices, n_vslices;
};
Workspace workspace_layout(const lava_layer_desc* d, int n_layers);

// Tuning and test knobs of the library (lava_set_option / lava_get_option).  The defaults come from
// the environment, read once when the first option is looked at; nothing on a call path calls getenv.
struct Options {
  int select_cluster;      // 0: choose by size, else 8 or 16 CTAs per selection cluster
  int score_chunk_tiles;   // 0: choose per launch, else tiles per chunk of the two-pass score kernel
  int score_lead_tiles;    // -1: choose, else the extra tiles pass 1 leads pass 2 by
  int force_generic;       // 1: score on the CUDA-core path whatever the geometry
  int score_kernel;        // 0: choose, 1: two-pass kernel, 2: single-pass (logits kept in TMEM)
  long long wait_limit_cycles;  // SM cycles after which a device-side wait that may be abandoned gives up
};
Options& options();
int sm_count();            // multiprocessors of the current device (cached per device), 0 on error

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Host-side error plumbing.
lava_status fail(lava_status st, const char* fmt, ...);
lava_status check_cuda(cudaError_t e, const char* what);
lava_status make_geom(const lava_layer_desc* d, Geom* out);
void count_launches(int n);  // bookkeeping for lava_launch_count()

// Launchers implemented in the kernel translation units.  Each returns LAVA_OK or the status of
// a failed launch; all run on `stream`.
lava_status launch_score_generic(const Geom& g, int n_layers, const void* q, const void* k,
                                 const void* v, long long q_ls, long long k_ls, long long v_ls,
                                 const float* vbar_in, float* scores, float* vbar_out,
                                 double* entropy, char* ws, const Workspace& lay,
                                 cudaStream_t stream);
// Blackwell tensor-core score path (bf16, head_dim 128, G*w <= 128).
struct Sm100Layout {
  int heads_total, chunks1, chunks2, out_keys;  // chunks per head at max_seqlen, pass 1 / pass 2
  int chunk_tiles;                              // tiles per chunk chosen for this launch
  size_t off_sync, sync_bytes, off_part, off_ent, total;
};
bool sm100_supported(const Geom& g);
Sm100Layout sm100_layout(const Geom& g, int n_layers);
lava_status launch_score_sm100(const Geom& g, int n_layers, const void* q, const void* k,
                               const void* v, long long q_ls, long long k_ls, long long v_ls,
                               const float* vbar_in, float* scores, float* vbar_out,
                               double* entropy, char* ws_base, size_t ws_off, cudaStream_t stream);
// Tensor maps of the query window ([layer][batch*H_q*w rows][128]) and of K
// ([layer][H_kv][tokens][128]) in boxes of 64 x 128 bf16 elements with the 128-byte swizzle.
lava_status encode_score_maps(const Geom& g, int n_layers, const void* q, const void* k,
                              long long q_ls, long long k_ls, CUtensorMap* map_q,
                              CUtensorMap* map_k);
// Single-pass Blackwell score path (logits and exponentials stay in tensor memory).
struct TmemLayout {
  int ok, nunit, tmax, kfold, gmax, heads_total, units_total;
  long long kjobs_cap;
  size_t off_sync, sync_bytes, off_part, off_gpart, off_ent, total;
};
bool tmem_supported(const Geom& g);
bool tmem_fits(const Geom& g, int grid);
int tmem_grid(const Geom& g, int n_layers);
TmemLayout tmem_layout(const Geom& g, int n_layers);
lava_status launch_score_tmem(const Geom& g, int n_layers, const void* q, const void* k,
                              const void* v, long long q_ls, long long k_ls, long long v_ls,
                              const float* vbar_in, float* scores, float* vbar_out,
                              double* entropy, char* ws_base, size_t ws_off, cudaStream_t stream);
lava_status launch_fill_ones(float* dst, long long count, cudaStream_t stream);
lava_status launch_token_norm_scale(const Geom& g, int n_layers, const void* v, long long v_ls,
                                    float* scores, cudaStream_t stream);
// entropy of every (layer, sequence) from the final score array (fixed summation order)
lava_status launch_entropy_from_scores(const Geom& g, int n_layers, const float* scores,
                                       double* entropy, cudaStream_t stream);
lava_status launch_wo_norm(const void* w_o, int dtype, long long rows, long long cols,
                           float* out, cudaStream_t stream);
lava_status launch_budgets(int n_layers, int batch, const double* entropy,
                           const long long* total, const long long* lo, const long long* hi,
                           int mode, long long* budget, long long* row_off, unsigned* status,
                           cudaStream_t stream);
lava_status launch_select(const Geom& g, int n_layers, const float* scores,
                          const long long* layer_budget, int* keep_idx, int* head_offsets,
                          unsigned* status, cudaStream_t stream);
// Lists of what every (layer, sequence) still holds during Algorithm 2's cascade: score and
// position of each held prefix entry, heads in order and positions ascending inside a head; the
// list of problem p starts at entry row_off[p] and its heads are delimited like the packed rows
// (head g's entries start at head_offsets[p][g] - g*w).
struct HeldLists {
  const float* score_old = nullptr;
  const int* pos_old = nullptr;
  const long long* row_off_old = nullptr;
  const int* hoff_old = nullptr;
  float* score_new = nullptr;
  int* pos_new = nullptr;
  int* src_pos = nullptr;           // for every new entry: its index in the old list
  const long long* row_off_new = nullptr;
};
// Re-selection of `problems` (layer, sequence) lists, each down to layer_budget[p] rows.
lava_status launch_reselect(const Geom& g, int problems, long long max_held,
                            const long long* layer_budget, int* head_offsets_new,
                            const HeldLists& io, cudaStream_t stream);
lava_status launch_compact(const Geom& g, int n_layers, const void* k, const void* v,
                           long long k_ls, long long v_ls, const int* keep_idx,
                           const int* head_offsets, const long long* row_off, void* k_out,
                           void* v_out, cudaStream_t stream);

}  // namespace lava
