// Layer-wide top-k over the flat score array of one (layer, sequence) (Algorithm 1, Evict).
//
// Exact radix select on the fp32 bit patterns (scores are >= 0, so the unsigned patterns order
// like the values): three digit passes (11, 11, 10 bits) find the k-th largest pattern tau and
// the number of entries equal to tau that still fit; an ordered compaction then emits, head
// after head and in ascending position, every entry above tau plus the first ties in flat
// index order.  Equal scores therefore resolve to the lower flat index, deterministically.
//
// One thread-block cluster of 8 CTAs works on one (layer, sequence); each CTA owns a
// contiguous eighth of the flat array.  Histograms and counts are exchanged through
// distributed shared memory with hardware cluster barriers (no spin waits, no global atomics).
#include <cooperative_groups.h>

#include "lava_internal.cuh"

namespace cg = cooperative_groups;

namespace lava {
namespace {

constexpr int kCluster = 8;
constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kBins = 2048;

struct SelectShared {
  unsigned hist[kBins];     // this CTA's digit histogram; peers read it through DSMEM
  unsigned total[kBins];    // cluster-wide histogram (every CTA builds the same copy)
  unsigned warp_sum[kWarps + 1];
  unsigned counts[2];       // entries above tau / equal to tau inside this CTA's chunk
  unsigned found_digit, found_before;
  int head_before[1];       // placeholder to keep the struct trivially sized
};

// Inclusive block scan of one unsigned per thread (thread order); returns (exclusive, total).
__device__ inline unsigned block_exclusive_scan(unsigned x, unsigned* warp_sum, unsigned* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned incl = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  __syncthreads();  // protects warp_sum against readers of the previous call
  if (lane == 31) warp_sum[warp] = incl;
  __syncthreads();
  unsigned before = 0, all = 0;
#pragma unroll
  for (int wdx = 0; wdx < kWarps; ++wdx) {
    const unsigned v = warp_sum[wdx];
    if (wdx < warp) before += v;
    all += v;
  }
  *total = all;
  return before + incl - x;
}

__global__ void __cluster_dims__(kCluster, 1, 1) __launch_bounds__(kThreads)
select_topk_kernel(Geom g, const float* scores, const long long* layer_budget, int* keep_idx,
                   int* head_offsets) {
  __shared__ SelectShared sh;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int prob = blockIdx.y, layer = prob / g.batch, b = prob - layer * g.batch;
  const SeqInfo s = seq_info(g, b);
  const long long m_total = (long long)g.n_kv_heads * s.prefix;  // candidates
  const unsigned* keys =
      reinterpret_cast<const unsigned*>(scores + (size_t)layer * g.total_scores + s.score_off);
  int* out = keep_idx + (size_t)layer * g.total_scores + s.score_off;
  int* hoff = head_offsets + (size_t)prob * (g.n_kv_heads + 1);

  const long long window_rows = (long long)g.n_kv_heads * min(g.window, s.n);
  long long k_sel = layer_budget[prob] - window_rows;
  if (k_sel < 0) k_sel = 0;
  if (k_sel > m_total) k_sel = m_total;

  // contiguous chunk of this CTA
  const long long per = (m_total + kCluster - 1) / kCluster;
  const long long c0 = min(m_total, per * rank), c1 = min(m_total, c0 + per);

  // ---- radix passes: find tau and the number of ties to take -------------------------------
  unsigned prefix_val = 0, prefix_mask = 0;
  long long k_rem = k_sel;
  if (k_sel > 0) {
    const int shifts[3] = {21, 10, 0};
    const int widths[3] = {11, 11, 10};
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = shifts[pass];
      const unsigned dmask = (1u << widths[pass]) - 1u;
      for (int i = threadIdx.x; i < kBins; i += kThreads) sh.hist[i] = 0;
      __syncthreads();
      for (long long i0 = c0; i0 < c1; i0 += kThreads) {  // warp-uniform trip count
        const long long i = i0 + threadIdx.x;
        const unsigned key = i < c1 ? keys[i] : 0u;
        const bool mine = i < c1 && (key & prefix_mask) == prefix_val;
        const unsigned digit = (key >> shift) & dmask;
        // one shared-memory atomic per distinct digit in the warp
        const unsigned active = __ballot_sync(0xffffffffu, mine);
        if (mine) {
          const unsigned peers = __match_any_sync(active, digit);
          if ((threadIdx.x & 31) == (unsigned)(__ffs(peers) - 1))
            atomicAdd(&sh.hist[digit], (unsigned)__popc(peers));
        }
      }
      cluster.sync();  // every CTA's histogram is complete
      for (int i = threadIdx.x; i < kBins; i += kThreads) {
        unsigned sum = 0;
#pragma unroll
        for (int r = 0; r < kCluster; ++r) sum += cluster.map_shared_rank(sh.hist, r)[i];
        sh.total[i] = sum;
      }
      cluster.sync();  // peers have finished reading this CTA's histogram
      // Walk the digits from the top: thread t owns digits [kBins-1-4t-3, kBins-1-4t].
      unsigned mine4[4], local = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        mine4[j] = sh.total[kBins - 1 - (threadIdx.x * 4 + j)];
        local += mine4[j];
      }
      unsigned all;
      unsigned before = block_exclusive_scan(local, sh.warp_sum, &all);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        // `before` entries have a larger digit than this one
        if ((long long)before < k_rem && k_rem <= (long long)before + mine4[j]) {
          sh.found_digit = kBins - 1 - (threadIdx.x * 4 + j);
          sh.found_before = before;
        }
        before += mine4[j];
      }
      __syncthreads();
      prefix_val |= sh.found_digit << shift;
      prefix_mask |= dmask << shift;
      k_rem -= sh.found_before;
      __syncthreads();
    }
  }
  const unsigned tau = k_sel > 0 ? prefix_val : 0xffffffffu;
  const unsigned ties_wanted = k_sel > 0 ? (unsigned)k_rem : 0u;  // >= 1 when k_sel > 0

  // ---- count (above, equal) per CTA chunk ---------------------------------------------------
  unsigned n_gt = 0, n_eq = 0;
  for (long long i = c0 + threadIdx.x; i < c1; i += kThreads) {
    const unsigned key = keys[i];
    n_gt += key > tau;
    n_eq += key == tau;
  }
  unsigned tot_gt, tot_eq;
  block_exclusive_scan(n_gt, sh.warp_sum, &tot_gt);
  block_exclusive_scan(n_eq, sh.warp_sum, &tot_eq);
  if (threadIdx.x == 0) {
    sh.counts[0] = tot_gt;
    sh.counts[1] = tot_eq;
  }
  cluster.sync();
  unsigned kept_base = 0, tie_base = 0;  // kept entries / ties in lower-ranked chunks
  for (int r = 0; r < rank; ++r) {
    const unsigned* c = cluster.map_shared_rank(sh.counts, r);
    const unsigned gt = c[0], eq = c[1];
    const unsigned room = ties_wanted > tie_base ? ties_wanted - tie_base : 0u;
    kept_base += gt + min(eq, room);
    tie_base += eq;
  }
  cluster.sync();  // counts stay valid until every CTA has read them

  // ---- ordered compaction of this CTA's chunk ---------------------------------------------
  unsigned kept_run = kept_base, tie_run = tie_base;
  for (long long i0 = c0; i0 < c1; i0 += kThreads) {
    const long long i = i0 + threadIdx.x;
    const bool valid = i < c1;
    const unsigned key = valid ? keys[i] : 0u;
    const bool gt = valid && key > tau, eq = valid && key == tau;
    unsigned tile_eq, tile_keep;
    const unsigned eq_before = block_exclusive_scan(eq ? 1u : 0u, sh.warp_sum, &tile_eq);
    const bool keep = gt || (eq && tie_run + eq_before < ties_wanted);
    const unsigned keep_before = block_exclusive_scan(keep ? 1u : 0u, sh.warp_sum, &tile_keep);
    if (valid) {
      const int head = (int)(i / s.prefix);
      const int pos = (int)(i - (long long)head * s.prefix);
      if (keep) out[kept_run + keep_before] = pos;
      // the first entry of a head records how many kept entries precede the head
      if (pos == 0) hoff[head] = (int)(kept_run + keep_before) + head * g.window;
    }
    kept_run += tile_keep;
    tie_run += tile_eq;
  }
  if (rank == 0 && threadIdx.x == 0) {
    hoff[g.n_kv_heads] = (int)(k_sel + window_rows);
    if (s.prefix == 0)  // no candidates: every head holds only its (possibly short) window
      for (int h = 0; h < g.n_kv_heads; ++h) hoff[h] = h * min(g.window, s.n);
  }
}


// ------------------------------------------------------------------------------------------
// Register-resident variant: every thread loads its E keys once and keeps them for all passes.
// A warp owns E consecutive rows of 32 keys (row i, lane l <-> key base + 32 i + l), so loads
// are coalesced and the element order inside a warp is (row, lane): exclusive counts along a
// row come from one ballot, and no block-wide scan runs per 512 keys.  Serves problems of up to
// 32768 keys per CTA (cluster of 8 or 16 CTAs); larger ones take the streaming kernel above.
// ------------------------------------------------------------------------------------------
constexpr int kRegMaxPerCta = 32768;

struct RegShared {
  unsigned hist[kBins];
  unsigned total[kBins];
  unsigned warp_sum[kWarps + 1];
  unsigned found_digit, found_before;
  uint2 warp_cnt[kWarps];   // (above tau, equal to tau) per warp of this CTA; peers read it
};

template <int E>
__global__ void __launch_bounds__(kThreads)
select_topk_reg_kernel(Geom g, const float* scores, const long long* layer_budget, int* keep_idx,
                       int* head_offsets) {
  __shared__ RegShared sh;
  cg::cluster_group cluster = cg::this_cluster();
  const int csize = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int prob = blockIdx.x / csize, layer = prob / g.batch, b = prob - layer * g.batch;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const SeqInfo s = seq_info(g, b);
  const int m_total = g.n_kv_heads * s.prefix;  // candidates (fits 31 bits)
  const unsigned* keys =
      reinterpret_cast<const unsigned*>(scores + (size_t)layer * g.total_scores + s.score_off);
  int* out = keep_idx + (size_t)layer * g.total_scores + s.score_off;
  int* hoff = head_offsets + (size_t)prob * (g.n_kv_heads + 1);

  const long long window_rows = (long long)g.n_kv_heads * min(g.window, s.n);
  long long k_sel = layer_budget[prob] - window_rows;
  if (k_sel < 0) k_sel = 0;
  if (k_sel > m_total) k_sel = m_total;

  // this CTA's range, and inside it this warp's E rows of 32 keys
  const int per = (m_total + csize - 1) / csize;
  const int c0 = min(m_total, per * rank), c1 = min(m_total, c0 + per);
  const int wbase = c0 + warp * (E * 32);
  unsigned key[E];
#pragma unroll
  for (int i = 0; i < E; ++i) {
    const int idx = wbase + i * 32 + lane;
    key[i] = idx < c1 ? keys[idx] : 0u;
  }

  // ---- radix passes: find tau and the number of ties to take -------------------------------
  unsigned prefix_val = 0, prefix_mask = 0;
  long long k_rem = k_sel;
  if (k_sel > 0) {
    const int shifts[3] = {21, 10, 0};
    const int widths[3] = {11, 11, 10};
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = shifts[pass];
      const unsigned dmask = (1u << widths[pass]) - 1u;
      for (int i = threadIdx.x; i < kBins; i += kThreads) sh.hist[i] = 0;
      __syncthreads();
#pragma unroll
      for (int i = 0; i < E; ++i) {
        const bool mine = wbase + i * 32 + lane < c1 && (key[i] & prefix_mask) == prefix_val;
        const unsigned digit = (key[i] >> shift) & dmask;
        // one shared-memory atomic per distinct digit in the warp
        const unsigned active = __ballot_sync(0xffffffffu, mine);
        if (mine) {
          const unsigned peers = __match_any_sync(active, digit);
          if (lane == (__ffs(peers) - 1)) atomicAdd(&sh.hist[digit], (unsigned)__popc(peers));
        }
      }
      cluster.sync();  // every CTA's histogram is complete
      for (int i = threadIdx.x; i < kBins; i += kThreads) {
        unsigned sum = 0;
        for (int r = 0; r < csize; ++r) sum += cluster.map_shared_rank(sh.hist, r)[i];
        sh.total[i] = sum;
      }
      cluster.sync();  // peers have finished reading this CTA's histogram
      // Walk the digits from the top: thread t owns digits [kBins-1-4t-3, kBins-1-4t].
      unsigned mine4[4], local = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        mine4[j] = sh.total[kBins - 1 - (threadIdx.x * 4 + j)];
        local += mine4[j];
      }
      unsigned all;
      unsigned before = block_exclusive_scan(local, sh.warp_sum, &all);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if ((long long)before < k_rem && k_rem <= (long long)before + mine4[j]) {
          sh.found_digit = kBins - 1 - (threadIdx.x * 4 + j);
          sh.found_before = before;
        }
        before += mine4[j];
      }
      __syncthreads();
      prefix_val |= sh.found_digit << shift;
      prefix_mask |= dmask << shift;
      k_rem -= sh.found_before;
      __syncthreads();
    }
  }
  const unsigned tau = k_sel > 0 ? prefix_val : 0xffffffffu;
  const unsigned ties_wanted = k_sel > 0 ? (unsigned)k_rem : 0u;  // >= 1 when k_sel > 0

  // ---- counts per warp, then the number of kept entries / ties before this warp ---------------
  unsigned n_gt = 0, n_eq = 0;
#pragma unroll
  for (int i = 0; i < E; ++i) {
    const bool valid = wbase + i * 32 + lane < c1;
    n_gt += __popc(__ballot_sync(0xffffffffu, valid && key[i] > tau));
    n_eq += __popc(__ballot_sync(0xffffffffu, valid && key[i] == tau));
  }
  if (lane == 0) sh.warp_cnt[warp] = make_uint2(n_gt, n_eq);
  cluster.sync();
  // warps in element order: (CTA rank, warp); lane l folds entries l, l + 32, ...
  unsigned kept_base = 0, tie_base = 0;
  {
    const int mine = rank * kWarps + warp;  // entries before this warp
    // ties are taken in order, so the kept count needs a sequential fold over the tie counts;
    // lanes first add up the "above" counts and the ties of their entries, in order
    unsigned gt_sum = 0, eq_sum = 0;
    for (int e = lane; e < mine; e += 32) {
      const uint2 c = cluster.map_shared_rank(sh.warp_cnt, e / kWarps)[e % kWarps];
      gt_sum += c.x;
      eq_sum += c.y;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      gt_sum += __shfl_xor_sync(0xffffffffu, gt_sum, o);
      eq_sum += __shfl_xor_sync(0xffffffffu, eq_sum, o);
    }
    tie_base = eq_sum;                                   // ties in earlier warps
    kept_base = gt_sum + min(eq_sum, ties_wanted);       // the earliest ties are the ones taken
  }
  cluster.sync();  // counts stay valid until every CTA has read them

  // ---- ordered emit ------------------------------------------------------------------------------
  int head = 0, pos = 0;
  if (s.prefix > 0) {
    const int first = wbase + lane;
    head = first / s.prefix;
    pos = first - head * s.prefix;
  }
  unsigned kept_run = kept_base, tie_run = tie_base;
#pragma unroll
  for (int i = 0; i < E; ++i) {
    const int idx = wbase + i * 32 + lane;
    const bool valid = idx < c1;
    const bool gt = valid && key[i] > tau, eq = valid && key[i] == tau;
    const unsigned eq_mask = __ballot_sync(0xffffffffu, eq);
    const unsigned lt = (1u << lane) - 1u;
    const bool keep = gt || (eq && tie_run + __popc(eq_mask & lt) < ties_wanted);
    const unsigned keep_mask = __ballot_sync(0xffffffffu, keep);
    const unsigned my_slot = kept_run + __popc(keep_mask & lt);
    if (valid) {
      if (keep) out[my_slot] = pos;
      // the first entry of a head records how many kept entries precede the head
      if (pos == 0) hoff[head] = (int)my_slot + head * g.window;
    }
    kept_run += __popc(keep_mask);
    tie_run += __popc(eq_mask);
    pos += 32;
    while (s.prefix > 0 && pos >= s.prefix) {
      pos -= s.prefix;
      ++head;
    }
  }
  if (rank == 0 && threadIdx.x == 0) {
    hoff[g.n_kv_heads] = (int)(k_sel + window_rows);
    if (s.prefix == 0)  // no candidates: every head holds only its (possibly short) window
      for (int h = 0; h < g.n_kv_heads; ++h) hoff[h] = h * min(g.window, s.n);
  }
}

template <int E>
cudaError_t launch_reg(const Geom& g, int problems, int csize, const float* scores,
                       const long long* layer_budget, int* keep_idx, int* head_offsets,
                       cudaStream_t stream) {
  auto kern = select_topk_reg_kernel<E>;
  if (csize > 8) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(csize * problems);
  cfg.blockDim = dim3(kThreads);
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = csize;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, g, scores, layer_budget, keep_idx, head_offsets);
}

}  // namespace

lava_status launch_select(const Geom& g, int n_layers, const float* scores,
                          const long long* layer_budget, int* keep_idx, int* head_offsets,
                          unsigned* status, cudaStream_t stream) {
  (void)status;
  // candidates of the largest problem; the register-resident kernel takes up to 32768 per CTA
  const long long m_max = (long long)g.n_kv_heads * (g.max_seqlen > g.window ? g.max_seqlen - g.window : 0);
  const int problems = n_layers * g.batch;
  const int csize = m_max <= 8LL * kRegMaxPerCta ? 8 : 16;
  if (m_max <= (long long)csize * kRegMaxPerCta) {
    const long long per = (m_max + csize - 1) / csize;
    const int e = (int)((per + kThreads - 1) / kThreads);  // keys per thread
    cudaError_t err;
    if (e <= 8) err = launch_reg<8>(g, problems, csize, scores, layer_budget, keep_idx, head_offsets, stream);
    else if (e <= 16) err = launch_reg<16>(g, problems, csize, scores, layer_budget, keep_idx, head_offsets, stream);
    else if (e <= 32) err = launch_reg<32>(g, problems, csize, scores, layer_budget, keep_idx, head_offsets, stream);
    else err = launch_reg<64>(g, problems, csize, scores, layer_budget, keep_idx, head_offsets, stream);
    count_launches(1);
    return check_cuda(err, "select_topk launch");
  }
  dim3 grid(kCluster, n_layers * g.batch);
  select_topk_kernel<<<grid, kThreads, 0, stream>>>(g, scores, layer_budget, keep_idx,
                                                    head_offsets);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "select_topk launch");
}

}  // namespace lava
