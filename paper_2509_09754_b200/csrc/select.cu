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
  if (batch_has_short_sequence(g)) return;  // every CTA of the cluster sees the same lengths
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
        // Scores of one layer crowd into a few exponent buckets, so most lanes of a row share
        // the digit of the first active lane: those are counted by one atomic, the rest add
        // their own (spread digits rarely collide).
        const unsigned active = __ballot_sync(0xffffffffu, mine);
        if (active) {
          const int leader = __ffs(active) - 1;
          const unsigned d0 = __shfl_sync(0xffffffffu, digit, leader);
          const unsigned same = __ballot_sync(0xffffffffu, mine && digit == d0);
          if ((int)(threadIdx.x & 31) == leader) atomicAdd(&sh.hist[d0], (unsigned)__popc(same));
          else if (mine && digit != d0) atomicAdd(&sh.hist[digit], 1u);
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
// Register-resident variant: every thread keeps E consecutive keys in registers for all passes,
// so element order is thread order and nothing in the passes or the emit needs a warp vote.
// Keys reach the registers through a padded shared-memory staging area (coalesced global reads,
// conflict-free 16-byte shared reads).  The digit histogram is kept in kRep interleaved copies
// (copy = lane mod kRep): layer scores crowd into a few exponent buckets, and a single copy
// would serialise the shared-memory atomics of a warp on those few addresses.  Kept positions
// are packed in shared memory and leave with coalesced stores.  Serves problems of up to 32768
// keys per CTA (cluster of 8 or 16 CTAs); larger ones take the streaming kernel above.
// ------------------------------------------------------------------------------------------
constexpr int kRegMaxPerCta = 32768;

struct RegShared {
  unsigned hist[kBins];    // this CTA's folded histogram; peers read it through DSMEM
  unsigned total[kBins];   // cluster-wide histogram (peers write their share of the bins)
  unsigned warp_sum[kWarps + 1];
  unsigned found_digit, found_before;
  uint2 cta_cnt;           // (above tau, equal to tau) inside this CTA; peers read it
};

template <int E>
struct RegCfg {
  static constexpr int kRep = E >= 64 ? 16 : E >= 32 ? 8 : 4;  // histogram copies
  static constexpr int kMinCtas = E >= 64 ? 1 : 2;  // CTAs per SM the kernel is compiled for
  static constexpr int kPad = E + 4;             // staging words per thread (bank spread)
  static constexpr int kStageWords = kThreads * kPad;
  static constexpr int kHistWords = kBins * kRep;
  static constexpr int kBigWords = kStageWords > kHistWords ? kStageWords : kHistWords;
};

// LIST selects among the entries a layer still holds (Algorithm 2: a lower layer is evicted
// again with its stored scores): the keys of problem p are the `held` scores of its list, in
// list order, which is ascending flat index, so ties still go to the lower flat index.  The
// kept entries' scores and positions are copied to the new list and `src_pos` records where in
// the old list each came from.
template <int E, bool LIST>
__global__ void __launch_bounds__(kThreads, RegCfg<E>::kMinCtas)
select_topk_reg_kernel(Geom g, const float* scores, const long long* layer_budget, int* keep_idx,
                       int* head_offsets, HeldLists io) {
  using Cfg = RegCfg<E>;
  if (batch_has_short_sequence(g)) return;  // every CTA of the cluster sees the same lengths
  extern __shared__ __align__(16) unsigned big[];  // staging / histogram copies / packed output
  __shared__ RegShared sh;
  cg::cluster_group cluster = cg::this_cluster();
  const int csize = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  // one cluster per (layer, sequence); with per-head selection (the "- head dynamic" ablation of
  // Sec. 5.4) one per (layer, sequence, KV head), each on its head's segment alone
  const bool per_head = !LIST && (g.flags & LAVA_FLAG_PER_HEAD_TOPK) != 0;
  const int cl = blockIdx.x / csize;
  const int prob = per_head ? cl / g.n_kv_heads : cl, layer = prob / g.batch, b = prob - layer * g.batch;
  const int head0 = per_head ? cl - prob * g.n_kv_heads : 0;  // first head of this problem
  const int lane = threadIdx.x & 31;
  const SeqInfo s = seq_info(g, b);
  const int win = min(g.window, s.n);
  const int* hoff_old = LIST ? io.hoff_old + (size_t)prob * (g.n_kv_heads + 1) : nullptr;
  // candidates (fits 31 bits): the whole prefix of every head, or what the list still holds
  const int m_total = LIST ? max(0, hoff_old[g.n_kv_heads] - g.n_kv_heads * win)
                           : (per_head ? 1 : g.n_kv_heads) * s.prefix;
  const long long window_rows = (long long)g.n_kv_heads * win;
  long long k_sel = layer_budget[prob] - window_rows;
  if (k_sel < 0) k_sel = 0;
  int out_base = 0;  // kept entries of the heads before this problem's first head
  if (per_head) {
    // even shares of the selectable entries, the first (k mod H_kv) heads one more; a head
    // never keeps more than it has
    const long long share = k_sel / g.n_kv_heads, extra = k_sel % g.n_kv_heads;
    out_base = share >= s.prefix ? head0 * s.prefix
                                 : (int)(head0 * share + min((long long)head0, extra));
    k_sel = share + (head0 < extra ? 1 : 0);
  }
  if (k_sel > m_total) k_sel = m_total;
  const long long old0 = LIST ? io.row_off_old[prob] : 0, new0 = LIST ? io.row_off_new[prob] : 0;
  const unsigned* keys = reinterpret_cast<const unsigned*>(
      LIST ? io.score_old + old0
           : scores + (size_t)layer * g.total_scores + s.score_off + (long long)head0 * s.prefix);
  int* out = LIST ? io.pos_new + new0
                  : keep_idx + (size_t)layer * g.total_scores + s.score_off + out_base;
  int* hoff = head_offsets + (size_t)prob * (g.n_kv_heads + 1);

  // this CTA's range; thread t owns its elements [t E, t E + E)
  const int per = (m_total + csize - 1) / csize;
  const int c0 = min(m_total, per * rank), c1 = min(m_total, c0 + per);
  const int n_cta = c1 - c0;
  const int n_mine = max(0, min(E, n_cta - (int)threadIdx.x * E));  // valid keys of this thread
#pragma unroll 8
  for (int i = threadIdx.x; i < n_cta; i += kThreads)
    big[(i / E) * Cfg::kPad + (i % E)] = keys[c0 + i];
  __syncthreads();
  unsigned key[E];
#pragma unroll
  for (int j = 0; j < E; j += 4) {
    const uint4 q = *reinterpret_cast<const uint4*>(&big[threadIdx.x * Cfg::kPad + j]);
    key[j] = q.x;
    key[j + 1] = q.y;
    key[j + 2] = q.z;
    key[j + 3] = q.w;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < Cfg::kHistWords / 4; i += kThreads)
    reinterpret_cast<uint4*>(big)[i] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();

  // ---- radix passes: find tau and the number of ties to take -------------------------------
  unsigned prefix_val = 0, prefix_mask = 0;
  long long k_rem = k_sel;
  if (k_sel > 0) {
    const int shifts[3] = {21, 10, 0};
    const int widths[3] = {11, 11, 10};
    unsigned* my_copy = big + (lane & (Cfg::kRep - 1));
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = shifts[pass];
      const unsigned dmask = (1u << widths[pass]) - 1u;
#pragma unroll
      for (int j = 0; j < E; ++j) {
        const unsigned digit = (key[j] >> shift) & dmask;
        if (j < n_mine && (key[j] & prefix_mask) == prefix_val)
          atomicAdd(&my_copy[digit * Cfg::kRep], 1u);
      }
      __syncthreads();
      // Fold the copies and clear them: consecutive lanes take consecutive 16-byte pieces
      // (conflict-free); kRep / 4 neighbouring lanes hold the pieces of one bin.
      for (int i = threadIdx.x; i < Cfg::kHistWords / 4; i += kThreads) {
        uint4* cell = reinterpret_cast<uint4*>(big) + i;
        const uint4 q = *cell;
        *cell = make_uint4(0u, 0u, 0u, 0u);
        unsigned sum = q.x + q.y + q.z + q.w;
#pragma unroll
        for (int o = 1; o < Cfg::kRep / 4; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if ((i & (Cfg::kRep / 4 - 1)) == 0) sh.hist[i / (Cfg::kRep / 4)] = sum;
      }
      cluster.sync();  // every CTA's histogram is complete
      // CTA r sums bins [r * kBins / csize, ...) over the cluster and hands the sums to every
      // CTA: each thread issues independent remote loads, then csize remote stores.
      {
        const int share = kBins / csize;  // 256 or 128
        if ((int)threadIdx.x < share) {
          const int bin = rank * share + threadIdx.x;
          unsigned sum = 0;
          for (int r0 = 0; r0 < csize; r0 += 8) {  // cluster sizes are 8 and 16
            unsigned part[8];
#pragma unroll
            for (int r = 0; r < 8; ++r) part[r] = cluster.map_shared_rank(sh.hist, r0 + r)[bin];
#pragma unroll
            for (int r = 0; r < 8; ++r) sum += part[r];
          }
          for (int r = 0; r < csize; ++r) cluster.map_shared_rank(sh.total, r)[bin] = sum;
        }
      }
      cluster.sync();  // all sums have arrived; peers have finished reading this CTA's histogram
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

  // ---- counts: per thread, then block scan (both counts packed, each at most 32768) ----------
  unsigned n_gt = 0, n_eq = 0;
#pragma unroll
  for (int j = 0; j < E; ++j) {
    n_gt += (j < n_mine && key[j] > tau) ? 1u : 0u;
    n_eq += (j < n_mine && key[j] == tau) ? 1u : 0u;
  }
  unsigned cta_packed;
  const unsigned before_packed = block_exclusive_scan(n_gt | (n_eq << 16), sh.warp_sum, &cta_packed);
  const unsigned gt_before = before_packed & 0xffffu, eq_before = before_packed >> 16;
  const unsigned cta_gt = cta_packed & 0xffffu, cta_eq = cta_packed >> 16;
  if (threadIdx.x == 0) sh.cta_cnt = make_uint2(cta_gt, cta_eq);
  cluster.sync();
  unsigned gt_cta_before = 0, eq_cta_before = 0;  // counts in the CTAs before this one
#pragma unroll
  for (int r = 0; r < 16; ++r)
    if (r < rank) {
      const uint2 c = *cluster.map_shared_rank(&sh.cta_cnt, r);
      gt_cta_before += c.x;
      eq_cta_before += c.y;
    }
  // ties are taken in element order: the earliest ties_wanted of them
  const unsigned ties_before_cta = min(eq_cta_before, ties_wanted);
  const unsigned kept_cta_before = gt_cta_before + ties_before_cta;
  const unsigned cta_kept = cta_gt + (min(eq_cta_before + cta_eq, ties_wanted) - ties_before_cta);

  // ---- ordered emit: pack the kept positions in shared memory, then store them coalesced -----
  {
    const unsigned tie0 = eq_cta_before + eq_before;  // index of this thread's first tie
    const unsigned slot0 = gt_before + (min(tie0, ties_wanted) - ties_before_cta);  // in the CTA
    // bit j of keep_mask: key j is retained (above tau, or one of the first ties_wanted ties)
    unsigned long long keep_mask = 0ull;
    {
      unsigned ties_seen = 0;
#pragma unroll
      for (int j = 0; j < E; ++j) {
        const bool eq = j < n_mine && key[j] == tau;
        const bool keep = (j < n_mine && key[j] > tau) || (eq && tie0 + ties_seen < ties_wanted);
        keep_mask |= (unsigned long long)keep << j;
        ties_seen += eq ? 1u : 0u;
      }
    }
    int* packed = reinterpret_cast<int*>(big);
    if (LIST) {
      if (n_mine > 0) {
        const int first = c0 + (int)threadIdx.x * E;
        // heads whose list segment starts inside this thread's keys
        for (int h = 0; h < g.n_kv_heads; ++h) {
          const int j = hoff_old[h] - h * win - first;
          if (j >= 0 && j < n_mine)
            hoff[h] = (int)(kept_cta_before + slot0) + __popcll(keep_mask & ((1ull << j) - 1ull)) +
                      h * win;
        }
#pragma unroll
        for (int j = 0; j < E; ++j)
          if ((keep_mask >> j) & 1ull)
            packed[slot0 + __popcll(keep_mask & ((1ull << j) - 1ull))] = first + j;
      }
      __syncthreads();
      for (unsigned i = threadIdx.x; i < cta_kept; i += kThreads) {
        const int p = packed[i];
        const long long o = new0 + kept_cta_before + i;
        io.pos_new[o] = io.pos_old[old0 + p];
        io.score_new[o] = io.score_old[old0 + p];
        io.src_pos[o] = p;
      }
    } else {
    if (n_mine > 0) {
      const int first = c0 + (int)threadIdx.x * E;
      int head = first / s.prefix;
      const int pos0 = first - head * s.prefix;
      // heads that start inside this thread's keys record how many kept entries precede them
      for (int j = pos0 == 0 ? 0 : s.prefix - pos0; j < n_mine; j += s.prefix) {
        const int h = head0 + (first + j) / s.prefix;
        hoff[h] = out_base + (int)(kept_cta_before + slot0) +
                  __popcll(keep_mask & ((1ull << j) - 1ull)) + h * g.window;
      }
#pragma unroll
      for (int j = 0; j < E; ++j) {
        int pos = pos0 + j;
        while (pos >= s.prefix) pos -= s.prefix;  // at most once unless heads are shorter than E
        if ((keep_mask >> j) & 1ull)
          packed[slot0 + __popcll(keep_mask & ((1ull << j) - 1ull))] = pos;
      }
    }
    __syncthreads();
    for (unsigned i = threadIdx.x; i < cta_kept; i += kThreads) out[kept_cta_before + i] = packed[i];
    }
  }
  if (rank == 0 && threadIdx.x == 0) {
    if (LIST) {
      // heads whose segment starts past the last held entry (empty tail heads, or an empty list)
      for (int h = 0; h < g.n_kv_heads; ++h)
        if (hoff_old[h] - h * win >= m_total) hoff[h] = (int)k_sel + h * win;
      hoff[g.n_kv_heads] = (int)k_sel + g.n_kv_heads * win;
    } else if (!per_head) {
      hoff[g.n_kv_heads] = (int)(k_sel + window_rows);
      if (s.prefix == 0)  // no candidates: every head holds only its (possibly short) window
        for (int h = 0; h < g.n_kv_heads; ++h) hoff[h] = h * win;
    } else {
      if (s.prefix == 0) hoff[head0] = head0 * win;
      if (head0 == g.n_kv_heads - 1) hoff[g.n_kv_heads] = out_base + (int)k_sel + (int)window_rows;
    }
  }
  cluster.sync();  // peers may still be reading this CTA's counts
}

template <int E, bool LIST = false>
cudaError_t launch_reg(const Geom& g, int problems, int csize, const float* scores,
                       const long long* layer_budget, int* keep_idx, int* head_offsets,
                       cudaStream_t stream, HeldLists io = HeldLists()) {
  auto kern = select_topk_reg_kernel<E, LIST>;
  const int big_bytes = RegCfg<E>::kBigWords * (int)sizeof(unsigned);
  {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, big_bytes);
    if (e != cudaSuccess) return e;
  }
  if (csize > 8) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(csize * problems);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = big_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = csize;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, g, scores, layer_budget, keep_idx, head_offsets, io);
}

}  // namespace

lava_status launch_select(const Geom& g, int n_layers, const float* scores,
                          const long long* layer_budget, int* keep_idx, int* head_offsets,
                          unsigned* status, cudaStream_t stream) {
  (void)status;
  const bool per_head = (g.flags & LAVA_FLAG_PER_HEAD_TOPK) != 0;
  // candidates of the largest problem; the register-resident kernel takes up to 32768 per CTA
  const long long m_max = (long long)(per_head ? 1 : g.n_kv_heads) *
                          (g.max_seqlen > g.window ? g.max_seqlen - g.window : 0);
  const int problems = n_layers * g.batch * (per_head ? g.n_kv_heads : 1);
  // 16 CTAs once a cluster of 8 would need 64 keys per thread: at 32 keys per thread two CTAs
  // share an SM
  int csize = m_max <= 8LL * (kRegMaxPerCta / 2) ? 8 : 16;
  if (options().select_cluster == 8 && m_max <= 8LL * kRegMaxPerCta) csize = 8;
  if (options().select_cluster == 16) csize = 16;
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
  if (per_head)
    return fail(LAVA_ERR_UNSUPPORTED, "per-head selection covers up to 524288 positions per head");
  dim3 grid(kCluster, n_layers * g.batch);
  select_topk_kernel<<<grid, kThreads, 0, stream>>>(g, scores, layer_budget, keep_idx,
                                                    head_offsets);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "select_topk launch");
}

lava_status launch_reselect(const Geom& g, int problems, long long max_held,
                            const long long* layer_budget, int* head_offsets_new,
                            const HeldLists& io, cudaStream_t stream) {
  if (problems < 1) return LAVA_OK;
  int csize = max_held <= 8LL * (kRegMaxPerCta / 2) ? 8 : 16;
  if (max_held > (long long)csize * kRegMaxPerCta)
    return fail(LAVA_ERR_UNSUPPORTED, "a layer may hold at most %d entries per sequence here",
                16 * kRegMaxPerCta);
  const long long per = (max_held + csize - 1) / csize;
  const int e = (int)((per + kThreads - 1) / kThreads);
  cudaError_t err;
  if (e <= 8) err = launch_reg<8, true>(g, problems, csize, nullptr, layer_budget, nullptr, head_offsets_new, stream, io);
  else if (e <= 16) err = launch_reg<16, true>(g, problems, csize, nullptr, layer_budget, nullptr, head_offsets_new, stream, io);
  else if (e <= 32) err = launch_reg<32, true>(g, problems, csize, nullptr, layer_budget, nullptr, head_offsets_new, stream, io);
  else err = launch_reg<64, true>(g, problems, csize, nullptr, layer_budget, nullptr, head_offsets_new, stream, io);
  count_launches(1);
  return check_cuda(err, "reselect launch");
}

}  // namespace lava
