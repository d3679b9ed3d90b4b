// LAVa score, Blackwell single-pass path: bf16, head_dim 128, w in {16, 32, 64, 128}, pooling
// radius up to 4, sequences short enough that the exponentials of a whole head fit the tensor
// memory of the GPU (about 54K tokens; 18K when a query group needs two units).
//
// The softmax of a window query (Sec. 2) needs the row's normaliser over ALL keys before any
// probability can be added to the window mean of Definition 1.  Here every logit is computed and
// exponentiated exactly once: the key axis of a head is dealt tile by tile to all CTAs, each CTA
// keeps the exponentials of its tiles in tensor memory, the per-tile row statistics meet in
// global memory, and the window mean is formed from the stored exponentials once the head's
// normalisers are known.  K and V are read from HBM once.
//
// One persistent CTA per SM (cooperative launch: the CTAs wait on one another's flags).  A job
// is one 128-key tile of one unit (a KV head, or one half of its query group when the group has
// more than 128 window-query rows); tiles overlap by twice the pooling radius so that every
// owned key finds its pooling neighbours inside its own tile.  Jobs are dealt round-robin, and
// each CTA runs its jobs through four accumulator buffers of 128 columns:
//
//   producer warp     TMA: the K tile (once per K tile, shared by the two units of a split
//                     group) and the unit's query tile, into 128B-swizzled shared memory
//   MMA warp          S = Q_u K^T (rows = window queries, columns = keys) into tensor memory
//   4 statistics      one thread per window-query row: running maximum per 32-column block,
//     warps           e = exp2(z - max) written back over the logits, the row's sum over the
//                     keys the tile owns; the tile's log2-sum-exp per row goes to the publisher
//   publisher warp    writes the tile's row statistics to global memory and counts them; the
//                     CTA that delivers the last tile of a group of 16 folds the group, the one
//                     that completes the last group folds the head and raises its flag (fixed
//                     order of operations: the result does not depend on who folds)
//   prep warp         waits for the flag of the next job's head (and for its value norm),
//                     fetches the head's log2-sum-exp per row
//   4 score warps     one thread per row: e * exp2(block max - lse) / w, summed over the rows of
//                     each query head through shared memory (Definition 1), pooled (Sec. 5.1),
//                     scaled by Vbar * c_hat, reduced with the group maximum (Sec. 4.3), written
//                     once; entropy sums of Sec. 4.2 go to per-tile slots
//   8 value warps     stream the V rows of the CTA's tiles for max_k ||V[k]||_1 (Theorem 1)
//
// A head's tiles lie in at most four consecutive rounds of jobs (two when units are split), and
// the statistics warps run at most three jobs ahead of the score warps, so every wait for a
// head's flag ends (the launcher checks the bound).  Every wait is bounded in time all the same.
#include "sm100_ptx.cuh"

namespace lava {
namespace {

using namespace sm100;

constexpr int kTile = 128;
constexpr int kThreads = 640;        // 20 warps: 4 service, 4 statistics, 4 score, 8 value
constexpr int kVWarps = 8;
constexpr int kAcc = 4;              // accumulator buffers (128 TMEM columns each)
constexpr int kKStages = 3;
constexpr int kMaxBatch = 512;
constexpr int kFold = 16;            // tiles per first-level fold
constexpr int kMaxRadius = 4;
constexpr uint32_t kTileBytes = 128 * 128 * 2;
constexpr uint32_t kHalfBytes = kTileBytes / 2;
constexpr int kScrStride = 36;       // words per row of a score warp's transposition scratch

constexpr uint32_t kOffQ = 0;                                   // 2 query tiles
constexpr uint32_t kOffK = kOffQ + 2 * kTileBytes;              // 3 key tiles
constexpr uint32_t kOffScr = kOffK + kKStages * kTileBytes;     // 4 warps x 2 x [32][36] floats
constexpr uint32_t kScrBytes = 4 * 2 * 32 * kScrStride * 4;
constexpr uint32_t kOffCtl = kOffScr + kScrBytes;

struct Ctl {
  unsigned long long k_full[kKStages], k_empty[kKStages], q_full[2], q_empty[2];
  unsigned long long acc_full[kAcc], acc_empty[kAcc], e_ready[kAcc];
  unsigned long long pub_full[kAcc], pub_empty[kAcc], prep_full[kAcc], prep_empty[kAcc];
  unsigned long long bsync, drain;
  uint32_t tmem_base;
  volatile int abort_flag;
  long long wait_cycles;
  int tiles_layer;                    // K tiles of one layer: H_kv * sum over sequences
  float scale[kAcc];                  // Vbar * c_hat of the job's head
  alignas(16) float pub[kAcc][128];   // log2-sum-exp per row of a finished tile
  alignas(16) float lse_tab[kAcc][128];  // the head's log2-sum-exp per row
  alignas(16) float4 mtab[kAcc][128]; // the four block maxima of every row of a tile
  alignas(16) float pbuf[4][2][kTile];   // per score warp (and half warp when w = 16): row sums
  alignas(16) float abuf[4][kTile];   // window means per query head (or their maximum)
  int pref[kMaxBatch + 1];            // exclusive scan of tiles per sequence
};
constexpr uint32_t kSmemBytes = kOffCtl + sizeof(Ctl) + 1024;
static_assert(kSmemBytes <= 232448, "shared memory budget");

struct TmemParams {
  Geom g;
  int n_layers;
  int ok;                   // keys a tile owns: 128 - 2 * pool_radius
  int nunit;                // units per KV head: 1, or 2 when the query group is split
  int g0;                   // query heads in the first unit (split mode)
  int gmax;                 // first-level fold groups per unit at max_seqlen
  long long wait_cycles;
  const float* vbar_in;
  float* scores;
  const char* v;
  long long v_ls;
  // scratch
  float* part;              // [jobs][128] log2-sum-exp per tile and row
  float* gpart;             // [units][gmax][128] per group of kFold tiles
  float* head_lse;          // [units][128]
  int* gcount;              // [units][gmax]
  int* hcount;              // [units]
  int* flag;                // [units]
  int* vcount;              // [KV heads] finished value-norm slabs
  unsigned* vbar_bits;      // [KV heads]
  float2* ent_part;         // [K tiles][4] (sum s, sum s ln s) per score warp
  unsigned* status;
};

struct KJob {
  int layer, b, kvh, tile, ntiles;
  SeqInfo s;
};

__device__ inline KJob decode_job(const TmemParams& p, const Ctl* m, long long kappa) {
  KJob kj;
  kj.layer = (int)(kappa / m->tiles_layer);
  const int r = (int)(kappa - (long long)kj.layer * m->tiles_layer);
  int lo = 0, hi = p.g.batch;  // largest b with H_kv * pref[b] <= r
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (p.g.n_kv_heads * m->pref[mid] <= r) lo = mid; else hi = mid;
  }
  kj.b = lo;
  kj.ntiles = m->pref[lo + 1] - m->pref[lo];
  const int r2 = r - p.g.n_kv_heads * m->pref[lo];
  kj.kvh = r2 / kj.ntiles;
  kj.tile = r2 - kj.kvh * kj.ntiles;
  kj.s = seq_info(p.g, lo);
  return kj;
}

// Running (maximum, sum of exp2) fold of `count` rows of log2-sum-exp values, four rows' worth of
// components per lane, 16 rows per round, always in row order.
__device__ inline float4 fold_rows(const float4* rows, size_t stride, int count) {
  float big[4], sum[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    big[q] = -INFINITY;
    sum[q] = 0.f;
  }
#pragma unroll 1
  for (int i0 = 0; i0 < count; i0 += 16) {
    float4 pr[16];
#pragma unroll
    for (int u = 0; u < 16; ++u)
      pr[u] = (i0 + u < count) ? __ldcg(rows + (size_t)(i0 + u) * stride)
                               : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float l[16];
#pragma unroll
      for (int u = 0; u < 16; ++u)
        l[u] = q == 0 ? pr[u].x : q == 1 ? pr[u].y : q == 2 ? pr[u].z : pr[u].w;
      float bm = l[0];
#pragma unroll
      for (int u = 1; u < 16; ++u) bm = fmaxf(bm, l[u]);
      const float nb = fmaxf(big[q], bm);
      const float ref = nb == -INFINITY ? 0.f : nb;  // keeps -inf - -inf out of the exponent
      float acc = sum[q] * fast_exp2(big[q] - ref);
#pragma unroll
      for (int u = 0; u < 16; ++u) acc += fast_exp2(l[u] - ref);
      sum[q] = acc;
      big[q] = nb;
    }
  }
  float4 out;
  out.x = sum[0] > 0.f ? big[0] + fast_log2(sum[0]) : -INFINITY;
  out.y = sum[1] > 0.f ? big[1] + fast_log2(sum[1]) : -INFINITY;
  out.z = sum[2] > 0.f ? big[2] + fast_log2(sum[2]) : -INFINITY;
  out.w = sum[3] > 0.f ? big[3] + fast_log2(sum[3]) : -INFINITY;
  return out;
}

// Sum of 32 values by a fixed tree that leaves the inputs untouched.
__device__ inline float tree_sum32_keep(const float (&c)[32]) {
  float t[16];
#pragma unroll
  for (int i = 0; i < 16; i += 2) {
    const float2 r = __fadd2_rn(make_float2(c[i], c[i + 1]), make_float2(c[i + 16], c[i + 17]));
    t[i] = r.x;
    t[i + 1] = r.y;
  }
#pragma unroll
  for (int i = 0; i < 8; i += 2) {
    const float2 r = __fadd2_rn(make_float2(t[i], t[i + 1]), make_float2(t[i + 8], t[i + 9]));
    t[i] = r.x;
    t[i + 1] = r.y;
  }
#pragma unroll
  for (int i = 0; i < 4; i += 2) {
    const float2 r = __fadd2_rn(make_float2(t[i], t[i + 1]), make_float2(t[i + 4], t[i + 5]));
    t[i] = r.x;
    t[i + 1] = r.y;
  }
  return (t[0] + t[1]) + (t[2] + t[3]);
}

__global__ void __launch_bounds__(kThreads, 1)
lava_score_tmem_kernel(const __grid_constant__ CUtensorMap map_q,
                       const __grid_constant__ CUtensorMap map_k, const TmemParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  Ctl* m = reinterpret_cast<Ctl*>(gen + kOffCtl);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const Geom& g = p.g;
  const int W = g.window, rad = g.pool_radius, nunit = p.nunit;

  // ---- tiles per sequence (exclusive scan), barriers, tensor memory ---------------------------
  {
    __shared__ int wsum[kThreads / 32];
    int c = 0;
    if ((int)threadIdx.x < g.batch) {
      const SeqInfo s = seq_info(g, threadIdx.x);
      if (s.n < g.window && blockIdx.x == 0) atomicOr(p.status, LAVA_DEV_SHORT_SEQUENCE);
      c = ceil_div(s.n, p.ok);
    }
    int inc = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += y;
    }
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    int before = 0;
    for (int wdx = 0; wdx < warp; ++wdx) before += wsum[wdx];
    if ((int)threadIdx.x < g.batch) m->pref[threadIdx.x + 1] = before + inc;
    if (threadIdx.x == 0) m->pref[0] = 0;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    m->tiles_layer = g.n_kv_heads * m->pref[g.batch];
    for (int s = 0; s < kKStages; ++s) {
      mbar_init(smem_u32(&m->k_full[s]), 1);
      mbar_init(smem_u32(&m->k_empty[s]), 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&m->q_full[s]), 1);
      mbar_init(smem_u32(&m->q_empty[s]), 1);
    }
    for (int s = 0; s < kAcc; ++s) {
      mbar_init(smem_u32(&m->acc_full[s]), 1);
      mbar_init(smem_u32(&m->acc_empty[s]), 4);   // one arrival per score warp
      mbar_init(smem_u32(&m->e_ready[s]), 4);     // one arrival per statistics warp
      mbar_init(smem_u32(&m->pub_full[s]), 4);
      mbar_init(smem_u32(&m->pub_empty[s]), 1);
      mbar_init(smem_u32(&m->prep_full[s]), 1);
      mbar_init(smem_u32(&m->prep_empty[s]), 4);
    }
    mbar_init(smem_u32(&m->bsync), 4);
    mbar_init(smem_u32(&m->drain), 1);
    m->abort_flag = 0;
    m->wait_cycles = p.wait_cycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&m->tmem_base), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = m->tmem_base;
  const long long total_k = (long long)p.n_layers * m->tiles_layer;  // K tiles of the launch
  const float sc2 = g.scale_log2;

  if (warp == 0) {
    // ================= producer: K tile once per K tile, query tile once per job ===============
    if (lane == 0) {
      long long nk = 0, nq = 0;
      bool ok = true;
      for (long long kappa = blockIdx.x; kappa < total_k && ok && !m->abort_flag;
           kappa += gridDim.x) {
        const KJob kj = decode_job(p, m, kappa);
        const int st = (int)(nk % kKStages);
        ok = wait_bar(smem_u32(&m->k_empty[st]), (uint32_t)((nk / kKStages) & 1) ^ 1, m, p.status);
        if (!ok) break;
        {
          const uint32_t bar = smem_u32(&m->k_full[st]);
          mbar_expect_tx(bar, kTileBytes);
          // the tile starts pool_radius keys before the first key it owns
          const int tok = (int)kj.s.tok0 + kj.tile * p.ok - rad;
          tma_load_4d_plain(base + kOffK + st * kTileBytes, &map_k, 0, tok, kj.kvh, kj.layer, bar);
          tma_load_4d_plain(base + kOffK + st * kTileBytes + kHalfBytes, &map_k, 64, tok, kj.kvh,
                            kj.layer, bar);
          ++nk;
        }
        for (int half = 0; half < nunit && ok; ++half) {
          const int qs = (int)(nq & 1);
          ok = wait_bar(smem_u32(&m->q_empty[qs]), (uint32_t)((nq >> 1) & 1) ^ 1, m, p.status);
          if (!ok) break;
          const uint32_t bar = smem_u32(&m->q_full[qs]);
          mbar_expect_tx(bar, kTileBytes);
          const int row0 = (kj.b * g.n_q_heads + kj.kvh * g.group + half * p.g0) * W;
          tma_load_3d(base + kOffQ + qs * kTileBytes, &map_q, 0, row0, kj.layer, bar);
          tma_load_3d(base + kOffQ + qs * kTileBytes + kHalfBytes, &map_q, 64, row0, kj.layer, bar);
          ++nq;
        }
      }
      // copies still in flight land before this CTA gives up its shared memory
      for (long long j = (nk > kKStages ? nk - kKStages : 0); j < nk; ++j)
        wait_bar(smem_u32(&m->k_full[j % kKStages]), (uint32_t)((j / kKStages) & 1), m, p.status,
                 false);
      for (long long j = (nq > 2 ? nq - 2 : 0); j < nq; ++j)
        wait_bar(smem_u32(&m->q_full[j & 1]), (uint32_t)((j >> 1) & 1), m, p.status, false);
    }
  } else if (warp == 1) {
    // ================= MMA issuer ==============================================================
    if (lane == 0) {
      long long nk = 0, j = 0;
      bool ok = true;
      for (long long kappa = blockIdx.x; kappa < total_k && ok; kappa += gridDim.x, ++nk) {
        const int st = (int)(nk % kKStages);
        ok = wait_bar(smem_u32(&m->k_full[st]), (uint32_t)((nk / kKStages) & 1), m, p.status);
        for (int half = 0; half < nunit && ok; ++half, ++j) {
          const int qs = (int)(j & 1), buf = (int)(j & (kAcc - 1));
          ok = wait_bar(smem_u32(&m->q_full[qs]), (uint32_t)((j >> 1) & 1), m, p.status) &&
               wait_bar(smem_u32(&m->acc_empty[buf]), (uint32_t)((j >> 2) & 1) ^ 1, m, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t d = tmem + (uint32_t)buf * 128u;
          const uint32_t qa = base + kOffQ + qs * kTileBytes, ka = base + kOffK + st * kTileBytes;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (uint32_t)(kk >> 2) * kHalfBytes + (uint32_t)(kk & 3) * 32u;
            umma_bf16(d, make_desc(qa + off), make_desc(ka + off), kIdesc, kk > 0);
          }
          umma_commit(smem_u32(&m->q_empty[qs]));
          umma_commit(smem_u32(&m->acc_full[buf]));
        }
        if (ok) umma_commit(smem_u32(&m->k_empty[st]));
      }
      // every MMA this thread issued has completed before TMEM is released
      umma_commit(smem_u32(&m->drain));
      wait_bar(smem_u32(&m->drain), 0, m, p.status, false);
    }
  } else if (warp == 2) {
    // ================= publisher: tile statistics leave the CTA; folds ========================
    long long j = 0;
    bool alive = true;
    for (long long kappa = blockIdx.x; kappa < total_k && alive; kappa += gridDim.x) {
      const KJob kj = decode_job(p, m, kappa);
      for (int half = 0; half < nunit && alive; ++half, ++j) {
        const int buf = (int)(j & (kAcc - 1));
        bool ok = true;
        if (lane == 0)
          ok = wait_bar(smem_u32(&m->pub_full[buf]), (uint32_t)((j >> 2) & 1), m, p.status);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) {
          alive = false;
          break;
        }
        const float4 mine = reinterpret_cast<const float4*>(m->pub[buf])[lane];
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&m->pub_empty[buf]));
        const long long job = kappa * nunit + half;               // index of this job's row
        const long long job0 = (kappa - kj.tile) * nunit + half;  // tile 0 of the unit
        reinterpret_cast<float4*>(p.part + (size_t)job * 128)[lane] = mine;
        __syncwarp();
        const int unit = ((kj.layer * g.batch + kj.b) * g.n_kv_heads + kj.kvh) * nunit + half;
        const int gi = kj.tile / kFold;
        const int gsz = min(kFold, kj.ntiles - gi * kFold);
        const int ngroups = ceil_div(kj.ntiles, kFold);
        int old = 0;
        if (lane == 0) old = atom_add_acq_rel(&p.gcount[(size_t)unit * p.gmax + gi], 1);
        old = __shfl_sync(0xffffffffu, old, 0);
        if (old != gsz - 1) continue;
        // the group is complete: fold its tiles, in tile order
        __syncwarp();
        {
          const float4* rows =
              reinterpret_cast<const float4*>(p.part + (size_t)(job0 + (long long)gi * kFold * nunit) * 128) + lane;
          const float4 gl = fold_rows(rows, (size_t)32 * nunit, gsz);
          reinterpret_cast<float4*>(p.gpart + ((size_t)unit * p.gmax + gi) * 128)[lane] = gl;
        }
        __syncwarp();
        if (lane == 0) old = atom_add_acq_rel(&p.hcount[unit], 1);
        old = __shfl_sync(0xffffffffu, old, 0);
        if (old != ngroups - 1) continue;
        // the head is complete: fold its groups, in group order, and raise the flag
        __syncwarp();
        {
          const float4* rows = reinterpret_cast<const float4*>(p.gpart + (size_t)unit * p.gmax * 128) + lane;
          const float4 hl = fold_rows(rows, 32, ngroups);
          reinterpret_cast<float4*>(p.head_lse + (size_t)unit * 128)[lane] = hl;
        }
        __syncwarp();
        if (lane == 0) st_release(&p.flag[unit], 1);
      }
    }
  } else if (warp == 3) {
    // ================= prep: the head's normalisers and value norm for the score warps =========
    long long j = 0;
    bool alive = true;
    for (long long kappa = blockIdx.x; kappa < total_k && alive; kappa += gridDim.x) {
      const KJob kj = decode_job(p, m, kappa);
      const int rhead = (kj.layer * g.batch + kj.b) * g.n_kv_heads + kj.kvh;
      for (int half = 0; half < nunit && alive; ++half, ++j) {
        const int buf = (int)(j & (kAcc - 1));
        const int unit = rhead * nunit + half;
        bool ok = true;
        if (lane == 0) {
          ok = wait_bar(smem_u32(&m->prep_empty[buf]), (uint32_t)((j >> 2) & 1) ^ 1, m, p.status);
          const int want_v = p.vbar_in ? 0 : kVWarps * kj.ntiles;
          const long long t0 = clock64();
          while (ok && (ld_acquire(&p.flag[unit]) == 0 ||
                        (want_v && ld_acquire(&p.vcount[rhead]) < want_v))) {
            if (m->abort_flag) ok = false;
            __nanosleep(64);
            if (clock64() - t0 > m->wait_cycles) {
              give_up(m, p.status);
              ok = false;
            }
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) {
          alive = false;
          break;
        }
        __syncwarp();
        reinterpret_cast<float4*>(m->lse_tab[buf])[lane] =
            __ldcg(reinterpret_cast<const float4*>(p.head_lse + (size_t)unit * 128) + lane);
        if (lane == 0) {
          const float vb = p.vbar_in ? p.vbar_in[rhead] : __uint_as_float(__ldcg(p.vbar_bits + rhead));
          m->scale[buf] = vb * g.c_hat;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&m->prep_full[buf]));
      }
    }
  } else if (warp >= 4 && warp < 8) {
    // ================= statistics warps: one thread per window-query row ======================
    const int quad = warp & 3, row = quad * 32 + lane;
    const int t_in_win = row & (W - 1);
    long long j = 0;
    bool alive = true;
    for (long long kappa = blockIdx.x; kappa < total_k && alive; kappa += gridDim.x) {
      const KJob kj = decode_job(p, m, kappa);
      const int i0 = kj.tile * p.ok - rad;  // key of column 0
      // every column is a prefix key that all window queries see
      const bool fast = i0 >= 0 && i0 + kTile <= kj.s.prefix;
      for (int half = 0; half < nunit && alive; ++half, ++j) {
        const int buf = (int)(j & (kAcc - 1));
        const int heads = nunit == 1 ? g.group : (half ? g.group - p.g0 : p.g0);
        // keys this query may see: i < n and i <= P + t (Sec. 2); rows beyond the unit see none
        const int last = row < heads * W ? min(kj.s.n, kj.s.prefix + t_in_win + 1) : 0;
        if (!__all_sync(0xffffffffu, wait_bar(smem_u32(&m->pub_empty[buf]),
                                              (uint32_t)((j >> 2) & 1) ^ 1, m, p.status)) ||
            !__all_sync(0xffffffffu, wait_bar(smem_u32(&m->acc_full[buf]),
                                              (uint32_t)((j >> 2) & 1), m, p.status))) {
          alive = false;
          break;
        }
        tc_fence_after();
        const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)buf * 128u;
        float mx = -INFINITY, z = 0.f;
        float mb[4];
#pragma unroll
        for (int blk = 0; blk < 4; ++blk) {
          float cur[32];
          tmem_ld32_issue(taddr + blk * 32, cur);
          tmem_ld_wait(cur);
          float zb;
          if (fast) {
            float t[4] = {cur[0], cur[1], cur[2], cur[3]};
#pragma unroll
            for (int i = 4; i < 32; i += 4) {
              t[0] = fmaxf(t[0], cur[i]);
              t[1] = fmaxf(t[1], cur[i + 1]);
              t[2] = fmaxf(t[2], cur[i + 2]);
              t[3] = fmaxf(t[3], cur[i + 3]);
            }
            const float nm = fmaxf(fmaxf(t[0], t[1]), fmaxf(t[2], t[3])) * sc2;
            if (nm > mx) {
              z *= fast_exp2(mx - nm);
              mx = nm;
            }
            const float neg = -mx;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float2 r = __ffma2_rn(make_float2(cur[i], cur[i + 1]), make_float2(sc2, sc2),
                                          make_float2(neg, neg));
              cur[i] = fast_exp2(r.x);
              cur[i + 1] = fast_exp2(r.y);
            }
            zb = tree_sum32_keep(cur);
            // the halo columns belong to the neighbouring tiles' sums
            if (blk == 0) {
#pragma unroll
              for (int c = 0; c < kMaxRadius; ++c)
                if (c < rad) zb -= cur[c];
            }
            if (blk == 3) {
#pragma unroll
              for (int c = 0; c < kMaxRadius; ++c)
                if (c < rad) zb -= cur[31 - c];
            }
          } else {
            // edge tiles: columns before key 0, beyond what the query sees, or in the halo
            const int vlo = -i0 - blk * 32, vhi = last - i0 - blk * 32;           // visible
            const int olo = rad - blk * 32, ohi = rad + p.ok - blk * 32;         // owned
            float bm = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (i >= vlo && i < vhi) bm = fmaxf(bm, cur[i]);
            const float nm = bm * sc2;
            if (nm > mx) {
              z *= fast_exp2(mx - nm);
              mx = nm;
            }
            zb = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              float e = 0.f;
              if (i >= vlo && i < vhi) e = fast_exp2(fmaf(cur[i], sc2, -mx));  // mx is finite here
              cur[i] = e;
              if (i >= olo && i < ohi) zb += e;
            }
          }
          z += zb;
          mb[blk] = mx;
          tmem_st32(taddr + blk * 32, cur);
          tmem_st_wait();
        }
        tc_fence_before();
        m->mtab[buf][row] = make_float4(mb[0], mb[1], mb[2], mb[3]);
        m->pub[buf][row] = z > 0.f ? mx + fast_log2(z) : -INFINITY;
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(smem_u32(&m->e_ready[buf]));
          mbar_arrive(smem_u32(&m->pub_full[buf]));
        }
      }
    }
  } else if (warp >= 8 && warp < 12) {
    // ================= score warps ==============================================================
    const int quad = warp & 3, row = quad * 32 + lane;
    const float inv_w = 1.0f / (float)W;
    const bool avg = g.pool_kind == LAVA_POOL_AVG;
    const uint32_t gbar = smem_u32(&m->bsync);
    uint32_t gphase = 0;
    bool alive = true;
    auto group_sync = [&]() {
      __syncwarp();
      if (lane == 0) mbar_arrive(gbar);
      if (!__all_sync(0xffffffffu, wait_bar(gbar, gphase & 1, m, p.status))) alive = false;
      ++gphase;
    };
    float* scr0 = reinterpret_cast<float*>(gen + kOffScr) + (size_t)quad * 2 * 32 * kScrStride;
    long long j = 0;
    float pend = 0.f;  // split groups: the first unit's score of this thread's key
    for (long long kappa = blockIdx.x; kappa < total_k && alive; kappa += gridDim.x) {
      const KJob kj = decode_job(p, m, kappa);
      const int i0 = kj.tile * p.ok - rad;
      float es = 0.f, et = 0.f;
      for (int half = 0; half < nunit && alive; ++half, ++j) {
        const int buf = (int)(j & (kAcc - 1));
        const int heads = nunit == 1 ? g.group : (half ? g.group - p.g0 : p.g0);
        if (!__all_sync(0xffffffffu, wait_bar(smem_u32(&m->prep_full[buf]),
                                              (uint32_t)((j >> 2) & 1), m, p.status)) ||
            !__all_sync(0xffffffffu, wait_bar(smem_u32(&m->e_ready[buf]),
                                              (uint32_t)((j >> 2) & 1), m, p.status))) {
          alive = false;
          break;
        }
        tc_fence_after();
        const float lse = m->lse_tab[buf][row];
        const float4 mb4 = m->mtab[buf][row];
        const float scale = m->scale[buf];
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&m->prep_empty[buf]));
        // e was taken relative to the running maximum of its block: exp2(max - lse) / w turns it
        // into this query's share of the window mean
        float rf[4];
        {
          const bool live = row < heads * W && lse > -INFINITY;
          rf[0] = live ? fast_exp2(mb4.x - lse) * inv_w : 0.f;
          rf[1] = live ? fast_exp2(mb4.y - lse) * inv_w : 0.f;
          rf[2] = live ? fast_exp2(mb4.z - lse) * inv_w : 0.f;
          rf[3] = live ? fast_exp2(mb4.w - lse) * inv_w : 0.f;
        }
        const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)buf * 128u;
#pragma unroll
        for (int blk = 0; blk < 4; ++blk) {
          float cur[32];
          tmem_ld32_issue(taddr + blk * 32, cur);
          tmem_ld_wait(cur);
          const float f = rf[blk];
          float* scr = scr0 + (blk & 1) * 32 * kScrStride;
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float2 a = __fmul2_rn(make_float2(cur[i], cur[i + 1]), make_float2(f, f));
            const float2 b = __fmul2_rn(make_float2(cur[i + 2], cur[i + 3]), make_float2(f, f));
            *reinterpret_cast<float4*>(scr + lane * kScrStride + i) = make_float4(a.x, a.y, b.x, b.y);
          }
          __syncwarp();
          // lane <-> key column: the sum over the warp's 32 rows, in row order (four chains)
          const float* col = scr + lane;
          if (W == 16) {
            float s0[2] = {0.f, 0.f}, s1[2] = {0.f, 0.f};
#pragma unroll
            for (int t = 0; t < 16; t += 2) {
              s0[0] += col[t * kScrStride];
              s0[1] += col[(t + 1) * kScrStride];
              s1[0] += col[(t + 16) * kScrStride];
              s1[1] += col[(t + 17) * kScrStride];
            }
            m->pbuf[quad][0][blk * 32 + lane] = s0[0] + s0[1];
            m->pbuf[quad][1][blk * 32 + lane] = s1[0] + s1[1];
          } else {
            float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int t = 0; t < 32; t += 4) {
              s[0] += col[t * kScrStride];
              s[1] += col[(t + 1) * kScrStride];
              s[2] += col[(t + 2) * kScrStride];
              s[3] += col[(t + 3) * kScrStride];
            }
            m->pbuf[quad][0][blk * 32 + lane] = (s[0] + s[1]) + (s[2] + s[3]);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&m->acc_empty[buf]));
        group_sync();  // every warp's row sums are in place
        if (!alive) break;
        // thread <-> key column `row` of the tile
        const int i = i0 + row;
        const bool inside = i >= 0 && i < kj.s.prefix;
        {
          float a[8];
#pragma unroll
          for (int h = 0; h < 8; ++h) {
            float v = 0.f;
            if (h < heads) {
              if (W == 16) v = m->pbuf[h >> 1][h & 1][row];
              else if (W == 32) v = m->pbuf[h & 3][0][row];
              else if (W == 64) v = m->pbuf[(2 * h) & 3][0][row] + m->pbuf[(2 * h + 1) & 3][0][row];
              else v = (m->pbuf[0][0][row] + m->pbuf[1][0][row]) + (m->pbuf[2][0][row] + m->pbuf[3][0][row]);
            }
            a[h] = v;
          }
          if (avg) {
#pragma unroll
            for (int h = 0; h < 4; ++h)
              if (h < heads) m->abuf[h][row] = inside ? a[h] : 0.f;
          } else {
            // max-pooling commutes with the group maximum: reduce over the query heads first
            float top = 0.f;
#pragma unroll
            for (int h = 0; h < 8; ++h) top = fmaxf(top, a[h]);
            m->abuf[0][row] = inside ? top : 0.f;
          }
        }
        group_sync();
        if (!alive) break;
        if (row >= rad && row < rad + p.ok && i < kj.s.prefix) {
          float best = 0.f;
          if (avg) {
            for (int h = 0; h < heads; ++h) {
              const float* av = &m->abuf[h][row];
              float pv = 0.f;
              for (int q = -rad; q <= rad; ++q) pv += av[q];
              best = fmaxf(best, pv / (float)g.pool_kernel);
            }
          } else {
            const float* av = &m->abuf[0][row];
            best = av[0];
            for (int q = 1; q <= rad; ++q) best = fmaxf(best, fmaxf(av[-q], av[q]));
          }
          float sc = best * scale;
          if (nunit == 2 && half == 0) {
            pend = sc;
          } else {
            if (nunit == 2) sc = fmaxf(sc, pend);
            p.scores[(size_t)kj.layer * g.total_scores + kj.s.score_off +
                     (long long)kj.kvh * kj.s.prefix + i] = sc;
            if (sc > 0.f) {
              es += sc;
              et += sc * __logf(sc);
            }
          }
        }
      }
      if (!alive) break;
      // entropy sums of the tile in a fixed order: lanes of a warp here, warps and tiles in the
      // finishing kernel
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        es += __shfl_down_sync(0xffffffffu, es, o);
        et += __shfl_down_sync(0xffffffffu, et, o);
      }
      if (lane == 0) p.ent_part[(size_t)kappa * 4 + quad] = make_float2(es, et);
    }
  } else if (warp >= 12) {
    // ================= value-norm warps: the V rows of the CTA's tiles ========================
    // Row L1 norms through the register-operand tensor path: a warp takes 16 rows, clears the
    // sign bits of the packed bf16 values and multiplies the 16 x 128 slab by a matrix of ones
    // (mma.sync m16n8k16, fp32 accumulate, exact products), which leaves the row sums in the
    // accumulator.  Thread (gq = lane / 4, tq = lane % 4) loads pieces tq, tq+4, tq+8, tq+12 of
    // rows gq and gq+8.  Eight warps cover the at most 128 rows a tile owns; the next tile's
    // loads are in flight while this one is reduced.
    if (!p.vbar_in) {
      const int vw = warp - 12, gq = lane >> 2, tq = lane & 3;
      struct Slab {
        const char* base;
        int row0, row_hi, rhead;
      };
      long long kappa = blockIdx.x;
      auto next_slab = [&](Slab& sl) -> bool {
        if (kappa >= total_k || m->abort_flag) return false;
        const KJob kj = decode_job(p, m, kappa);
        kappa += gridDim.x;
        sl.base = p.v + ((size_t)kj.layer * p.v_ls + (long long)kj.kvh * g.v_sh +
                         kj.s.tok0 * g.v_st) * 2 + tq * 16;
        sl.row0 = kj.tile * p.ok + vw * 16 + gq;
        sl.row_hi = min(kj.s.n, (kj.tile + 1) * p.ok);
        sl.rhead = (kj.layer * g.batch + kj.b) * g.n_kv_heads + kj.kvh;
        return true;
      };
      auto issue = [&](uint4 (&buf)[8], const Slab& sl) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const int r = sl.row0 + hh * 8;
          const char* src = sl.base + (long long)r * g.v_st * 2;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            buf[hh * 4 + q] = make_uint4(0, 0, 0, 0);
            if (r < sl.row_hi) buf[hh * 4 + q] = ld_stream16(src + q * 64);
          }
        }
      };
      const uint32_t ones = 0x3f803f80u;  // bf16 (1, 1)
      auto reduce = [&](const uint4 (&buf)[8], const Slab& sl) {
        float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;  // d0: row gq, d2: row gq + 8
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint4 lo = buf[q], hi = buf[4 + q];
          mma_bf16_16816(d0, d1, d2, d3, lo.x & 0x7fff7fffu, hi.x & 0x7fff7fffu,
                         lo.y & 0x7fff7fffu, hi.y & 0x7fff7fffu, ones, ones);
          mma_bf16_16816(d0, d1, d2, d3, lo.z & 0x7fff7fffu, hi.z & 0x7fff7fffu,
                         lo.w & 0x7fff7fffu, hi.w & 0x7fff7fffu, ones, ones);
        }
        float best = fmaxf(d0, d2);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
        if (lane == 0) {
          atomicMax(&p.vbar_bits[sl.rhead], __float_as_uint(best));
          __threadfence();
          atomicAdd(&p.vcount[sl.rhead], 1);
        }
      };
      uint4 bufa[8], bufb[8];
      Slab sa, sb;
      bool have_a = next_slab(sa), have_b = false;
      if (have_a) issue(bufa, sa);
      while (have_a) {
        have_b = next_slab(sb);
        if (have_b) issue(bufb, sb);
        reduce(bufa, sa);
        if (!have_b) break;
        have_a = next_slab(sa);
        if (have_a) issue(bufa, sa);
        reduce(bufb, sb);
      }
    }
  }

  // ---- teardown: everything this CTA started has finished before shared memory and TMEM go --
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

// entropy of one (layer, sequence) from the per-tile sums, folded in a fixed order; also hands
// out the value norms
__global__ void __launch_bounds__(256)
entropy_finalize_tmem_kernel(Geom g, int ok, const float2* ent_part, double* entropy,
                             const float* vbar_in, const unsigned* vbar_bits, float* vbar_out) {
  __shared__ double rs[8], rt[8];
  const int prob = blockIdx.x, layer = prob / g.batch, b = prob - layer * g.batch;
  const SeqInfo s = seq_info(g, b);
  if (vbar_out && (int)threadIdx.x < g.n_kv_heads) {
    const size_t head = (size_t)prob * g.n_kv_heads + threadIdx.x;
    vbar_out[head] = vbar_in ? vbar_in[head] : __uint_as_float(vbar_bits[head]);
  }
  long long before = 0, all = 0;  // tiles of the sequences before this one / of a whole layer
  for (int bb = 0; bb < g.batch; ++bb) {
    const int t = ceil_div(seq_info(g, bb).n, ok);
    if (bb < b) before += t;
    all += t;
  }
  const long long first = ((long long)layer * all + before) * g.n_kv_heads * 4;
  const long long count = (long long)ceil_div(s.n, ok) * g.n_kv_heads * 4;
  double sum_s = 0.0, sum_t = 0.0;
  for (long long i = threadIdx.x; i < count; i += 256) {
    const float2 e = ent_part[first + i];
    sum_s += (double)e.x;
    sum_t += (double)e.y;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    sum_s += __shfl_down_sync(0xffffffffu, sum_s, o);
    sum_t += __shfl_down_sync(0xffffffffu, sum_t, o);
  }
  if ((threadIdx.x & 31) == 0) {
    rs[threadIdx.x >> 5] = sum_s;
    rt[threadIdx.x >> 5] = sum_t;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0, c = 0.0;
    for (int i = 0; i < 8; ++i) {
      a += rs[i];
      c += rt[i];
    }
    double e = 0.0;
    if (a > 0.0) e = (log(a) - c / a) / ((double)g.n_kv_heads * (double)s.n);
    entropy[(size_t)layer * g.batch + b] = e;
  }
}

size_t up256(size_t x) { return (x + 255) / 256 * 256; }

int first_unit_heads(const Geom& g) { return g.group * g.window > 128 ? (g.group + 1) / 2 : 0; }

}  // namespace

// Geometry the single-pass kernel covers, whatever the grid: the tensor-core path's geometry,
// a pooling radius of at most 4, and a head short enough for a part with up to 160 SMs.  Whether
// a launch really fits is decided against the actual grid in tmem_fits.
bool tmem_supported(const Geom& g) {
  if (!sm100_supported(g)) return false;
  if (g.pool_radius > kMaxRadius) return false;
  const int nunit = first_unit_heads(g) ? 2 : 1;
  const int tmax = ceil_div(g.max_seqlen, kTile - 2 * g.pool_radius);
  return tmax <= (nunit == 1 ? 3 * 160 + 1 : 160 + 1);
}

TmemLayout tmem_layout(const Geom& g, int n_layers) {
  TmemLayout l;
  l.ok = kTile - 2 * g.pool_radius;
  l.nunit = first_unit_heads(g) ? 2 : 1;
  l.tmax = ceil_div(g.max_seqlen, l.ok);
  l.gmax = ceil_div(l.tmax, kFold);
  // tiles of a layer: sum over sequences of ceil(n / ok) <= total / ok + batch
  const long long tiles_cap = (g.total_tokens / l.ok + g.batch) * g.n_kv_heads;
  l.kjobs_cap = (long long)n_layers * tiles_cap;
  l.heads_total = n_layers * g.batch * g.n_kv_heads;
  l.units_total = l.heads_total * l.nunit;
  size_t off = 0;
  l.off_sync = off;  // gcount, hcount, flag, vcount, vbar_bits: zeroed every launch
  off = up256(off + sizeof(int) * ((size_t)l.units_total * (l.gmax + 2) + 2 * (size_t)l.heads_total));
  l.sync_bytes = off;
  l.off_part = off;
  off = up256(off + sizeof(float) * 128 * (size_t)l.kjobs_cap * l.nunit);
  l.off_gpart = off;
  off = up256(off + sizeof(float) * 128 * (size_t)l.units_total * l.gmax);
  l.off_head = off;
  off = up256(off + sizeof(float) * 128 * (size_t)l.units_total);
  l.off_ent = off;
  off = up256(off + sizeof(float2) * 4 * (size_t)l.kjobs_cap);
  l.total = off;
  return l;
}

// Does a launch on `grid` CTAs keep every head inside the rounds the accumulator buffers span?
bool tmem_fits(const Geom& g, int grid) {
  const int nunit = first_unit_heads(g) ? 2 : 1;
  const int tmax = ceil_div(g.max_seqlen, kTile - 2 * g.pool_radius);
  return tmax <= (nunit == 1 ? 3 * grid + 1 : grid + 1);
}

int tmem_grid(const Geom& g, int n_layers) {
  const int sms = sm_count();
  const long long cap = tmem_layout(g, n_layers).kjobs_cap;
  return (int)(cap < sms ? cap : sms);
}

lava_status launch_score_tmem(const Geom& g, int n_layers, const void* q, const void* k,
                              const void* v, long long q_ls, long long k_ls, long long v_ls,
                              const float* vbar_in, float* scores, float* vbar_out,
                              double* entropy, char* ws_base, size_t ws_off, cudaStream_t stream) {
  char* ws = ws_base + ws_off;
  CUtensorMap map_q, map_k;
  lava_status rc = encode_score_maps(g, n_layers, q, k, q_ls, k_ls, &map_q, &map_k);
  if (rc != LAVA_OK) return rc;
  const TmemLayout lay = tmem_layout(g, n_layers);
  const int grid = tmem_grid(g, n_layers);
  if (grid <= 0) return fail(LAVA_ERR_CUDA, "the multiprocessor count of the device is not available");
  if (lay.kjobs_cap * lay.nunit > 0x3fffffffLL)
    return fail(LAVA_ERR_UNSUPPORTED, "too many tiles for the 32-bit job index");

  TmemParams p;
  p.g = g;
  p.n_layers = n_layers;
  p.ok = lay.ok;
  p.nunit = lay.nunit;
  p.g0 = first_unit_heads(g);
  p.gmax = lay.gmax;
  p.wait_cycles = options().wait_limit_cycles;
  p.vbar_in = vbar_in;
  p.scores = scores;
  p.v = (const char*)v;
  p.v_ls = v_ls;
  int* sync = reinterpret_cast<int*>(ws + lay.off_sync);
  p.gcount = sync;
  p.hcount = p.gcount + (size_t)lay.units_total * lay.gmax;
  p.flag = p.hcount + lay.units_total;
  p.vcount = p.flag + lay.units_total;
  p.vbar_bits = reinterpret_cast<unsigned*>(p.vcount + lay.heads_total);
  p.part = reinterpret_cast<float*>(ws + lay.off_part);
  p.gpart = reinterpret_cast<float*>(ws + lay.off_gpart);
  p.head_lse = reinterpret_cast<float*>(ws + lay.off_head);
  p.ent_part = reinterpret_cast<float2*>(ws + lay.off_ent);
  p.status = reinterpret_cast<unsigned*>(ws_base);

  rc = check_cuda(cudaMemsetAsync(ws + lay.off_sync, 0, lay.sync_bytes, stream), "sync scratch clear");
  if (rc != LAVA_OK) return rc;
  rc = check_cuda(cudaFuncSetAttribute(lava_score_tmem_kernel,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes),
                  "cudaFuncSetAttribute(single-pass score)");
  if (rc != LAVA_OK) return rc;
  void* args[3] = {&map_q, &map_k, &p};
  rc = check_cuda(cudaLaunchCooperativeKernel((const void*)lava_score_tmem_kernel, dim3(grid),
                                              dim3(kThreads), args, kSmemBytes, stream),
                  "score (single-pass) launch");
  if (rc != LAVA_OK) return rc;
  entropy_finalize_tmem_kernel<<<n_layers * g.batch, 256, 0, stream>>>(
      g, lay.ok, p.ent_part, entropy, vbar_in, p.vbar_bits, vbar_out);
  count_launches(2);
  return check_cuda(cudaGetLastError(), "entropy finalize launch");
}

}  // namespace lava
