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
// One persistent CTA per SM (cooperative launch: the CTAs wait on one another's counters).  A
// job is one 128-key tile of one unit (a KV head, or one half of its query group when the group
// has more than 128 window-query rows); tiles overlap by twice the pooling radius so that every
// owned key finds its pooling neighbours inside its own tile.  Jobs are dealt round-robin.
// Tensor memory holds one fp32 accumulator tile (released as soon as its last block of logits is
// in registers, so the next job's MMA overlaps the rest of the work) and six buffers of exponentials.  The
// exponentials are kept as fp16 pairs, scaled so that the largest of a 32-key block is 2^15:
// every stored term carries a relative rounding error of at most 2^-12, small terms are denormal
// with an absolute error below 2^-40 of the block's largest; the normalisers and every sum are
// fp32.  Six buffers instead of the three that fp32 storage would allow are what hides the
// exchange of the row statistics between the CTAs.
//
//   producer warp     TMA: the K tile (once per K tile, shared by the two units of a split
//                     group) and the unit's query tile, into 128B-swizzled shared memory
//   MMA warp          S = Q_u K^T (rows = window queries, columns = keys) into tensor memory
//   8 statistics      one thread per window-query row and half of the tile's columns: running
//     warps           maximum per 32-column block, e = exp2(z - max + 15) packed to fp16 into an
//                     exponent buffer, the row's fp32 sum over the keys the tile owns; the
//                     tile's log2-sum-exp per row goes to the publisher
//   publisher warp    writes the tile's row statistics to global memory and counts them; the
//                     CTA that delivers the last tile of a group folds the group and counts it
//                     on the head
//   prep warp         waits until every group of the next job's head is in (and its value norm),
//                     folds the groups, in order, into the head's log2-sum-exp per row (every
//                     CTA does this for itself, with the same operations: same bits everywhere)
//   4 score warps     the window mean of Definition 1 on the register-operand tensor path: a
//                     warp's 32 rows of packed exponentials go through shared memory and come
//                     back transposed (ldmatrix) as the A operand of mma.sync m16n8k16; the B
//                     operand carries exp2(block max - lse) / w of every row as an fp16 pair
//                     (high and low part), so the fp32 accumulator holds the head's window mean
//                     of 16 keys.  Then pooling (Sec. 5.1), Vbar * c_hat, the group maximum
//                     (Sec. 4.3), one store per key; entropy sums of Sec. 4.2 per CTA
//   4 value warps     stream the V rows of the CTA's tiles for max_k ||V[k]||_1 (Theorem 1)
//
// A head's tiles lie in at most four consecutive rounds of jobs (two when units are split), and
// the statistics warps run at most five jobs ahead of the score warps, so every wait for a
// head's statistics ends (the launcher checks the bound).  Every wait is bounded in time all the
// same.
#include <cuda_fp16.h>

#include "sm100_ptx.cuh"

namespace lava {
namespace {

using namespace sm100;

constexpr int kTile = 128;
constexpr int kThreads = 640;        // 20 warps: 4 service, 8 statistics, 4 score, 4 value
constexpr int kStatWarp0 = 4, kScoreWarp0 = 12, kValueWarp0 = 16;
constexpr int kVWarps = 4;           // two 16-row slabs of V per tile and value warp
constexpr int kEB = 6;               // buffers of exponentials (64 TMEM columns of fp16 pairs each)
constexpr int kKStages = 3;
constexpr int kMaxBatch = 512;
constexpr int kMaxRadius = 4;
constexpr int kMaxCtas = 192;        // CTAs the per-CTA entropy slots are sized for
constexpr float kExpBias = 15.0f;    // stored exponentials are scaled by 2^15 (fp16 tops out at 2^16)
constexpr float kRowBias = 34.0f;    // the per-row factors exp2(ref - lse) / w are scaled by 2^34
                                     // so that they are normal fp16 numbers down to 2^-48
constexpr uint32_t kTileBytes = 128 * 128 * 2;
constexpr uint32_t kHalfBytes = kTileBytes / 2;
constexpr uint32_t kAccCols = 128;   // TMEM: columns 0..127 accumulator, then the exponent buffers
constexpr uint32_t kScrRow = 80;     // bytes per row of a score warp's scratch (64 used: no bank conflicts)
constexpr uint32_t kScrTile = 32 * kScrRow;

constexpr uint32_t kOffQ = 0;                                   // 2 query tiles
constexpr uint32_t kOffK = kOffQ + 2 * kTileBytes;              // 3 key tiles
constexpr uint32_t kOffScr = kOffK + kKStages * kTileBytes;     // 4 warps x 2 x 32 rows x 80 B
constexpr uint32_t kScrBytes = 4 * 2 * kScrTile;
constexpr uint32_t kOffCtl = kOffScr + kScrBytes;

struct Ctl {
  unsigned long long k_full[kKStages], k_empty[kKStages], q_full[2], q_empty[2];
  unsigned long long acc_full, acc_empty;           // the accumulator tile
  unsigned long long e_ready[kEB], e_empty[kEB];    // exponent buffers
  unsigned long long pub_full[kEB], pub_empty[kEB], prep_full[kEB], prep_empty[kEB];
  unsigned long long bsync, drain;
  uint32_t tmem_base;
  volatile int abort_flag;
  long long wait_cycles;
  int tiles_layer;                    // K tiles of one layer: H_kv * sum over sequences
  float scale[kEB];                   // Vbar * c_hat of the job's head
  alignas(16) float pub[kEB][2][128]; // log2-sum-exp per row of a finished tile, per column half
  alignas(16) float lse_tab[kEB][128];   // the head's log2-sum-exp per row
  alignas(16) float4 mtab[kEB][128];  // the four block references of every row of a tile
  alignas(16) float pbuf[2][4][2][kTile];  // [job parity][score warp][half warp when w = 16][key]
  alignas(16) uint32_t ftab[4][2][2][16];  // [score warp][block parity][high, low][row pair] fp16 pairs
  int pref[kMaxBatch + 1];            // exclusive scan of tiles per sequence
};
constexpr uint32_t kSmemBytes = kOffCtl + sizeof(Ctl) + 1024;
static_assert(kSmemBytes <= 232448 - 256, "shared memory budget");

struct TmemParams {
  Geom g;
  int n_layers;
  int ok;                   // keys a tile owns: 128 - 2 * pool_radius
  int nunit;                // units per KV head: 1, or 2 when the query group is split
  int g0;                   // query heads in the first unit (split mode)
  int kfold;                // tiles per first-level fold group
  int gmax;                 // first-level fold groups per unit at max_seqlen (at most 16)
  int tmax;                 // tiles per unit at max_seqlen
  long long wait_cycles;
  const float* vbar_in;
  float* scores;
  const char* v;
  long long v_ls;
  // scratch
  float* part;              // [jobs][128] log2-sum-exp per tile and row
  float* gpart;             // [units][gmax][128] per group of kfold tiles
  int* gcount;              // [units][gmax] tiles published per group
  int* hcount;              // [units] groups folded per unit
  int* vcount;              // [KV heads] finished value-norm slabs
  unsigned* vbar_bits;      // [KV heads]
  float2* ent_part;         // [layer * batch][kMaxCtas][4] (sum s, sum s ln s) per CTA and score warp
  unsigned* status;
};

struct KJob {
  int layer, b, kvh, tile, ntiles;
  bool idle;   // a padding slot: no tile (heads longer than a round are padded to whole rounds)
  SeqInfo s;
};

// Slot kappa of the launch -> the K tile it holds.  Slots are dealt round-robin to the CTAs.  A
// sequence whose heads have more tiles than there are CTAs gets each head padded to whole rounds
// (pad > 0: slots per head), so that every CTA works on the same head at the same time and the
// head's statistics are complete one round after its first tile; shorter heads are packed.
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
  const int slots = m->pref[lo + 1] - m->pref[lo];  // slots per head of this sequence
  const int r2 = r - p.g.n_kv_heads * m->pref[lo];
  kj.kvh = r2 / slots;
  kj.tile = r2 - kj.kvh * slots;
  kj.s = seq_info(p.g, lo);
  kj.ntiles = ceil_div(kj.s.n, p.ok);
  kj.idle = kj.tile >= kj.ntiles;
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

__device__ inline uint32_t pack_half2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

template <int W>
__global__ void __launch_bounds__(kThreads, 1)
lava_score_tmem_kernel(const __grid_constant__ CUtensorMap map_q,
                       const __grid_constant__ CUtensorMap map_k, const TmemParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  Ctl* m = reinterpret_cast<Ctl*>(gen + kOffCtl);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const Geom& g = p.g;
  const int rad = g.pool_radius, nunit = p.nunit;
  if (batch_has_short_sequence(g)) {  // every CTA sees the same lengths: all of them leave
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(p.status, LAVA_DEV_SHORT_SEQUENCE);
    return;
  }

  // ---- tiles per sequence (exclusive scan), barriers, tensor memory ---------------------------
  __shared__ int bad_len;
  {
    __shared__ int wsum[kThreads / 32];
    if (threadIdx.x == 0) bad_len = 0;
    __syncthreads();
    int c = 0;
    if ((int)threadIdx.x < g.batch) {
      const SeqInfo s = seq_info(g, threadIdx.x);
      if (s.n < g.window && blockIdx.x == 0) atomicOr(p.status, LAVA_DEV_SHORT_SEQUENCE);
      c = ceil_div(s.n, p.ok);
      if (c > p.tmax) {  // longer than the caller's max_seqlen: the scratch is not sized for it
        atomicOr(p.status, LAVA_DEV_BAD_SEQLEN);
        bad_len = 1;
        c = 0;
      }
      if (c > (int)gridDim.x) c = ceil_div(c, (int)gridDim.x) * (int)gridDim.x;  // whole rounds
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
    mbar_init(smem_u32(&m->acc_full), 1);
    mbar_init(smem_u32(&m->acc_empty), 8);        // one arrival per statistics warp
    for (int s = 0; s < kEB; ++s) {
      mbar_init(smem_u32(&m->e_ready[s]), 8);     // one arrival per statistics warp
      mbar_init(smem_u32(&m->e_empty[s]), 4);     // one arrival per score warp
      mbar_init(smem_u32(&m->pub_full[s]), 8);
      mbar_init(smem_u32(&m->pub_empty[s]), 1);
      mbar_init(smem_u32(&m->prep_full[s]), 1);
      mbar_init(smem_u32(&m->prep_empty[s]), 4);
    }
    mbar_init(smem_u32(&m->bsync), 4);
    mbar_init(smem_u32(&m->drain), 1);
    m->abort_flag = bad_len;  // nothing runs on a batch the scratch was not sized for
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
        if (kj.idle) continue;
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
      for (long long kappa = blockIdx.x; kappa < total_k && ok; kappa += gridDim.x) {
        if (decode_job(p, m, kappa).idle) continue;
        const int st = (int)(nk % kKStages);
        ok = wait_bar(smem_u32(&m->k_full[st]), (uint32_t)((nk / kKStages) & 1), m, p.status);
        for (int half = 0; half < nunit && ok; ++half, ++j) {
          const int qs = (int)(j & 1);
          ok = wait_bar(smem_u32(&m->q_full[qs]), (uint32_t)((j >> 1) & 1), m, p.status);
          // the statistics warps have read the previous job's logits out of the accumulator
          ok = ok && wait_bar(smem_u32(&m->acc_empty), (uint32_t)(j & 1) ^ 1, m, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t qa = base + kOffQ + qs * kTileBytes, ka = base + kOffK + st * kTileBytes;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (uint32_t)(kk >> 2) * kHalfBytes + (uint32_t)(kk & 3) * 32u;
            umma_bf16(tmem, make_desc(qa + off), make_desc(ka + off), kIdesc, kk > 0);
          }
          umma_commit(smem_u32(&m->acc_full));
          umma_commit(smem_u32(&m->q_empty[qs]));
        }
        if (ok) umma_commit(smem_u32(&m->k_empty[st]));
        ++nk;
      }
      // every MMA this thread issued has completed before TMEM is released
      umma_commit(smem_u32(&m->drain));
      wait_bar(smem_u32(&m->drain), 0, m, p.status, false);
    }
  } else if (warp == 2) {
    // ================= publisher: tile statistics leave the CTA; first-level folds =============
    // Publishing never waits for memory: the tile's row goes out with a release-add on its
    // group's counter.  Each group is folded by the CTA that owns one fixed tile of it (which one
    // rotates with the head, so the work spreads over the CTAs); that CTA keeps the group in a
    // short list and looks at its counter between its own jobs, so a group that is still
    // filling never holds up a publication.
    struct Pending {
      int unit, gi, gsz;
      long long row0;  // index of the group's first row in `part`
    };
    constexpr int kPend = 4;
    Pending pend[kPend];
    int npend = 0;
    bool alive = true;
    // folds every listed group that is complete (all of them, waiting, when `drain` is set)
    auto service = [&](bool drain) {
      for (int k = 0; k < npend && alive;) {
        int* gc = &p.gcount[(size_t)pend[k].unit * p.gmax + pend[k].gi];
        int ready = 0;
        if (lane == 0) {
          ready = ld_relaxed(gc) >= pend[k].gsz;
          if (!ready && drain) {
            const long long t0 = clock64();
            while (ld_relaxed(gc) < pend[k].gsz) {
              if (m->abort_flag) break;
              __nanosleep(32);
              if (clock64() - t0 > m->wait_cycles) {
                give_up(m, p.status);
                break;
              }
            }
            ready = ld_relaxed(gc) >= pend[k].gsz;
          }
        }
        ready = __shfl_sync(0xffffffffu, ready, 0);
        if (!ready) {
          if (drain) alive = false;
          ++k;
          continue;
        }
        __threadfence();  // the counter was read before the rows it announces
        const float4* rows = reinterpret_cast<const float4*>(p.part + (size_t)pend[k].row0 * 128) + lane;
        const float4 gl = fold_rows(rows, (size_t)32 * nunit, pend[k].gsz);
        reinterpret_cast<float4*>(p.gpart + ((size_t)pend[k].unit * p.gmax + pend[k].gi) * 128)[lane] = gl;
        __syncwarp();
        if (lane == 0) red_add_release(&p.hcount[pend[k].unit], 1);
        pend[k] = pend[npend - 1];
        --npend;
      }
    };
    long long j = 0;
    for (long long kappa = blockIdx.x; kappa < total_k && alive; kappa += gridDim.x) {
      const KJob kj = decode_job(p, m, kappa);
      if (kj.idle) continue;
      for (int half = 0; half < nunit && alive; ++half, ++j) {
        const int eb = (int)(j % kEB);
        // wait for the statistics warps; meanwhile look after the listed groups
        {
          const uint32_t bar = smem_u32(&m->pub_full[eb]), parity = (uint32_t)((j / kEB) & 1);
          const long long t0 = clock64();
          for (;;) {
            int got = 0;
            if (lane == 0) got = mbar_try(bar, parity, 200) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (got) break;
            int stop = 0;
            if (lane == 0) {
              if (m->abort_flag) {
                stop = 1;
              } else if (clock64() - t0 > m->wait_cycles) {
                give_up(m, p.status);
                stop = 1;
              }
            }
            if (__shfl_sync(0xffffffffu, stop, 0)) {
              alive = false;
              break;
            }
            service(false);
          }
          if (!alive) break;
        }
        // lane l carries rows 4l .. 4l+3; the two column halves of the tile are merged first
        const float4 a4 = reinterpret_cast<const float4*>(m->pub[eb][0])[lane];
        const float4 b4 = reinterpret_cast<const float4*>(m->pub[eb][1])[lane];
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&m->pub_empty[eb]));
        float4 mine;
        mine.x = lse2(a4.x, b4.x);
        mine.y = lse2(a4.y, b4.y);
        mine.z = lse2(a4.z, b4.z);
        mine.w = lse2(a4.w, b4.w);
        const long long job = kappa * nunit + half;               // index of this job's row
        const long long job0 = (kappa - kj.tile) * nunit + half;  // tile 0 of the unit
        reinterpret_cast<float4*>(p.part + (size_t)job * 128)[lane] = mine;
        __syncwarp();
        const int unit = ((kj.layer * g.batch + kj.b) * g.n_kv_heads + kj.kvh) * nunit + half;
        const int gi = kj.tile / p.kfold;
        const int gsz = min(p.kfold, kj.ntiles - gi * p.kfold);
        if (lane == 0) red_add_release(&p.gcount[(size_t)unit * p.gmax + gi], 1);
        // the owner of tile (unit mod group size) of a group folds it
        if (kj.tile - gi * p.kfold == unit % gsz) {
          if (npend == kPend) service(true);  // never more than a few: make room
          if (!alive) break;
          pend[npend].unit = unit;
          pend[npend].gi = gi;
          pend[npend].gsz = gsz;
          pend[npend].row0 = job0 + (long long)gi * p.kfold * nunit;
          ++npend;
        }
        service(false);
      }
    }
    if (alive) service(true);
  } else if (warp == 3) {
    // ================= prep: the head's normalisers and value norm for the score warps =========
    // One round trip to global memory serves several jobs: lanes 0..15 look at the CTA's next
    // sixteen slots and read the counters of their heads (groups folded, value-norm slabs done);
    // the slots that are complete, in order, are then prepared.  A head's fold is kept for the
    // CTA's next tile of that head.
    const long long nslots = blockIdx.x < total_k ? (total_k - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    long long icur = 0, j = 0;  // next slot of this CTA to look at; jobs prepared so far
    bool alive = true;
    int have_unit = -1;
    float4 have = make_float4(0.f, 0.f, 0.f, 0.f);
    float have_scale = 0.f;
    long long t_idle = clock64();
    while (alive && icur < nslots) {
      const long long islot = icur + lane;
      const bool mine = lane < 16 && islot < nslots;
      int rhead = -1, ngroups = 0;
      bool idle = true, done = true;
      if (mine) {
        const KJob kj = decode_job(p, m, blockIdx.x + islot * gridDim.x);
        idle = kj.idle;
        if (!idle) {
          rhead = (kj.layer * g.batch + kj.b) * g.n_kv_heads + kj.kvh;
          ngroups = ceil_div(kj.ntiles, p.kfold);
          const int c0 = ld_relaxed(&p.hcount[rhead * nunit]);
          const int c1 = nunit == 2 ? ld_relaxed(&p.hcount[rhead * nunit + 1]) : ngroups;
          const int cv = p.vbar_in ? 0 : ld_relaxed(&p.vcount[rhead]);
          done = c0 >= ngroups && c1 >= ngroups &&
                 (p.vbar_in || cv >= kVWarps * min(kj.ntiles, (int)gridDim.x));
        }
      }
      const unsigned okmask = __ballot_sync(0xffffffffu, done);
      const int nready = okmask == 0xffffffffu ? 32 : __ffs(~okmask) - 1;  // slots complete in a row
      if (nready <= 0) {
        int stop = 0;
        if (lane == 0) {
          if (m->abort_flag) {
            stop = 1;
          } else if (clock64() - t_idle > m->wait_cycles) {
            give_up(m, p.status);
            stop = 1;
          }
        }
        if (__shfl_sync(0xffffffffu, stop, 0)) break;
        __nanosleep(32);
        continue;
      }
      __threadfence();  // the counters were read before the data they announce
      const int take = (int)min((long long)min(nready, 16), nslots - icur);
      for (int l = 0; l < take && alive; ++l) {
        const int rhead_l = __shfl_sync(0xffffffffu, rhead, l);
        const int ngroups_l = __shfl_sync(0xffffffffu, ngroups, l);
        if (__shfl_sync(0xffffffffu, idle ? 1 : 0, l)) continue;
        for (int half = 0; half < nunit && alive; ++half, ++j) {
          const int unit_l = rhead_l * nunit + half;
          const int eb = (int)(j % kEB);
          bool ok = true;
          if (lane == 0)
            ok = wait_bar(smem_u32(&m->prep_empty[eb]), (uint32_t)((j / kEB) & 1) ^ 1, m, p.status);
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (!ok) {
            alive = false;
            break;
          }
          if (unit_l != have_unit) {
            float vb = 0.f;
            if (lane == 0)
              vb = p.vbar_in ? p.vbar_in[rhead_l] : __uint_as_float(__ldcg(p.vbar_bits + rhead_l));
            // every CTA folds the head's groups itself, in group order: same bits everywhere
            have = fold_rows(reinterpret_cast<const float4*>(p.gpart + (size_t)unit_l * p.gmax * 128) + lane,
                             32, ngroups_l);
            have_scale = vb * g.c_hat;
            have_unit = unit_l;
          }
          reinterpret_cast<float4*>(m->lse_tab[eb])[lane] = have;
          if (lane == 0) m->scale[eb] = have_scale;
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&m->prep_full[eb]));
        }
      }
      icur += take;
      t_idle = clock64();
    }
  } else if (warp >= kStatWarp0 && warp < kScoreWarp0) {
    // ================= statistics warps: one thread per window-query row and column half ======
    const int quad = warp & 3, chalf = (warp - kStatWarp0) >> 2, row = quad * 32 + lane;
    const int t_in_win = row & (W - 1);
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    long long j = 0;
    bool alive = true;
    for (long long kappa = blockIdx.x; kappa < total_k && alive; kappa += gridDim.x) {
      const KJob kj = decode_job(p, m, kappa);
      if (kj.idle) continue;
      const int i0 = kj.tile * p.ok - rad;  // key of column 0
      // every column is a prefix key that all window queries see (the columns before key 0 of a
      // head's first tile are given key 0's logit: they are halo columns, outside every sum, and
      // the score warps mask them)
      const bool fast = (i0 >= 0 || kj.tile == 0) && i0 + kTile <= kj.s.prefix;
      for (int half = 0; half < nunit && alive; ++half, ++j) {
        const int eb = (int)(j % kEB);
        const int heads = nunit == 1 ? g.group : (half ? g.group - p.g0 : p.g0);
        // keys this query may see: i < n and i <= P + t (Sec. 2); rows beyond the unit see none
        const int last = row < heads * W ? min(kj.s.n, kj.s.prefix + t_in_win + 1) : 0;
        if (!__all_sync(0xffffffffu, wait_bar(smem_u32(&m->pub_empty[eb]),
                                              (uint32_t)((j / kEB) & 1) ^ 1, m, p.status)) ||
            !__all_sync(0xffffffffu, wait_bar(smem_u32(&m->e_empty[eb]),
                                              (uint32_t)((j / kEB) & 1) ^ 1, m, p.status)) ||
            !__all_sync(0xffffffffu, wait_bar(smem_u32(&m->acc_full), (uint32_t)(j & 1), m,
                                              p.status))) {
          alive = false;
          break;
        }
        tc_fence_after();
        float mx = -INFINITY, z = 0.f;  // z sums exp2(logit - mx + 15)
        float* refs = reinterpret_cast<float*>(&m->mtab[eb][row]);
#pragma unroll 1
        for (int bb = 0; bb < 2; ++bb) {
          const int blk = chalf * 2 + bb;
          float cur[32];
          tmem_ld32_issue(lane_addr + blk * 32, cur);
          tmem_ld_wait(cur);
          if (bb == 1) {  // this warp's logits are in registers: the next MMA may overwrite them
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&m->acc_empty));
          }
          float zb;
          if (fast) {
            if (blk == 0 && i0 < 0) {
#pragma unroll
              for (int c = 0; c < kMaxRadius; ++c)
                if (c < rad) cur[c] = cur[rad];
            }
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
            const float neg = kExpBias - mx;
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
            const float neg = kExpBias - mx;
            zb = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              float e = 0.f;
              if (i >= vlo && i < vhi) e = fast_exp2(fmaf(cur[i], sc2, neg));  // mx is finite here
              cur[i] = e;
              if (i >= olo && i < ohi) zb += e;
            }
          }
          z += zb;
          refs[blk] = mx - kExpBias;
          uint32_t packed[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) packed[i] = pack_half2(cur[2 * i], cur[2 * i + 1]);
          tmem_st16(lane_addr + kAccCols + (uint32_t)eb * 64u + (uint32_t)blk * 16u, packed);
          tmem_st_wait();
        }
        tc_fence_before();
        m->pub[eb][chalf][row] = z > 0.f ? (mx - kExpBias) + fast_log2(z) : -INFINITY;
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(smem_u32(&m->e_ready[eb]));
          mbar_arrive(smem_u32(&m->pub_full[eb]));
        }
      }
    }
  } else if (warp >= kScoreWarp0 && warp < kValueWarp0) {
    // ================= score warps ==============================================================
    const int quad = warp & 3, row = quad * 32 + lane;
    const int fg = lane >> 2, ft = lane & 3;  // fragment coordinates of the register-operand MMA
    const float inv_w = 1.0f / (float)W;
    const bool avg = g.pool_kind == LAVA_POOL_AVG;
    const uint32_t gbar = smem_u32(&m->bsync);
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16) + kAccCols;
    uint32_t gphase = 0;
    bool alive = true;
    auto group_sync = [&]() {
      __syncwarp();
      if (lane == 0) mbar_arrive(gbar);
      if (!__all_sync(0xffffffffu, wait_bar(gbar, gphase & 1, m, p.status))) alive = false;
      ++gphase;
    };
    uint8_t* scr0 = gen + kOffScr + (size_t)quad * 2 * kScrTile;
    const uint32_t scr0_s = base + kOffScr + (uint32_t)quad * 2 * kScrTile;
    // ldmatrix: lane l supplies row (l % 8) of matrix (l / 8); matrices 0..3 are (keys 0-7,
    // rows 0-7), (keys 8-15, rows 0-7), (keys 0-7, rows 8-15), (keys 8-15, rows 8-15)
    const uint32_t ldm_off = (uint32_t)(((lane >> 4) * 8 + (lane & 7)) * kScrRow + ((lane >> 3) & 1) * 16);
    long long j = 0;
    float pend = 0.f;    // split groups: the first unit's score of this thread's key
    float es = 0.f, et = 0.f;
    int ent_prob = -1;   // (layer, sequence) the entropy sums belong to
    auto flush_entropy = [&]() {
      // lanes of a warp in a fixed order; warps and CTAs are added up, in order, by the
      // finishing kernel
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        es += __shfl_down_sync(0xffffffffu, es, o);
        et += __shfl_down_sync(0xffffffffu, et, o);
      }
      if (lane == 0 && ent_prob >= 0)
        p.ent_part[((size_t)ent_prob * kMaxCtas + blockIdx.x) * 4 + quad] = make_float2(es, et);
      es = 0.f;
      et = 0.f;
    };
    for (long long kappa = blockIdx.x; kappa < total_k && alive; kappa += gridDim.x) {
      const KJob kj = decode_job(p, m, kappa);
      if (kj.idle) continue;
      const int i0 = kj.tile * p.ok - rad;
      const int prob = kj.layer * g.batch + kj.b;
      if (prob != ent_prob) {
        flush_entropy();
        ent_prob = prob;
      }
      float* score_row = p.scores + (size_t)kj.layer * g.total_scores + kj.s.score_off;
      for (int half = 0; half < nunit && alive; ++half, ++j) {
        const int eb = (int)(j % kEB), jp = (int)(j & 1);
        const int heads = nunit == 1 ? g.group : (half ? g.group - p.g0 : p.g0);
        if (!__all_sync(0xffffffffu, wait_bar(smem_u32(&m->prep_full[eb]),
                                              (uint32_t)((j / kEB) & 1), m, p.status)) ||
            !__all_sync(0xffffffffu, wait_bar(smem_u32(&m->e_ready[eb]),
                                              (uint32_t)((j / kEB) & 1), m, p.status))) {
          alive = false;
          break;
        }
        tc_fence_after();
        const float lse = m->lse_tab[eb][row];
        const float scale = m->scale[eb];
        const bool live = row < heads * W && lse > -INFINITY;
        const float* refs = reinterpret_cast<const float*>(&m->mtab[eb][row]);
        const uint32_t e_addr = lane_addr + (uint32_t)eb * 64u;
        uint32_t pk[16];
        tmem_ld16_issue(e_addr, pk);
#pragma unroll 1
        for (int blk = 0; blk < 4; ++blk) {
          // e was taken relative to the block's reference: exp2(ref - lse) / w turns it into this
          // query's share of the window mean; kept as a high and a low fp16 part (scaled by 2^34)
          const float f = live ? fast_exp2(refs[blk] - lse + kRowBias) * inv_w : 0.f;
          const __half fh = __float2half_rn(f);
          const __half fl = __float2half_rn(f - __half2float(fh));
          __half* ft_hi = reinterpret_cast<__half*>(m->ftab[quad][blk & 1][0]);
          __half* ft_lo = reinterpret_cast<__half*>(m->ftab[quad][blk & 1][1]);
          ft_hi[lane] = fh;
          ft_lo[lane] = fl;
          uint8_t* scr = scr0 + (blk & 1) * kScrTile;
          tmem_ld16_wait(pk);
#pragma unroll
          for (int i = 0; i < 4; ++i)
            *reinterpret_cast<uint4*>(scr + lane * kScrRow + i * 16) =
                make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
          if (blk < 3) tmem_ld16_issue(e_addr + (uint32_t)(blk + 1) * 16u, pk);  // next block in flight
          __syncwarp();
          // B operand: B[k = row][n] holds the row's factor in column 0 (high part) and 1 (low
          // part); with w = 16 the second head of the warp (rows 16..31) uses columns 2 and 3
          uint32_t bfrag[2][2];
#pragma unroll
          for (int ks = 0; ks < 2; ++ks) {
            const int col0 = (W == 16) ? 2 * ks : 0;
            uint32_t v0 = 0u, v1 = 0u;
            if (fg == col0 || fg == col0 + 1) {
              const uint32_t* tab = m->ftab[quad][blk & 1][fg - col0];
              v0 = tab[8 * ks + ft];      // rows 16 ks + 2 ft, + 1
              v1 = tab[8 * ks + 4 + ft];  // rows 16 ks + 8 + 2 ft, + 1
            }
            bfrag[ks][0] = v0;
            bfrag[ks][1] = v1;
          }
          const uint32_t scr_s = scr0_s + (uint32_t)(blk & 1) * kScrTile + ldm_off;
#pragma unroll
          for (int kg = 0; kg < 2; ++kg) {
            float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
              uint32_t a0, a1, a2, a3;
              ldmatrix_x4_trans(a0, a1, a2, a3, scr_s + (uint32_t)ks * 16u * kScrRow + (uint32_t)kg * 32u);
              mma_f16_16816(d0, d1, d2, d3, a0, a1, a2, a3, bfrag[ks][0], bfrag[ks][1]);
            }
            // d0 + d1: key fg, d2 + d3: key fg + 8 (columns 2 ft and 2 ft + 1 of the result)
            constexpr float kUnscale = 5.8207660913467407e-11f;  // 2^-34
            if (ft == 0 || (W == 16 && ft == 1)) {
              float* dst = m->pbuf[jp][quad][ft] + blk * 32 + kg * 16 + fg;
              dst[0] = (d0 + d1) * kUnscale;
              dst[8] = (d2 + d3) * kUnscale;
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(smem_u32(&m->e_empty[eb]));
          mbar_arrive(smem_u32(&m->prep_empty[eb]));
        }
        group_sync();  // every warp's window means are in place
        if (!alive) break;
        // thread <-> key column `row` of the tile: pool over the neighbouring keys, group maximum
        const int i = i0 + row;
        const bool owned = row >= rad && row < rad + p.ok && i < kj.s.prefix;
        const float (*pb)[2][kTile] = m->pbuf[jp];
        // window mean of head h at column c; keys outside the prefix hold the neutral element of
        // both pools (values are >= 0)
        auto mean_at = [&](int c, int h) -> float {
          const int key = i0 + c;
          if (h >= heads || key < 0 || key >= kj.s.prefix) return 0.f;
          if (W == 16) return pb[h >> 1][h & 1][c];
          if (W == 32) return pb[h][0][c];
          if (W == 64) return pb[2 * h][0][c] + pb[2 * h + 1][0][c];
          return (pb[0][0][c] + pb[1][0][c]) + (pb[2][0][c] + pb[3][0][c]);
        };
        constexpr int NH = 128 / W;  // heads a unit can hold
        float best = 0.f;
        if (!avg) {
          // max-pooling commutes with the group maximum: reduce over the query heads first;
          // the neighbours' values come from the neighbouring lanes, across a warp's edge from
          // shared memory
          float top = 0.f;
#pragma unroll
          for (int h = 0; h < NH; ++h) top = fmaxf(top, mean_at(row, h));
          best = top;
          for (int q = 1; q <= rad; ++q) {
            float up = __shfl_down_sync(0xffffffffu, top, q), dn = __shfl_up_sync(0xffffffffu, top, q);
            if (owned && lane + q > 31) {
              up = 0.f;
#pragma unroll
              for (int h = 0; h < NH; ++h) up = fmaxf(up, mean_at(row + q, h));
            }
            if (owned && lane - q < 0) {
              dn = 0.f;
#pragma unroll
              for (int h = 0; h < NH; ++h) dn = fmaxf(dn, mean_at(row - q, h));
            }
            best = fmaxf(best, fmaxf(up, dn));
          }
        } else {
#pragma unroll
          for (int h = 0; h < (NH < 4 ? NH : 4); ++h) {
            const float own = mean_at(row, h);
            float acc = own;
            for (int q = 1; q <= rad; ++q) {
              float up = __shfl_down_sync(0xffffffffu, own, q), dn = __shfl_up_sync(0xffffffffu, own, q);
              if (owned && lane + q > 31) up = mean_at(row + q, h);
              if (owned && lane - q < 0) dn = mean_at(row - q, h);
              acc += up + dn;
            }
            best = fmaxf(best, acc / (float)g.pool_kernel);
          }
        }
        if (owned) {
          float sc = best * scale;
          if (nunit == 2 && half == 0) {
            pend = sc;
          } else {
            if (nunit == 2) sc = fmaxf(sc, pend);
            score_row[(long long)kj.kvh * kj.s.prefix + i] = sc;
            if (sc > 0.f) {
              es += sc;
              et += sc * __logf(sc);
            }
          }
        }
      }
    }
    if (alive) flush_entropy();
  } else if (warp >= kValueWarp0) {
    // ================= value-norm warps: the V rows of the CTA's tiles ========================
    // Row L1 norms through the register-operand tensor path: a warp takes 16 rows, clears the
    // sign bits of the packed bf16 values and multiplies the 16 x 128 slab by a matrix of ones
    // (mma.sync m16n8k16, fp32 accumulate, exact products), which leaves the row sums in the
    // accumulator.  Thread (gq = lane / 4, tq = lane % 4) loads pieces tq, tq+4, tq+8, tq+12 of
    // rows gq and gq+8.  A tile owns at most 128 rows: two slabs per warp; the next slab's loads are
    // in flight while this one is reduced.  A warp's maximum over its slabs of one head leaves
    // the CTA once, when the CTA's tiles of that head are done (the head's counter then tells how
    // many warps of how many CTAs have reported).
    if (!p.vbar_in) {
      const int vw = warp - kValueWarp0, gq = lane >> 2, tq = lane & 3;
      struct Slab {
        const char* base;
        int row0, row_hi, rhead;
      };
      long long kappa = blockIdx.x;
      int sub = 0;  // which of the warp's two slabs of the tile
      auto next_slab = [&](Slab& sl) -> bool {
        KJob kj;
        for (;;) {
          if (kappa >= total_k || m->abort_flag) return false;
          kj = decode_job(p, m, kappa);
          if (!kj.idle) break;
          kappa += gridDim.x;
        }
        sl.base = p.v + ((size_t)kj.layer * p.v_ls + (long long)kj.kvh * g.v_sh +
                         kj.s.tok0 * g.v_st) * 2 + tq * 16;
        sl.row0 = kj.tile * p.ok + (vw + kVWarps * sub) * 16 + gq;
        if (++sub == 2) {
          sub = 0;
          kappa += gridDim.x;
        }
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
      float best = 0.f;
      int best_head = -1;
      auto publish = [&]() {
        if (best_head < 0) return;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
        if (lane == 0) {
          atomicMax(&p.vbar_bits[best_head], __float_as_uint(best));
          __threadfence();
          atomicAdd(&p.vcount[best_head], 1);
        }
        best = 0.f;
      };
      auto reduce = [&](const uint4 (&buf)[8], const Slab& sl) {
        if (sl.rhead != best_head) {  // warp-uniform
          publish();
          best_head = sl.rhead;
        }
        float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;  // d0: row gq, d2: row gq + 8
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint4 lo = buf[q], hi = buf[4 + q];
          mma_bf16_16816(d0, d1, d2, d3, lo.x & 0x7fff7fffu, hi.x & 0x7fff7fffu,
                         lo.y & 0x7fff7fffu, hi.y & 0x7fff7fffu, ones, ones);
          mma_bf16_16816(d0, d1, d2, d3, lo.z & 0x7fff7fffu, hi.z & 0x7fff7fffu,
                         lo.w & 0x7fff7fffu, hi.w & 0x7fff7fffu, ones, ones);
        }
        best = fmaxf(best, fmaxf(d0, d2));
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
      publish();
    }
  }

  // ---- teardown: everything this CTA started has finished before shared memory and TMEM go --
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

// entropy of one (layer, sequence) from the per-CTA sums, folded in a fixed order; also hands
// out the value norms
__global__ void __launch_bounds__(256)
entropy_finalize_tmem_kernel(Geom g, int grid, const float2* ent_part, double* entropy,
                             const float* vbar_in, const unsigned* vbar_bits, float* vbar_out) {
  __shared__ double rs[8], rt[8];
  const int prob = blockIdx.x, layer = prob / g.batch, b = prob - layer * g.batch;
  const SeqInfo s = seq_info(g, b);
  if (vbar_out && (int)threadIdx.x < g.n_kv_heads) {
    const size_t head = (size_t)prob * g.n_kv_heads + threadIdx.x;
    vbar_out[head] = vbar_in ? vbar_in[head] : __uint_as_float(vbar_bits[head]);
  }
  const float2* mine = ent_part + (size_t)prob * kMaxCtas * 4;
  double sum_s = 0.0, sum_t = 0.0;
  for (int i = threadIdx.x; i < grid * 4; i += 256) {
    const float2 e = mine[i];
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
  // two fold levels of at most 16 rows each where possible (one round of loads per level)
  l.kfold = l.tmax <= 256 ? 16 : ceil_div(l.tmax, 16);
  l.gmax = ceil_div(l.tmax, l.kfold);
  // slots of a layer: sum over sequences of ceil(n / ok) <= total / ok + batch, plus the padding of
  // heads longer than a round of CTAs to whole rounds (less than one round per sequence)
  const long long pad_cap = l.tmax > 64 ? (long long)g.batch * kMaxCtas : 0;
  const long long tiles_cap = (g.total_tokens / l.ok + g.batch + pad_cap) * g.n_kv_heads;
  l.kjobs_cap = (long long)n_layers * tiles_cap;
  l.heads_total = n_layers * g.batch * g.n_kv_heads;
  l.units_total = l.heads_total * l.nunit;
  size_t off = 0;
  l.off_sync = off;  // gcount, hcount, vcount, vbar_bits, entropy slots: zeroed every launch
  off = up256(off + sizeof(int) * ((size_t)l.units_total * (l.gmax + 1) + 2 * (size_t)l.heads_total));
  l.off_ent = off;
  off = up256(off + sizeof(float2) * 4 * kMaxCtas * (size_t)n_layers * g.batch);
  l.sync_bytes = off;
  l.off_part = off;
  off = up256(off + sizeof(float) * 128 * (size_t)l.kjobs_cap * l.nunit);
  l.off_gpart = off;
  off = up256(off + sizeof(float) * 128 * (size_t)l.units_total * l.gmax);
  l.total = off;
  return l;
}

// Does a launch on `grid` CTAs keep every head inside the rounds the exponent buffers span?
bool tmem_fits(const Geom& g, int grid) {
  const int nunit = first_unit_heads(g) ? 2 : 1;
  const int tmax = ceil_div(g.max_seqlen, kTile - 2 * g.pool_radius);
  return grid > 0 && tmax <= (nunit == 1 ? 3 * grid + 1 : grid + 1);
}

int tmem_grid(const Geom& g, int n_layers) {
  int sms = sm_count();
  if (sms > kMaxCtas) sms = kMaxCtas;
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
  p.kfold = lay.kfold;
  p.gmax = lay.gmax;
  p.tmax = lay.tmax;
  p.wait_cycles = options().wait_limit_cycles;
  p.vbar_in = vbar_in;
  p.scores = scores;
  p.v = (const char*)v;
  p.v_ls = v_ls;
  int* sync = reinterpret_cast<int*>(ws + lay.off_sync);
  p.gcount = sync;
  p.hcount = p.gcount + (size_t)lay.units_total * lay.gmax;
  p.vcount = p.hcount + lay.units_total;
  p.vbar_bits = reinterpret_cast<unsigned*>(p.vcount + lay.heads_total);
  p.ent_part = reinterpret_cast<float2*>(ws + lay.off_ent);
  p.part = reinterpret_cast<float*>(ws + lay.off_part);
  p.gpart = reinterpret_cast<float*>(ws + lay.off_gpart);
  p.status = reinterpret_cast<unsigned*>(ws_base);

  rc = check_cuda(cudaMemsetAsync(ws + lay.off_sync, 0, lay.sync_bytes, stream), "sync scratch clear");
  if (rc != LAVA_OK) return rc;
  void (*kern)(const CUtensorMap, const CUtensorMap, const TmemParams) = nullptr;
  switch (g.window) {
    case 16: kern = lava_score_tmem_kernel<16>; break;
    case 32: kern = lava_score_tmem_kernel<32>; break;
    case 64: kern = lava_score_tmem_kernel<64>; break;
    default: kern = lava_score_tmem_kernel<128>; break;
  }
  rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kSmemBytes),
                  "cudaFuncSetAttribute(single-pass score)");
  if (rc != LAVA_OK) return rc;
  void* args[3] = {&map_q, &map_k, &p};
  rc = check_cuda(cudaLaunchCooperativeKernel((const void*)kern, dim3(grid),
                                              dim3(kThreads), args, kSmemBytes, stream),
                  "score (single-pass) launch");
  if (rc != LAVA_OK) return rc;
  entropy_finalize_tmem_kernel<<<n_layers * g.batch, 256, 0, stream>>>(
      g, grid, p.ent_part, entropy, vbar_in, p.vbar_bits, vbar_out);
  count_launches(2);
  return check_cuda(cudaGetLastError(), "entropy finalize launch");
}

}  // namespace lava
