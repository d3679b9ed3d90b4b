// LAVa score, Blackwell path: bf16, head_dim 128, w in {16, 32, 64, 128}, up to 256 window-query
// rows per KV head (a unit holds at most 128; larger query groups run as two units).
//
// One persistent, warp-specialised kernel (one CTA per SM, cooperative launch so that every CTA
// is resident) runs two pipelines over 128-key tiles of K, both fed by TMA into 128B-swizzled
// shared memory and contracted with tcgen05.mma into TMEM:
//
//   pass 1 (statistics)  S = Q_g K^T  (rows = the unit's window queries, columns = keys)
//       one thread per row reads its TMEM lane and keeps a running (max, sum of exp2) over the
//       keys the query may see (Sec. 2: softmax over i <= j).  Work is dealt to CTAs in chunks
//       of consecutive tiles of one head; a chunk's statistics leave the CTA once, through a
//       publisher warp that also counts the head's published chunks.  Seven more warps stream
//       the chunk's V rows for the value norm (Theorem 1: max_k ||V[k]||_1).
//   pass 2 (scores)      S^T = K Q_g^T (rows = keys, columns = window queries)
//       one thread per key: a_h[i] = (1/w) sum_t exp2(z - lse_t) per query head in registers,
//       pooled over the token axis through shared memory, scaled by Vbar * c_hat, reduced with
//       the GQA group maximum, written once; entropy sums go to ordered per-chunk slots
//       (Definition 1, Sec. 4.2, Sec. 4.3, Sec. 5.1 pooling).
//
// The exponentials bound the kernel, so the eight consumer warps are not split by pass: two
// groups of four warps each own one TMEM buffer of BOTH pipelines and take their tiles in a
// static order that alternates the passes, which keeps two exp-issuing warps on every scheduler.
//
// Pass 2 trails pass 1 by a bounded number of tiles (K tiles are loaded with an evict-last hint
// in pass 1 and evict-first in pass 2, V rows with evict-first), so part of its K tiles are
// still in L2; how many depends on the chunk length (see chunk_tiles_for).  Every wait
// (mbarrier, head counters) is bounded in time; on expiry the kernel sets
// LAVA_DEV_WAIT_EXPIRED, drains its copies, frees TMEM and returns.
#include "sm100_ptx.cuh"

namespace lava {
namespace {

using namespace sm100;

constexpr int kTile = 128;           // keys per tile
constexpr int kThreads = 640;        // 20 warps: 5 service, 8 consumer, 7 value-norm
constexpr int kVWarps = 7;
constexpr int kVRows = kVWarps * 2;  // V rows per load step (16 threads per row)
constexpr int kMma2Warp = 19;        // issues the pass-2 MMAs (warp 2 issues pass 1)
constexpr int kStages = 2;           // K stages per pipeline
constexpr int kMaxBatch = 512;       // sequences the in-kernel chunk schedule can index
constexpr uint32_t kTileBytes = 128 * 128 * 2;  // one [128 x 128] bf16 tile = 2 swizzled blocks
constexpr uint32_t kHalfBytes = kTileBytes / 2;

// shared memory map (bytes from a 1024-aligned base)
// Two small operands in the un-swizzled K-major layout (8 x 16-byte core matrices, 128 B apart
// along the rows, 2048 B apart along k) feed one extra k-step of every pass-2 tile: a [128 x 16]
// tile whose first three columns are ones, and per head a [128 x 16] tile that carries, per window
// query, minus its log2-sum-exp (in logit units) split into three bf16 terms.  The MMA thereby
// adds the softmax normaliser to every logit, and the score warps need no per-column constants.
constexpr uint32_t kOffOnes = 0;
constexpr uint32_t kOffBias = 4096;          // two slots of 4 KB
constexpr uint32_t kSmallTileBytes = 4096;
constexpr uint32_t kOffQ1 = 16384;
constexpr uint32_t kOffQ2 = kOffQ1 + kTileBytes;
constexpr uint32_t kOffK1 = kOffQ2 + kTileBytes;
constexpr uint32_t kOffK2 = kOffK1 + kStages * kTileBytes;
constexpr uint32_t kOffMisc = kOffK2 + kStages * kTileBytes;  // 16 KB + 192 KB
constexpr uint32_t kMiscBytes = 15360;
constexpr uint32_t kSmemBytes = kOffMisc + kMiscBytes + 1024;  // + alignment slack

struct Prep {                 // what the score warps need to know about a head
  float scale;                // Vbar * c_hat
  float pad[3];
};

struct Misc {
  unsigned long long k1_full[kStages], k1_empty[kStages], k2_full[kStages], k2_empty[kStages];
  unsigned long long q1_full, q1_empty, q2_full, q2_empty;
  unsigned long long s1_full[2], s1_empty[2], s2_full[2], s2_empty[2];
  unsigned long long pub_full[2], pub_empty[2], prep_full[2], prep_empty[2];
  unsigned long long gsync[2];        // rendezvous of the four warps of a consumer group
  unsigned long long drain, drain2;
  uint32_t tmem_base;
  volatile int abort_flag;
  long long wait_cycles;              // limit of the waits that an abort may end (launch parameter)
  int sched_total1, sched_total2;     // chunks per layer of pass 1 / pass 2
  int lead_tiles;                     // tile slots pass 1 runs ahead of pass 2 in a CTA's order
  alignas(16) float pub[2][2][128];   // [slot][group][query]: log2-sum-exp of a finished chunk
  Prep prep[2];
  alignas(16) float a[2][2][4][kTile];  // [group][tile parity][query head][key]: window means
  int pref1[kMaxBatch + 1], pref2[kMaxBatch + 1];  // exclusive scans of chunks per sequence
};
static_assert(sizeof(Misc) <= kMiscBytes, "misc region too small");

struct Sm100Params {
  Geom g;
  int n_layers;
  int chunk_tiles;          // tiles per chunk
  int out_keys;             // keys a pass-2 tile owns: 128 - 2 * pool_radius
  int cph1_max, cph2_max;   // chunks per head at max_seqlen (strides of the scratch arrays)
  int lead_extra;           // tiles pass 1 leads pass 2 by, beyond what head completion needs
  int split;                // 1: every KV head is scored as two halves of its query group
  int g0;                   // query heads in the first half (split mode)
  long long wait_cycles;    // SM cycles after which a wait on another role or CTA gives up
  const float* vbar_in;
  float* scores;
  float* vbar_out;
  const char* v;
  long long v_ls;
  // scratch
  float* part;              // [heads_total][cph1_max][128] log2-sum-exp per chunk and query
  int* counters;            // [heads_total] published pass-1 chunks
  int* vcount;              // [heads_total] finished value-norm warps
  unsigned* vbar_bits;      // [heads_total]
  float2* ent_part;         // [heads_total][cph2_max][8 consumer warps] (sum s, sum s ln s)
  unsigned* status;
};

// ------------------------------------------------------------------------------------------
// chunk schedule (identical in every role and every CTA, so no descriptors travel)
// ------------------------------------------------------------------------------------------
struct Chunk {
  int head;    // linear index of the scored unit (a KV head, or one half of its query group in
               // split mode): counters, chunk partials and entropy slots are per unit
  int rhead;   // linear KV head index = (layer * batch + b) * H_kv + kvh (value norms)
  int layer, b, kvh;
  int half;    // which half of the query group (0 unless split)
  int q0;      // first query head of the unit inside the sequence's H_q heads
  int group;   // query heads of the unit
  int index;   // chunk number inside the head
  int cph;     // chunks of this head
  int tile0, ntiles;
  SeqInfo s;
};

__device__ inline int tiles_of(const Sm100Params& p, const SeqInfo& s, int pass) {
  return pass == 1 ? ceil_div(s.n, kTile) : ceil_div(s.prefix, p.out_keys);
}

__device__ inline Chunk decode_chunk(const Sm100Params& p, const Misc* m, int c, int pass) {
  const int* pref = pass == 1 ? m->pref1 : m->pref2;
  const int per_layer = pass == 1 ? m->sched_total1 : m->sched_total2;
  Chunk ck;
  ck.layer = c / per_layer;
  const int r = c - ck.layer * per_layer;
  const int hkv = p.g.n_kv_heads << p.split;  // scored units per sequence
  int lo = 0, hi = p.g.batch;  // largest b with hkv * pref[b] <= r
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (hkv * pref[mid] <= r) lo = mid; else hi = mid;
  }
  ck.b = lo;
  ck.cph = pref[lo + 1] - pref[lo];
  const int r2 = r - hkv * pref[lo];
  const int unit = r2 / ck.cph;
  ck.index = r2 - unit * ck.cph;
  ck.head = (ck.layer * p.g.batch + ck.b) * hkv + unit;
  ck.half = p.split ? (unit & 1) : 0;
  ck.kvh = unit >> p.split;
  ck.rhead = (ck.layer * p.g.batch + ck.b) * p.g.n_kv_heads + ck.kvh;
  ck.group = p.split ? (ck.half ? p.g.group - p.g0 : p.g0) : p.g.group;
  ck.q0 = ck.kvh * p.g.group + ck.half * p.g0;
  ck.s = seq_info(p.g, ck.b);
  // the head's tiles are spread evenly over its chunks (none longer than chunk_tiles): a short
  // last chunk would leave the CTAs with unequal loads
  const long long tiles = tiles_of(p, ck.s, pass);
  ck.tile0 = (int)(ck.index * tiles / ck.cph);
  ck.ntiles = (int)((ck.index + 1) * tiles / ck.cph) - ck.tile0;
  return ck;
}

// ------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------
template <int W>
__global__ void __launch_bounds__(kThreads, 1)
lava_score_sm100_kernel(const __grid_constant__ CUtensorMap map_q,
                        const __grid_constant__ CUtensorMap map_k, const Sm100Params p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  Misc* m = reinterpret_cast<Misc*>(gen + kOffMisc);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const Geom& g = p.g;
  const int units = g.n_kv_heads << p.split;  // scored units per sequence
  if (batch_has_short_sequence(g)) {  // every CTA sees the same lengths: all of them leave
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(p.status, LAVA_DEV_SHORT_SEQUENCE);
    return;
  }

  // ---- chunk schedule: exclusive scans of chunks per sequence, both passes -------------------
  {
    __shared__ int wsum[2][kThreads / 32];
    int c1 = 0, c2 = 0;
    if ((int)threadIdx.x < g.batch) {
      const SeqInfo s = seq_info(g, threadIdx.x);
      if (s.n < g.window && blockIdx.x == 0) atomicOr(p.status, LAVA_DEV_SHORT_SEQUENCE);
      c1 = ceil_div(ceil_div(s.n, kTile), p.chunk_tiles);
      c2 = ceil_div(ceil_div(s.prefix, p.out_keys), p.chunk_tiles);
    }
    int i1 = c1, i2 = c2;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y1 = __shfl_up_sync(0xffffffffu, i1, o), y2 = __shfl_up_sync(0xffffffffu, i2, o);
      if (lane >= o) {
        i1 += y1;
        i2 += y2;
      }
    }
    if (lane == 31) {
      wsum[0][warp] = i1;
      wsum[1][warp] = i2;
    }
    __syncthreads();
    int b1 = 0, b2 = 0;
    for (int wdx = 0; wdx < warp; ++wdx) {
      b1 += wsum[0][wdx];
      b2 += wsum[1][wdx];
    }
    if ((int)threadIdx.x < g.batch) {
      m->pref1[threadIdx.x + 1] = b1 + i1;
      m->pref2[threadIdx.x + 1] = b2 + i2;
    }
    if (threadIdx.x == 0) {
      m->pref1[0] = 0;
      m->pref2[0] = 0;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      m->sched_total1 = units * m->pref1[g.batch];
      m->sched_total2 = units * m->pref2[g.batch];
      // How far pass 1 must lead pass 2 in a CTA's own order (see the consumer warps).  With
      // rho = pass-2 chunks per pass-1 chunk: rho * (1 + (longest head + drift) / grid) chunks,
      // where drift is how far the two passes' chunk numbering can diverge inside a layer.
      const double t1 = (double)m->sched_total1, t2 = (double)m->sched_total2;
      const double rho = t1 > 0.0 ? t2 / t1 : 1.0;
      double drift = 0.0, longest = 0.0;
      for (int b = 0; b < g.batch; ++b) {
        const double c1 = m->pref1[b + 1] - m->pref1[b], c2 = m->pref2[b + 1] - m->pref2[b];
        const double at = fabs(units * (m->pref1[b] * rho - m->pref2[b]));
        drift = fmax(drift, at + units * fabs(c1 * rho - c2));
        longest = fmax(longest, c1);
      }
      const double lead = p.chunk_tiles * rho * (1.0 + (longest + drift) / (double)gridDim.x);
      m->lead_tiles = (int)ceil(lead) + p.lead_extra;
    }
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&m->k1_full[s]), 1);
      mbar_init(smem_u32(&m->k1_empty[s]), 1);
      mbar_init(smem_u32(&m->k2_full[s]), 1);
      mbar_init(smem_u32(&m->k2_empty[s]), 1);
    }
    mbar_init(smem_u32(&m->q1_full), 1);
    mbar_init(smem_u32(&m->q1_empty), 1);
    mbar_init(smem_u32(&m->q2_full), 1);
    mbar_init(smem_u32(&m->q2_empty), 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&m->s1_full[s]), 1);
      mbar_init(smem_u32(&m->s1_empty[s]), 4);   // one arrival per warp of the group
      mbar_init(smem_u32(&m->s2_full[s]), 1);
      mbar_init(smem_u32(&m->s2_empty[s]), 4);
      mbar_init(smem_u32(&m->pub_full[s]), 8);   // the eight consumer warps
      mbar_init(smem_u32(&m->pub_empty[s]), 1);
      mbar_init(smem_u32(&m->prep_full[s]), 1);
      mbar_init(smem_u32(&m->prep_empty[s]), 8);
      mbar_init(smem_u32(&m->gsync[s]), 4);
    }
    mbar_init(smem_u32(&m->drain), 1);
    mbar_init(smem_u32(&m->drain2), 1);
    m->abort_flag = 0;
    m->wait_cycles = p.wait_cycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  // ones tile: columns 0..2 of every row hold bf16 1.0; bias tiles start as zeros
  for (int i = threadIdx.x; i < (int)(3 * kSmallTileBytes / 16); i += kThreads) {
    uint4 val = make_uint4(0, 0, 0, 0);
    if (i < 128) val = make_uint4(0x3f803f80u, 0x00003f80u, 0, 0);  // k-core 0 of row i
    *reinterpret_cast<uint4*>(gen + kOffOnes + i * 16) = val;
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 2) tmem_alloc(smem_u32(&m->tmem_base), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = m->tmem_base;
  const long long total1 = (long long)p.n_layers * m->sched_total1;
  const long long total2 = (long long)p.n_layers * m->sched_total2;

  if (warp == 0) {
    // ================= pass-1 producer: Q of the head, K tiles =============================
    if (lane == 0) {
      const uint64_t keep = policy_evict_last();
      int q_loads = 0;
      long long n = 0;  // K loads issued
      for (long long c = blockIdx.x; c < total1 && !m->abort_flag; c += gridDim.x) {
        const Chunk ck = decode_chunk(p, m, c, 1);
        if (!wait_bar(smem_u32(&m->q1_empty), (q_loads & 1) ^ 1, m, p.status)) break;
        {
          const uint32_t bar = smem_u32(&m->q1_full);
          mbar_expect_tx(bar, kTileBytes);
          const int row0 = (ck.b * g.n_q_heads + ck.q0) * W;
          tma_load_3d(base + kOffQ1, &map_q, 0, row0, ck.layer, bar);
          tma_load_3d(base + kOffQ1 + kHalfBytes, &map_q, 64, row0, ck.layer, bar);
          ++q_loads;
        }
        bool ok = true;
        for (int t = 0; t < ck.ntiles && ok; ++t) {
          const int st = (int)(n % kStages);
          ok = wait_bar(smem_u32(&m->k1_empty[st]), (uint32_t)((n / kStages) & 1) ^ 1, m, p.status);
          if (!ok) break;
          const uint32_t bar = smem_u32(&m->k1_full[st]);
          mbar_expect_tx(bar, kTileBytes);
          const int tok = (int)ck.s.tok0 + (ck.tile0 + t) * kTile;
          tma_load_4d(base + kOffK1 + st * kTileBytes, &map_k, 0, tok, ck.kvh, ck.layer, bar, keep);
          tma_load_4d(base + kOffK1 + st * kTileBytes + kHalfBytes, &map_k, 64, tok, ck.kvh,
                      ck.layer, bar, keep);
          ++n;
        }
        if (!ok) break;
      }
      // copies still in flight land before this CTA gives up its shared memory
      for (long long j = (n > kStages ? n - kStages : 0); j < n; ++j)
        wait_bar(smem_u32(&m->k1_full[j % kStages]), (uint32_t)((j / kStages) & 1), m, p.status,
                 false);
      if (q_loads > 0)
        wait_bar(smem_u32(&m->q1_full), (uint32_t)((q_loads - 1) & 1), m, p.status, false);
    }
  } else if (warp == 1) {
    // ================= pass-2 producer: head data for the score warps, Q, K tiles ============
    const uint64_t drop = policy_evict_first();
    int q_loads = 0;
    long long n = 0, j = 0;  // K loads issued, chunks prepared
    for (long long c = blockIdx.x; c < total2; c += gridDim.x, ++j) {
      const Chunk ck = decode_chunk(p, m, c, 2);
      const int slot = (int)(j & 1);
      // wait until every pass-1 chunk of the head has been published and its value norm is final
      bool ok = true;
      const int cph1 = ceil_div(ceil_div(ck.s.n, kTile), p.chunk_tiles);
      if (lane == 0) {
        const int want_v = p.vbar_in ? 0 : kVWarps * cph1;
        const long long t0 = clock64();
        while (ld_acquire(&p.counters[ck.head]) < cph1 ||
               (want_v && ld_acquire(&p.vcount[ck.rhead]) < want_v)) {
          if (m->abort_flag) break;
          __nanosleep(100);
          if (clock64() - t0 > m->wait_cycles) give_up(m, p.status);
        }
        ok = !m->abort_flag &&
             wait_bar(smem_u32(&m->prep_empty[slot]), (uint32_t)((j >> 1) & 1) ^ 1, m, p.status);
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      // Fold the head's chunk partials, in chunk order, into one log2-sum-exp per window query
      // (lane l: queries 4l .. 4l+3).  Every CTA that scores a chunk of the head does this for
      // itself, with the same operations in the same order, so all of them get the same bits
      // and no CTA waits for another one's fold.
      {
        const float4* pp =
            reinterpret_cast<const float4*>(p.part + (size_t)ck.head * p.cph1_max * 128) + lane;
        float big[4], sum[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          big[q] = -INFINITY;
          sum[q] = 0.f;
        }
#pragma unroll 1
        for (int i0 = 0; i0 < cph1; i0 += 16) {
          float4 pr[16];
#pragma unroll
          for (int u = 0; u < 16; ++u)
            pr[u] = (i0 + u < cph1) ? __ldcg(pp + (size_t)(i0 + u) * 32)
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
        // per window query: minus the log2-sum-exp in logit units, as three bf16 terms
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int r = 4 * lane + q;
          uint32_t w0 = 0xf149u, w1 = 0;  // about -1e30 for a query without any key
          if (sum[q] > 0.f) {
            const float b = -(big[q] + fast_log2(sum[q])) / g.scale_log2;
            const __nv_bfloat16 b0 = __float2bfloat16_rn(b);
            const float r1 = b - __bfloat162float(b0);
            const __nv_bfloat16 b1 = __float2bfloat16_rn(r1);
            const __nv_bfloat16 b2 = __float2bfloat16_rn(r1 - __bfloat162float(b1));
            w0 = (uint32_t)__bfloat16_as_ushort(b0) | ((uint32_t)__bfloat16_as_ushort(b1) << 16);
            w1 = (uint32_t)__bfloat16_as_ushort(b2);
          }
          *reinterpret_cast<uint4*>(gen + kOffBias + slot * kSmallTileBytes + r * 16) =
              make_uint4(w0, w1, 0, 0);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      if (lane == 0) {
        const float vb = p.vbar_in ? p.vbar_in[ck.rhead]
                                   : __uint_as_float(__ldcg(p.vbar_bits + ck.rhead));
        m->prep[slot].scale = vb * g.c_hat;
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&m->prep_full[slot]));
        ok = wait_bar(smem_u32(&m->q2_empty), (q_loads & 1) ^ 1, m, p.status);
        if (ok) {
          const uint32_t bar = smem_u32(&m->q2_full);
          mbar_expect_tx(bar, kTileBytes);
          const int row0 = (ck.b * g.n_q_heads + ck.q0) * W;
          tma_load_3d(base + kOffQ2, &map_q, 0, row0, ck.layer, bar);
          tma_load_3d(base + kOffQ2 + kHalfBytes, &map_q, 64, row0, ck.layer, bar);
          ++q_loads;
        }
        for (int t = 0; t < ck.ntiles && ok; ++t) {
          const int st = (int)(n % kStages);
          ok = wait_bar(smem_u32(&m->k2_empty[st]), (uint32_t)((n / kStages) & 1) ^ 1, m, p.status);
          if (!ok) break;
          const uint32_t bar = smem_u32(&m->k2_full[st]);
          mbar_expect_tx(bar, kTileBytes);
          // the tile starts pool_radius keys before the first key it owns (halo for pooling)
          const int tok = (int)ck.s.tok0 + (ck.tile0 + t) * p.out_keys - g.pool_radius;
          tma_load_4d(base + kOffK2 + st * kTileBytes, &map_k, 0, tok, ck.kvh, ck.layer, bar, drop);
          tma_load_4d(base + kOffK2 + st * kTileBytes + kHalfBytes, &map_k, 64, tok, ck.kvh,
                      ck.layer, bar, drop);
          ++n;
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
    }
    if (lane == 0) {
      for (long long i = (n > kStages ? n - kStages : 0); i < n; ++i)
        wait_bar(smem_u32(&m->k2_full[i % kStages]), (uint32_t)((i / kStages) & 1), m, p.status,
                 false);
      if (q_loads > 0)
        wait_bar(smem_u32(&m->q2_full), (uint32_t)((q_loads - 1) & 1), m, p.status, false);
    }
  } else if (warp == 2 || warp == kMma2Warp) {
    // ================= MMA issuers: warp 2 serves pass 1, the last warp pass 2 ================
    if (lane == 0) {
      const bool first = warp == 2;
      const int pass = first ? 1 : 2;
      const long long total = first ? total1 : total2;
      unsigned long long* k_full = first ? m->k1_full : m->k2_full;
      unsigned long long* k_empty = first ? m->k1_empty : m->k2_empty;
      unsigned long long* s_full = first ? m->s1_full : m->s2_full;
      unsigned long long* s_empty = first ? m->s1_empty : m->s2_empty;
      const uint32_t q_full = smem_u32(first ? &m->q1_full : &m->q2_full);
      const uint32_t q_empty = smem_u32(first ? &m->q1_empty : &m->q2_empty);
      const uint32_t q_addr = base + (first ? kOffQ1 : kOffQ2);
      const uint32_t k_addr = base + (first ? kOffK1 : kOffK2);
      const uint32_t d_base = tmem + (first ? 0u : 256u);
      long long n = 0;
      int q_uses = 0;
      bool ok = true;
      for (long long c = blockIdx.x; c < total && ok; c += gridDim.x) {
        const int nt = decode_chunk(p, m, c, pass).ntiles;
        const int slot = q_uses & 1;  // chunk ordinal parity = slot of the head's bias tile
        ok = wait_bar(q_full, (uint32_t)(q_uses & 1), m, p.status);
        if (ok && !first)
          ok = wait_bar(smem_u32(&m->prep_full[slot]), (uint32_t)((q_uses >> 1) & 1), m, p.status);
        ++q_uses;
        for (int t = 0; t < nt && ok; ++t, ++n) {
          const int st = (int)(n % kStages), buf = (int)(n & 1);
          ok = wait_bar(smem_u32(&k_full[st]), (uint32_t)((n / kStages) & 1), m, p.status) &&
               wait_bar(smem_u32(&s_empty[buf]), (uint32_t)((n >> 1) & 1) ^ 1, m, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t d = d_base + (uint32_t)buf * 128u;
          const uint32_t kt = k_addr + st * kTileBytes;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (uint32_t)(kk >> 2) * kHalfBytes + (uint32_t)(kk & 3) * 32u;
            // pass 1: D[query, key] = Q K^T; pass 2: D[key, query] = K Q^T
            if (first) umma_bf16(d, make_desc(q_addr + off), make_desc(kt + off), kIdesc, kk > 0);
            else umma_bf16(d, make_desc(kt + off), make_desc(q_addr + off), kIdesc, kk > 0);
          }
          // pass 2: one more k-step adds minus the log2-sum-exp of every window query
          if (!first)
            umma_bf16(d, make_desc_plain(base + kOffOnes),
                      make_desc_plain(base + kOffBias + slot * kSmallTileBytes), kIdesc, 1);
          umma_commit(smem_u32(&k_empty[st]));
          umma_commit(smem_u32(&s_full[buf]));
        }
        // the query tile may be replaced once the MMAs of its last user have completed
        if (ok) umma_commit(q_empty);
      }
      // every MMA this thread issued has completed before TMEM is released
      unsigned long long* drain = first ? &m->drain : &m->drain2;
      umma_commit(smem_u32(drain));
      wait_bar(smem_u32(drain), 0, m, p.status, false);
    }
  } else if (warp == 3) {
    // ================= publisher: chunk statistics leave the CTA ============================
    long long j = 0;
    for (long long c = blockIdx.x; c < total1; c += gridDim.x, ++j) {
      const Chunk ck = decode_chunk(p, m, c, 1);
      const int slot = (int)(j & 1);
      bool ok = true;
      if (lane == 0)
        ok = wait_bar(smem_u32(&m->pub_full[slot]), (uint32_t)((j >> 1) & 1), m, p.status);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      // lane l carries rows 4l .. 4l+3; the two consumer groups' partials are merged first
      {
        const float4 a4 = reinterpret_cast<const float4*>(m->pub[slot][0])[lane];
        const float4 b4 = reinterpret_cast<const float4*>(m->pub[slot][1])[lane];
        float4 o4;
        o4.x = lse2(a4.x, b4.x);
        o4.y = lse2(a4.y, b4.y);
        o4.z = lse2(a4.z, b4.z);
        o4.w = lse2(a4.w, b4.w);
        float* dst = p.part + ((size_t)ck.head * p.cph1_max + ck.index) * 128;
        reinterpret_cast<float4*>(dst)[lane] = o4;
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&m->pub_empty[slot]));
        // release: the partial written above is visible to whoever sees the new count
        red_add_release(&p.counters[ck.head], 1);
      }
    }
  } else if (warp >= 4 && warp < 12) {
    // ================= consumers: two groups of four warps, each serving BOTH passes ==========
    // Group 0 owns TMEM buffer 0 of either pipeline (the even tiles a CTA sees), group 1 buffer
    // 1, so the exponential unit of every scheduler has two warps to draw from.
    //   pass 1: thread = (query head, window query) row, running (max, sum of exp2) per chunk
    //   pass 2: thread = key, window-mean attention per query head, pooling, score, entropy
    // The order in which the tiles are taken is static and alternates tile by tile: counting a
    // CTA's tiles in slots (chunk ordinal * chunk_tiles + tile), the pass-1 tile comes first
    // while its slot, scaled to pass-2 slots, is at most lead_tiles beyond the next pass-2
    // slot.  The lead is long enough that every pass-1 chunk of a head precedes, in every CTA,
    // every pass-2 tile of that head or a later one, so the wait for a head's statistics
    // always ends; it is short enough to keep the K tiles between the two passes in L2, and the
    // fine alternation keeps both TMA/MMA pipelines busy all the time.
    constexpr int NH = 128 / W;  // query heads that fit the 128 columns
    const int grp = (warp - 4) >> 2, quad = warp & 3, row = quad * 32 + lane;
    const int t_in_win = row % W;
    const int rad = g.pool_radius;
    const float inv_w = 1.0f / (float)W;
    const float sc2 = g.scale_log2;
    const bool avg = g.pool_kind == LAVA_POOL_AVG;
    const uint32_t gbar = smem_u32(&m->gsync[grp]);
    uint32_t gphase = 0;
    bool alive = true;
    // rendezvous of the group's four warps (bounded, and it ends when the CTA aborts)
    auto group_sync = [&]() {
      __syncwarp();  // the lanes' shared-memory writes are ordered before lane 0's arrival
      if (lane == 0) mbar_arrive(gbar);
      if (!__all_sync(0xffffffffu, wait_bar(gbar, gphase & 1, m, p.status))) alive = false;
      ++gphase;
    };

    // ---- cursors over the CTA's chunks of both passes ---------------------------------------
    // the order rule compares (pass-1 slot) * S2 with (pass-2 slot + lead) * S1; both sides are
    // kept as running sums so that a step costs an addition
    const long long sched1 = m->sched_total1, sched2 = m->sched_total2;
    long long ord1 = 0, ord2 = (long long)m->lead_tiles * sched1;
    // Tile n of a pass (counted over the CTA) belongs to group n & 1, so a group's own tiles are
    // two apart: t is the index of its next own tile inside the open chunk (it may point past the
    // chunk's end, into a later chunk), n the tile's number in the CTA.
    int c1 = blockIdx.x, t1 = grp, n1 = grp, j1 = 0, last1 = 0;
    ord1 += grp * sched2;
    bool has1 = c1 < total1;
    Chunk k1;
    float mx = -INFINITY, z = 0.f;
    auto open1 = [&]() {
      k1 = decode_chunk(p, m, c1, 1);
      // keys this query may see: i < n and i <= P + t
      last1 = row < k1.group * W ? min(k1.s.n, k1.s.prefix + t_in_win + 1) : 0;
    };
    if (has1) open1();
    int c2 = blockIdx.x, t2 = grp, n2 = grp, j2 = 0;
    ord2 += grp * sched1;
    bool has2 = c2 < total2, prepped = false;
    Chunk k2;
    float es = 0.f, et = 0.f;  // entropy sums of this thread's keys over the chunk
    float* dst_head = nullptr;   // score row of the open chunk's KV head
    float chunk_scale = 0.f;     // Vbar * c_hat of that head
    auto open2 = [&]() {
      k2 = decode_chunk(p, m, c2, 2);
      dst_head = p.scores + (size_t)k2.layer * g.total_scores + k2.s.score_off +
                 (long long)k2.kvh * k2.s.prefix;
    };
    if (has2) open2();

    while (alive) {
      // ---- close the pass-1 chunks that lie before this group's next tile ---------------------
      while (has1 && t1 >= k1.ntiles) {
        // hand the chunk's statistics (as one log2-sum-exp) to the publisher warp
        const int slot = j1 & 1;
        if (!__all_sync(0xffffffffu, wait_bar(smem_u32(&m->pub_empty[slot]),
                                              (uint32_t)((j1 >> 1) & 1) ^ 1, m, p.status))) {
          alive = false;
          break;
        }
        m->pub[slot][grp][row] = z > 0.f ? mx + fast_log2(z) : -INFINITY;
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&m->pub_full[slot]));
        mx = -INFINITY;
        z = 0.f;
        ++j1;
        c1 += gridDim.x;
        ord1 += (long long)(p.chunk_tiles - k1.ntiles) * sched2;  // the next chunk starts a new run of slots
        t1 -= k1.ntiles;
        has1 = c1 < total1;
        if (has1) open1();
      }
      // ---- the same for pass 2 ----------------------------------------------------------------
      while (alive && has2 && t2 >= k2.ntiles) {
        // entropy sums of the chunk in a fixed order: keys of a thread, lanes of a warp; the
        // eight warp sums of a chunk are added up, in order, by the finishing kernel
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          es += __shfl_down_sync(0xffffffffu, es, o);
          et += __shfl_down_sync(0xffffffffu, et, o);
        }
        if (lane == 0) {
          p.ent_part[((size_t)k2.head * p.cph2_max + k2.index) * 8 + grp * 4 + quad] =
              make_float2(es, et);
          mbar_arrive(smem_u32(&m->prep_empty[j2 & 1]));
        }
        es = 0.f;
        et = 0.f;
        prepped = false;
        ++j2;
        c2 += gridDim.x;
        ord2 += (long long)(p.chunk_tiles - k2.ntiles) * sched1;
        t2 -= k2.ntiles;
        has2 = c2 < total2;
        if (has2) open2();
      }
      if (!alive || (!has1 && !has2)) break;

      bool take1 = has1;
      if (has1 && has2) take1 = ord1 <= ord2;

      if (take1) {
        // ---- a pass-1 tile: running softmax statistics of 128 keys ------------------------------
        if (!__all_sync(0xffffffffu, wait_bar(smem_u32(&m->s1_full[grp]),
                                              (uint32_t)((n1 >> 1) & 1), m, p.status)))
          break;
        tc_fence_after();
        const int limit = max(0, min(kTile, last1 - (k1.tile0 + t1) * kTile));
        const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)grp * 128u;
#pragma unroll 1
        for (int blk = 0; blk < 4; ++blk) {
          const int cnt = limit - blk * 32;
          float cur[32];
          tmem_ld32_issue(taddr + blk * 32, cur);
          tmem_ld_wait(cur);
          if (cnt >= 32) {
            // stage by stage (maxima, scaled differences, exponentials, a fixed summation tree)
            // four running maxima (few live registers; the chains are independent)
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
              cur[i] = r.x;
              cur[i + 1] = r.y;
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) cur[i] = fast_exp2(cur[i]);
            z += tree_sum32(cur);
          } else if (cnt > 0) {
            float bm = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (i < cnt) bm = fmaxf(bm, cur[i]);
            const float nm = bm * sc2;
            if (nm > mx) {
              z *= fast_exp2(mx - nm);
              mx = nm;
            }
            float zz = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (i < cnt) zz += fast_exp2(fmaf(cur[i], sc2, -mx));
            z += zz;
          }
        }
        tc_fence_before();
        __syncwarp();  // every lane has finished reading the accumulator
        if (lane == 0) mbar_arrive(smem_u32(&m->s1_empty[grp]));
        t1 += 2;
        n1 += 2;
        ord1 += 2 * sched2;
      } else {
        // ---- a pass-2 tile: scores of 128 - 2 * pool_radius keys --------------------------------
        if (!prepped) {
          if (!__all_sync(0xffffffffu, wait_bar(smem_u32(&m->prep_full[j2 & 1]),
                                                (uint32_t)((j2 >> 1) & 1), m, p.status)))
            break;
          prepped = true;
          chunk_scale = m->prep[j2 & 1].scale;
        }
        if (!__all_sync(0xffffffffu, wait_bar(smem_u32(&m->s2_full[grp]),
                                              (uint32_t)((n2 >> 1) & 1), m, p.status)))
          break;
        const int tile = k2.tile0 + t2;
        tc_fence_after();
        float acc[NH];
#pragma unroll
        for (int h = 0; h < NH; ++h) acc[h] = 0.f;
        const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + 256u + (uint32_t)grp * 128u;
        // window queries come in blocks of 32 columns; a block lies inside one query head when
        // W >= 32, and holds two heads when W == 16
        const int nblk = (k2.group * W + 31) >> 5;  // 32-column blocks of window queries in use
#pragma unroll 1
        for (int blk = 0; blk < nblk; ++blk) {
          float cur[32];
          tmem_ld32_issue(taddr + blk * 32, cur);
          tmem_ld_wait(cur);
          // the MMA has already subtracted the log-sum-exp: p = exp2(scale * logit)
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float2 r = __fmul2_rn(make_float2(cur[i], cur[i + 1]), make_float2(sc2, sc2));
            cur[i] = fast_exp2(r.x);
            cur[i + 1] = fast_exp2(r.y);
          }
          if (W >= 32) {
            const float sum = tree_sum32(cur);
            const int h = (blk * 32) / W;
#pragma unroll
            for (int hh = 0; hh < NH; ++hh)
              if (hh == h) acc[hh] += sum;
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              cur[i] += cur[i + 8];
              cur[16 + i] += cur[24 + i];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              cur[i] += cur[i + 4];
              cur[16 + i] += cur[20 + i];
            }
            const float s0 = (cur[0] + cur[1]) + (cur[2] + cur[3]);
            const float s1 = (cur[16] + cur[17]) + (cur[18] + cur[19]);
#pragma unroll
            for (int hh = 0; hh < NH; hh += 2)
              if (hh == 2 * blk) {
                acc[hh] += s0;
                if (hh + 1 < NH) acc[hh + 1] += s1;
              }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&m->s2_empty[grp]));
        // lane <-> key: the tile starts pool_radius keys before the first key it owns; keys
        // outside the prefix hold the neutral element of both pools (values are >= 0)
        const int ab = (int)((n2 >> 1) & 1);
        const int i = tile * p.out_keys - rad + row;
        const bool inside = i >= 0 && i < k2.s.prefix;
        float(*abuf)[kTile] = m->a[grp][ab];
        if (avg) {
#pragma unroll
          for (int h = 0; h < NH; ++h)
            if (h < 4 && h < k2.group) abuf[h][row] = inside ? acc[h] * inv_w : 0.f;
        } else {
          // max-pooling commutes with the group maximum: reduce over the query heads first
          float top = 0.f;
#pragma unroll
          for (int h = 0; h < NH; ++h)
            if (h < k2.group) top = fmaxf(top, acc[h] * inv_w);
          abuf[0][row] = inside ? top : 0.f;
        }
        group_sync();
        if (!alive) break;
        const int own_lo = tile * p.out_keys, own_hi = min(k2.s.prefix, own_lo + p.out_keys);
        if (i >= own_lo && i < own_hi) {
          float best = 0.f;
          if (avg) {
            for (int h = 0; h < k2.group; ++h) {
              const float* a = &abuf[h][row];
              float pv = 0.f;
              for (int q = -rad; q <= rad; ++q) pv += a[q];
              best = fmaxf(best, pv / (float)g.pool_kernel);
            }
          } else {
            const float* a = &abuf[0][row];
            if (rad == 3) {
              best = fmaxf(fmaxf(fmaxf(a[-3], a[-2]), fmaxf(a[-1], a[0])),
                           fmaxf(fmaxf(a[1], a[2]), a[3]));
            } else {
              best = a[0];
              for (int q = 1; q <= rad; ++q) best = fmaxf(best, fmaxf(a[-q], a[q]));
            }
          }
          const float sc = best * chunk_scale;
          float* dst = dst_head + i;
          // split mode: the group maximum over the two halves is taken in memory (scores are
          // >= 0, so their bit patterns order like the values; the array starts as zeros)
          if (p.split) atomicMax(reinterpret_cast<unsigned*>(dst), __float_as_uint(sc));
          else *dst = sc;
          if (sc > 0.f) {
            es += sc;
            et += sc * __logf(sc);
          }
        }
        t2 += 2;
        n2 += 2;
        ord2 += 2 * sched1;
      }
    }
  } else if (warp >= 12 && warp < 12 + kVWarps) {
    // ================= value-norm warps: the V rows of the CTA's pass-1 chunks ===============
    // Row L1 norms through the register-operand tensor path: a warp takes 16 rows at a time,
    // clears the sign bits of the packed bf16 values and multiplies the 16 x 128 slab by a matrix
    // of ones (mma.sync m16n8k16, fp32 accumulate, exact products), which leaves the row sums in
    // the accumulator.  Which of a row's values lands in which k slot does not matter for a
    // sum, so every thread simply loads 16-byte pieces: thread (g, t) of a warp, g = lane / 4,
    // t = lane % 4, owns pieces t, t+4, t+8, t+12 of rows g and g+8.  Seven warps cover 112 rows
    // per step; one step is in flight while the previous one is reduced.
    if (!p.vbar_in) {
      const int vw = warp - 12;                   // 0..6
      const int gq = lane >> 2, tq = lane & 3;
      struct Group {
        const char* base;  // this thread's first 16 bytes of row 0 of the sequence
        int row0, row_hi, head;
        bool last;         // last group of its chunk
      };
      int c = blockIdx.x;
      Chunk ck;
      int grp = 0, ngrp = 0;
      auto next_group = [&](Group& gr) -> bool {
        while (grp == ngrp) {
          if (c >= total1 || m->abort_flag) return false;
          ck = decode_chunk(p, m, c, 1);
          c += gridDim.x;
          grp = 0;
          ngrp = ceil_div(min(ck.s.n, (ck.tile0 + ck.ntiles) * kTile) - ck.tile0 * kTile, 8 * kVRows);
          if (ck.half) ngrp = 0;  // the head's V rows belong to the first half's chunks
        }
        gr.base = p.v + ((size_t)ck.layer * p.v_ls + (long long)ck.kvh * g.v_sh +
                         ck.s.tok0 * g.v_st) * 2 + tq * 16;
        gr.row0 = ck.tile0 * kTile + grp * 8 * kVRows + vw * 16 + gq;
        gr.row_hi = min(ck.s.n, (ck.tile0 + ck.ntiles) * kTile);
        gr.head = ck.rhead;
        gr.last = ++grp == ngrp;
        return true;
      };
      // buf[0..3]: pieces of row g, buf[4..7]: pieces of row g + 8 (zeros beyond the chunk)
      auto issue = [&](uint4 (&buf)[8], const Group& gr) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int row = gr.row0 + half * 8;
          const char* src = gr.base + (long long)row * g.v_st * 2;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            buf[half * 4 + q] = make_uint4(0, 0, 0, 0);
            if (row < gr.row_hi) buf[half * 4 + q] = ld_stream16(src + q * 64);
          }
        }
      };
      float best = 0.f;
      const uint32_t ones = 0x3f803f80u;  // bf16 (1, 1)
      auto reduce = [&](const uint4 (&buf)[8], const Group& gr) {
        float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;  // d0: row g, d2: row g + 8
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint4 lo = buf[q], hi = buf[4 + q];
          // two k = 16 steps per pair of pieces: (x, y) and (z, w)
          mma_bf16_16816(d0, d1, d2, d3, lo.x & 0x7fff7fffu, hi.x & 0x7fff7fffu,
                         lo.y & 0x7fff7fffu, hi.y & 0x7fff7fffu, ones, ones);
          mma_bf16_16816(d0, d1, d2, d3, lo.z & 0x7fff7fffu, hi.z & 0x7fff7fffu,
                         lo.w & 0x7fff7fffu, hi.w & 0x7fff7fffu, ones, ones);
        }
        best = fmaxf(best, fmaxf(d0, d2));
        if (gr.last) {  // warp-uniform
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
          if (lane == 0) {
            atomicMax(&p.vbar_bits[gr.head], __float_as_uint(best));
            __threadfence();
            atomicAdd(&p.vcount[gr.head], 1);
          }
          best = 0.f;
        }
      };
      uint4 bufa[8], bufb[8];
      Group ga, gb;
      bool have_a = next_group(ga), have_b = false;
      if (have_a) issue(bufa, ga);
      while (have_a) {
        have_b = next_group(gb);
        if (have_b) issue(bufb, gb);
        reduce(bufa, ga);
        if (!have_b) break;
        have_a = next_group(ga);
        if (have_a) issue(bufa, ga);
        reduce(bufb, gb);
      }
    }
  }

  // ---- teardown: everything this CTA started has finished before shared memory and TMEM go --
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 2) tmem_dealloc(tmem, 512);
}

// entropy of one (layer, sequence) from the per-chunk sums, folded in a fixed order
__global__ void __launch_bounds__(256)
entropy_finalize_sm100_kernel(Geom g, const float2* ent_part, int cph2_max, int chunk_keys,
                              double* entropy, const float* vbar_in, const unsigned* vbar_bits,
                              float* vbar_out) {
  __shared__ double rs[8], rt[8];
  const int prob = blockIdx.x, layer = prob / g.batch, b = prob - layer * g.batch;
  const SeqInfo s = seq_info(g, b);
  const int used = ceil_div(s.prefix, chunk_keys);
  const int total = g.n_kv_heads * used;
  if (vbar_out && (int)threadIdx.x < g.n_kv_heads) {
    const size_t head = (size_t)prob * g.n_kv_heads + threadIdx.x;
    vbar_out[head] = vbar_in ? vbar_in[head] : __uint_as_float(vbar_bits[head]);
  }
  double sum_s = 0.0, sum_t = 0.0;
  for (int i = threadIdx.x; i < total; i += 256) {
    const int kvh = i / used, t = i - kvh * used;
    const float2* e = ent_part + (((size_t)prob * g.n_kv_heads + kvh) * cph2_max + t) * 8;
    double cs = 0.0, ct = 0.0;  // the eight consumer warps of the chunk, in order
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      cs += (double)e[u].x;
      ct += (double)e[u].y;
    }
    sum_s += cs;
    sum_t += ct;
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

// Split mode: the scores of a KV head are complete only after both halves of its query group
// have been merged in memory, so the entropy of one (layer, sequence) is summed from the final
// score array here (fixed order: thread-strided fp32 sums of at most a few hundred terms, then
// fp64 across lanes and warps).  Also hands out the value norms.
__global__ void __launch_bounds__(1024)
entropy_from_scores_kernel(Geom g, const float* scores, double* entropy, const float* vbar_in,
                           const unsigned* vbar_bits, float* vbar_out) {
  __shared__ double rs[32], rt[32];
  const int prob = blockIdx.x, layer = prob / g.batch, b = prob - layer * g.batch;
  if (batch_has_short_sequence(g)) return;
  const SeqInfo s = seq_info(g, b);
  if (vbar_out && (int)threadIdx.x < g.n_kv_heads) {
    const size_t head = (size_t)prob * g.n_kv_heads + threadIdx.x;
    vbar_out[head] = vbar_in ? vbar_in[head] : __uint_as_float(vbar_bits[head]);
  }
  const float* sc = scores + (size_t)layer * g.total_scores + s.score_off;
  const long long count = (long long)g.n_kv_heads * s.prefix;
  double sum_s = 0.0, sum_t = 0.0;
  for (long long i0 = threadIdx.x; i0 < count; i0 += 1024 * 256) {
    float es = 0.f, et = 0.f;  // at most 256 terms in fp32, then fp64
    for (long long i = i0; i < count && i < i0 + 1024LL * 256; i += 1024) {
      const float v = sc[i];
      if (v > 0.f) {
        es += v;
        et += v * __logf(v);
      }
    }
    sum_s += (double)es;
    sum_t += (double)et;
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
    for (int i = 0; i < 32; ++i) {
      a += rs[i];
      c += rt[i];
    }
    double e = 0.0;
    if (a > 0.0) e = (log(a) - c / a) / ((double)g.n_kv_heads * (double)s.n);
    entropy[(size_t)layer * g.batch + b] = e;
  }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) ==
            cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

size_t up256(size_t x) { return (x + 255) / 256 * 256; }

// Tiles per chunk.  A chunk boundary costs a reload of the head's query tile and a hand-over
// of statistics, so chunks should be long; but the launch needs many more chunks than CTAs to
// balance (chunks are dealt round-robin), and a head finishes pass 1 sooner when more CTAs
// share it.  Default: about twelve chunks per CTA, between 4 and 32 tiles.  LAVA_SM100_CHUNK_TILES
// overrides it (option "score_chunk_tiles").
constexpr int kMinChunkTiles = 4, kMaxChunkTiles = 64;
constexpr int kSmallLaunchChunkTiles = 8;  // floor of the chosen length: shorter chunks cost more in boundaries than they balance

// Query groups of more than 128 window-query rows are scored as two halves (each a unit of its
// own with at most 128 rows); returns the number of query heads in the first half, 0 if the
// group fits one unit.
int sm100_first_half(const Geom& g) {
  return g.group * g.window > 128 ? (g.group + 1) / 2 : 0;
}
int chunk_tiles_for(const Geom& g, int n_layers) {
  if (options().score_chunk_tiles > 0) return options().score_chunk_tiles;
  const long long tiles = (long long)n_layers * (g.n_kv_heads << (sm100_first_half(g) ? 1 : 0)) *
                          ceil_div((int)g.total_tokens, kTile);
  const int sms = sm_count() > 0 ? sm_count() : 148;  // without a device: the part this is tuned for
  // at least four chunks per CTA, and at least three chunks in a sequence of average length (a
  // batch of short sequences would otherwise be dealt in a few unequal pieces)
  long long r = tiles / ((long long)sms * 4);
  const long long mean_tiles = ceil_div((int)(g.total_tokens / g.batch), kTile);
  if (r > mean_tiles / 3) r = mean_tiles / 3;
  if (r < kSmallLaunchChunkTiles) r = mean_tiles < kSmallLaunchChunkTiles ? mean_tiles : kSmallLaunchChunkTiles;
  return (int)(r < kMinChunkTiles ? kMinChunkTiles : r > kMaxChunkTiles ? kMaxChunkTiles : r);
}

// Tiles pass 1 leads pass 2 by beyond what head completion needs (covers the time a head's
// statistics take to be published and folded, and the skew between CTAs): half a chunk.
// LAVA_SM100_LEAD_TILES overrides it.
int lead_extra_for(int chunk_tiles) {
  const int forced = options().score_lead_tiles;
  return forced >= 0 ? forced : (chunk_tiles + 1) / 2;
}

}  // namespace

lava_status launch_entropy_from_scores(const Geom& g, int n_layers, const float* scores,
                                       double* entropy, cudaStream_t stream) {
  entropy_from_scores_kernel<<<n_layers * g.batch, 1024, 0, stream>>>(g, scores, entropy, nullptr,
                                                                      nullptr, nullptr);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "entropy launch");
}

bool sm100_supported(const Geom& g) {
  if (g.dtype != LAVA_BF16 || g.head_dim != 128) return false;
  if (g.window != 16 && g.window != 32 && g.window != 64 && g.window != 128) return false;
  // heads of one scored unit: the whole query group, or its larger half when the group has more
  // than 128 window-query rows
  const int unit = g.group * g.window > 128 ? (g.group + 1) / 2 : g.group;
  if (unit * g.window > 128 || unit > 8) return false;
  if (g.pool_kind == LAVA_POOL_AVG && unit > 4) return false;  // room for 4 heads' window means
  if (g.pool_radius > 31) return false;
  if (g.batch > kMaxBatch) return false;
  return true;
}

Sm100Layout sm100_layout(const Geom& g, int n_layers) {
  Sm100Layout l;
  const int r = chunk_tiles_for(g, n_layers);
  l.chunk_tiles = r;
  l.heads_total = n_layers * g.batch * (g.n_kv_heads << (sm100_first_half(g) ? 1 : 0));  // units
  l.out_keys = kTile - 2 * g.pool_radius;
  const int tiles1 = ceil_div(g.max_seqlen, kTile);
  const int tiles2 = ceil_div(max(1, g.max_seqlen - g.window), l.out_keys);
  l.chunks1 = ceil_div(tiles1, r);  // chunks per head, pass 1
  l.chunks2 = ceil_div(tiles2, r);  // chunks per head, pass 2
  size_t off = 0;
  l.off_sync = off;   // chunk counters, value-norm counters and bits: zeroed every launch
  off = up256(off + sizeof(int) * 3 * (size_t)l.heads_total);
  l.sync_bytes = off;
  l.off_part = off;
  off = up256(off + sizeof(float) * 128 * (size_t)l.heads_total * l.chunks1);
  l.off_ent = off;
  off = up256(off + sizeof(float2) * 8 * (size_t)l.heads_total * l.chunks2);
  // The size asked of the caller does not depend on the chunk length chosen for this launch
  // (a workspace sized for a whole model also serves calls on fewer layers): it is the size
  // at the shortest chunk.
  const int rmin = r < kMinChunkTiles ? r : kMinChunkTiles;
  size_t cap = up256(sizeof(int) * 3 * (size_t)l.heads_total);
  cap = up256(cap + sizeof(float) * 128 * (size_t)l.heads_total * ceil_div(tiles1, rmin));
  cap = up256(cap + sizeof(float2) * 8 * (size_t)l.heads_total * ceil_div(tiles2, rmin));
  l.total = cap > off ? cap : off;
  return l;
}

lava_status encode_score_maps(const Geom& g, int n_layers, const void* q, const void* k,
                              long long q_ls, long long k_ls, CUtensorMap* map_q_out,
                              CUtensorMap* map_k_out) {
  EncodeTiledFn encode = encode_fn();
  if (!encode) return fail(LAVA_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
  CUtensorMap& map_q = *map_q_out;
  CUtensorMap& map_k = *map_k_out;
  // Q: [layer][batch*H_q*w rows][128]; K: [layer][H_kv][tokens][128]; boxes of 64 x 128 elements
  {
    const cuuint64_t rows = (cuuint64_t)g.batch * g.n_q_heads * g.window;
    const cuuint64_t dims[3] = {128, rows, (cuuint64_t)n_layers};
    const cuuint64_t ls = n_layers > 1 ? (cuuint64_t)q_ls * 2 : rows * 256;
    const cuuint64_t strides[2] = {256, ls};
    const cuuint32_t box[3] = {64, 128, 1}, es[3] = {1, 1, 1};
    if (encode(&map_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box,
               es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return fail(LAVA_ERR_CUDA, "tensor map for the query window could not be encoded");
  }
  {
    const cuuint64_t dims[4] = {128, (cuuint64_t)g.total_tokens, (cuuint64_t)g.n_kv_heads,
                                (cuuint64_t)n_layers};
    const cuuint64_t hs = (cuuint64_t)g.k_sh * 2;
    const cuuint64_t ls = n_layers > 1 ? (cuuint64_t)k_ls * 2
                                       : (cuuint64_t)g.k_sh * 2 * (cuuint64_t)g.n_kv_heads;
    const cuuint64_t strides[3] = {(cuuint64_t)g.k_st * 2, hs > 0 ? hs : 256, ls > 0 ? ls : 256};
    const cuuint32_t box[4] = {64, 128, 1, 1}, es[4] = {1, 1, 1, 1};
    if (encode(&map_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(k), dims, strides, box,
               es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return fail(LAVA_ERR_CUDA, "tensor map for K could not be encoded");
  }

  return LAVA_OK;
}

lava_status launch_score_sm100(const Geom& g, int n_layers, const void* q, const void* k,
                               const void* v, long long q_ls, long long k_ls, long long v_ls,
                               const float* vbar_in, float* scores, float* vbar_out,
                               double* entropy, char* ws_base, size_t ws_off, cudaStream_t stream) {
  char* ws = ws_base + ws_off;
  const Sm100Layout lay = sm100_layout(g, n_layers);

  CUtensorMap map_q, map_k;
  {
    const lava_status mrc = encode_score_maps(g, n_layers, q, k, q_ls, k_ls, &map_q, &map_k);
    if (mrc != LAVA_OK) return mrc;
  }

  const int sms = sm_count();
  if (sms <= 0) return fail(LAVA_ERR_CUDA, "the multiprocessor count of the device is not available");
  lava_status rc = LAVA_OK;

  Sm100Params p;
  p.g = g;
  p.n_layers = n_layers;
  p.chunk_tiles = lay.chunk_tiles;
  p.out_keys = lay.out_keys;
  p.cph1_max = lay.chunks1;
  p.cph2_max = lay.chunks2;
  p.lead_extra = lead_extra_for(lay.chunk_tiles);
  p.g0 = sm100_first_half(g);
  p.split = p.g0 ? 1 : 0;
  p.wait_cycles = options().wait_limit_cycles;
  p.vbar_in = vbar_in;
  p.scores = scores;
  p.vbar_out = vbar_out;
  p.v = (const char*)v;
  p.v_ls = v_ls;
  p.counters = reinterpret_cast<int*>(ws + lay.off_sync);
  p.vcount = p.counters + lay.heads_total;
  p.vbar_bits = reinterpret_cast<unsigned*>(p.vcount + lay.heads_total);
  p.part = reinterpret_cast<float*>(ws + lay.off_part);
  p.ent_part = reinterpret_cast<float2*>(ws + lay.off_ent);
  p.status = reinterpret_cast<unsigned*>(ws_base);  // the status word opens the workspace

  rc = check_cuda(cudaMemsetAsync(ws + lay.off_sync, 0, lay.sync_bytes, stream),
                  "sync scratch clear");
  if (rc != LAVA_OK) return rc;
  if (p.split) {  // the two halves of a query group meet in memory through a maximum
    rc = check_cuda(cudaMemsetAsync(scores, 0, sizeof(float) * (size_t)n_layers * g.total_scores,
                                    stream), "score clear");
    if (rc != LAVA_OK) return rc;
  }

  void (*kern)(const CUtensorMap, const CUtensorMap, const Sm100Params) = nullptr;
  switch (g.window) {
    case 16: kern = lava_score_sm100_kernel<16>; break;
    case 32: kern = lava_score_sm100_kernel<32>; break;
    case 64: kern = lava_score_sm100_kernel<64>; break;
    default: kern = lava_score_sm100_kernel<128>; break;
  }
  rc = check_cuda(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kSmemBytes), "cudaFuncSetAttribute(sm100 score)");
  if (rc != LAVA_OK) return rc;
  // an upper bound on the pass-1 chunks; CTAs beyond the real count find no work and exit
  const long long chunks = (long long)lay.heads_total * lay.chunks1;
  if ((long long)lay.heads_total * (lay.chunks2 > lay.chunks1 ? lay.chunks2 : lay.chunks1) > 0x3fffffffLL)
    return fail(LAVA_ERR_UNSUPPORTED, "too many chunks for the 32-bit chunk index");
  const int grid = (int)(chunks < sms ? chunks : sms);
  // Cooperative launch: the CTAs wait on one another's flags, so all must be resident at once.
  void* args[3] = {&map_q, &map_k, &p};
  rc = check_cuda(cudaLaunchCooperativeKernel((const void*)kern, dim3(grid), dim3(kThreads), args,
                                              kSmemBytes, stream), "score (sm100) launch");
  if (rc != LAVA_OK) return rc;
  if (p.split)
    entropy_from_scores_kernel<<<n_layers * g.batch, 1024, 0, stream>>>(g, scores, entropy, vbar_in,
                                                                        p.vbar_bits, vbar_out);
  else
    entropy_finalize_sm100_kernel<<<n_layers * g.batch, 256, 0, stream>>>(
        g, p.ent_part, lay.chunks2, p.chunk_tiles * lay.out_keys, entropy, vbar_in, p.vbar_bits,
        vbar_out);
  count_launches(2);
  return check_cuda(cudaGetLastError(), "entropy finalize launch");
}

}  // namespace lava
