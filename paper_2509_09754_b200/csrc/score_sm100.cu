// LAVa score, Blackwell path: bf16, head_dim 128, G*w <= 128, w in {16, 32, 64, 128}.
//
// One persistent, warp-specialised kernel (one CTA per SM) runs two pipelines over 128-key
// tiles of K, both fed by TMA into 128B-swizzled shared memory and contracted with tcgen05.mma
// into TMEM:
//
//   pass 1 (statistics)  S = Q_g K^T  (rows = the group's G*w window queries, columns = keys)
//       one thread per row reads its TMEM lane: masked row max and sum of exp2 over the keys
//       the query may see (Sec. 2: softmax over i <= j), published per (head, tile); four more
//       warps stream the matching V rows for the value norm (Theorem 1: max_k ||V[k]||_1).
//       The CTA that publishes the last tile of a head folds the partials into one
//       log-sum-exp per query and raises the head's ready flag.
//   pass 2 (scores)      S^T = K Q_g^T (rows = keys, columns = window queries)
//       one thread per key: a_h[i] = (1/w) sum_t exp2(z - lse_t) per query head in registers,
//       pooled over the token axis through shared memory, scaled by Vbar * c_hat, reduced with
//       the GQA group maximum, written once; per-tile entropy sums go to ordered slots
//       (Definition 1, Sec. 4.2, Sec. 4.3, Sec. 5.1 pooling).
//
// K is read from HBM once: pass 2 trails pass 1 by a bounded number of heads, so its tiles are
// still in L2.  Every wait (mbarrier, ready flag) is bounded; on expiry the kernel sets
// LAVA_DEV_WAIT_EXPIRED, drains its copies, frees TMEM and returns.
#include <cuda.h>

#include "lava_internal.cuh"

namespace lava {
namespace {

constexpr int kTile = 128;           // keys per tile
constexpr int kThreads = 512;        // 16 warps
constexpr int kStages = 2;           // K stages per pipeline
constexpr uint32_t kTileBytes = 128 * 128 * 2;  // one [128 x 128] bf16 tile = 2 swizzled blocks
constexpr uint32_t kHalfBytes = kTileBytes / 2;
constexpr uint32_t kSpinLimit = 1u << 22;

// shared memory map (bytes from a 1024-aligned base)
constexpr uint32_t kOffQ1 = 0;
constexpr uint32_t kOffQ2 = kOffQ1 + kTileBytes;
constexpr uint32_t kOffK1 = kOffQ2 + kTileBytes;
constexpr uint32_t kOffK2 = kOffK1 + kStages * kTileBytes;
constexpr uint32_t kOffMisc = kOffK2 + kStages * kTileBytes;  // 192 KB
constexpr uint32_t kMiscBytes = 12288;
constexpr uint32_t kSmemBytes = kOffMisc + kMiscBytes + 1024;  // + alignment slack

struct Misc {
  unsigned long long k1_full[kStages], k1_empty[kStages], k2_full[kStages], k2_empty[kStages];
  unsigned long long q1_full, q1_empty, q2_full, q2_empty;
  unsigned long long s1_full[2], s1_empty[2], s2_full[2], s2_empty[2];
  unsigned long long drain;
  uint32_t tmem_base;
  volatile int abort_flag;
  volatile int p2_head;     // head (linear index) the score warps are working on
  int last_flag;
  alignas(16) float lse[128];  // -(log2-sum-exp) of the current pass-2 head, per window query
  alignas(16) float a[2][8][kTile];  // window-mean attention per (query head, key) of the current tile
  float red[2][4];
  float vmax[4];
};
static_assert(sizeof(Misc) <= kMiscBytes, "misc region too small");

struct Sm100Params {
  Geom g;
  int n_layers;
  int heads_total;          // n_layers * batch * H_kv
  int tiles1_per_head;      // ceil(max_seqlen / 128)
  int tiles2_per_head;      // ceil(max_prefix / out_keys)
  int out_keys;             // keys a pass-2 tile owns: 128 - 2 * pool_radius
  int lag_heads;            // pass 1 may run this many heads ahead of pass 2
  const float* vbar_in;
  float* scores;
  float* vbar_out;
  const char* v;
  long long v_ls;
  // scratch
  float2* part;             // [heads_total][tiles1_per_head][128]
  int* counters;            // [heads_total]
  int* ready;               // [heads_total]
  unsigned* vbar_bits;      // [heads_total]
  float* neg_lse;           // [heads_total][128]
  double2* ent_part;        // [heads_total][tiles2_per_head]
  unsigned* status;
};

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ inline uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ inline void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ inline void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ inline void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ inline bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ inline void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2,
                                   uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ inline void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2,
                                   int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ inline void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem),
               "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ inline void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ inline void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ inline void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ inline void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, M = N = 128, K = 16
__device__ inline void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                 uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ inline void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ inline void named_barrier(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
// Barrier that also ORs a predicate over the participants: every thread gets the same answer,
// so "stop now" decisions taken after it are uniform.
__device__ inline bool named_barrier_or(int id, int count, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n.reg .pred p, q;\nsetp.ne.b32 q, %3, 0;\nbar.red.or.pred p, %1, %2, q;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(r)
      : "r"(id), "r"(count), "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}
__device__ inline float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ inline int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ inline void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 B apart.
__device__ inline uint64_t make_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;            // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;  // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;            // descriptor version of this architecture
  d |= (uint64_t)2 << 61;            // 128-byte swizzle
  return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

// Bounded mbarrier wait.  Returns false once the CTA is aborting (unless heed_abort is false:
// the drain waits at exit must outlast an abort to let copies in flight land).
__device__ inline bool wait_bar(uint32_t bar, uint32_t parity, Misc* m, unsigned* status,
                                bool heed_abort = true) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_test(bar, parity)) return true;
    if (it > 128) {
      if (heed_abort && m->abort_flag) return false;
      __nanosleep(64);
    }
  }
  m->abort_flag = 1;
  atomicOr(status, LAVA_DEV_WAIT_EXPIRED);
  return false;
}

// ------------------------------------------------------------------------------------------
// item decoding (identical in every role, so no descriptors travel between warps)
// ------------------------------------------------------------------------------------------
struct Item {
  int head;    // linear head index = (layer * batch + b) * H_kv + kvh
  int layer, b, kvh, tile;
  SeqInfo s;
  bool valid;
};

__device__ inline Item decode(const Sm100Params& p, long long idx, int tiles_per_head, int pass) {
  Item it;
  it.head = (int)(idx / tiles_per_head);
  it.tile = (int)(idx - (long long)it.head * tiles_per_head);
  const int prob = it.head / p.g.n_kv_heads;
  it.kvh = it.head - prob * p.g.n_kv_heads;
  it.layer = prob / p.g.batch;
  it.b = prob - it.layer * p.g.batch;
  it.s = seq_info(p.g, it.b);
  if (pass == 1) it.valid = (long long)it.tile * kTile < it.s.n;
  else it.valid = (long long)it.tile * p.out_keys < it.s.prefix;
  return it;
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
  const int rows_valid = g.group * W;
  const long long items1 = (long long)p.heads_total * p.tiles1_per_head;
  const long long items2 = (long long)p.heads_total * p.tiles2_per_head;

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
      mbar_init(smem_u32(&m->s1_empty[s]), 128);
      mbar_init(smem_u32(&m->s2_full[s]), 1);
      mbar_init(smem_u32(&m->s2_empty[s]), 128);
    }
    mbar_init(smem_u32(&m->drain), 1);
    m->abort_flag = 0;
    m->p2_head = 0;
    m->last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2) tmem_alloc(smem_u32(&m->tmem_base), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = m->tmem_base;

  if (warp == 0) {
    // ================= pass-1 producer: Q of the head, K tiles =============================
    if (lane == 0) {
      int prev_head = -1, q_loads = 0;
      long long n = 0;  // loads issued
      for (long long idx = blockIdx.x; idx < items1; idx += gridDim.x) {
        const Item it = decode(p, idx, p.tiles1_per_head, 1);
        if (!it.valid) continue;
        // stay within lag_heads of the score warps so pass 2 still finds its tiles in L2
        {
          uint32_t spins = 0;
          while (it.head > m->p2_head + p.lag_heads) {
            if (m->abort_flag) break;
            __nanosleep(128);
            if (++spins > kSpinLimit) {
              m->abort_flag = 1;
              atomicOr(p.status, LAVA_DEV_WAIT_EXPIRED);
              break;
            }
          }
          if (m->abort_flag) break;
        }
        if (it.head != prev_head) {
          if (!wait_bar(smem_u32(&m->q1_empty), (q_loads & 1) ^ 1, m, p.status)) break;
          const uint32_t bar = smem_u32(&m->q1_full);
          mbar_expect_tx(bar, kTileBytes);
          const int row0 = (it.b * g.n_q_heads + it.kvh * g.group) * W;
          tma_load_3d(base + kOffQ1, &map_q, 0, row0, it.layer, bar);
          tma_load_3d(base + kOffQ1 + kHalfBytes, &map_q, 64, row0, it.layer, bar);
          prev_head = it.head;
          ++q_loads;
        }
        const int st = (int)(n % kStages);
        if (!wait_bar(smem_u32(&m->k1_empty[st]), (uint32_t)((n / kStages) & 1) ^ 1, m, p.status))
          break;
        const uint32_t bar = smem_u32(&m->k1_full[st]);
        mbar_expect_tx(bar, kTileBytes);
        const int tok = (int)it.s.tok0 + it.tile * kTile;
        tma_load_4d(base + kOffK1 + st * kTileBytes, &map_k, 0, tok, it.kvh, it.layer, bar);
        tma_load_4d(base + kOffK1 + st * kTileBytes + kHalfBytes, &map_k, 64, tok, it.kvh, it.layer,
                    bar);
        ++n;
      }
      // copies still in flight land before this CTA gives up its shared memory
      for (long long j = (n > kStages ? n - kStages : 0); j < n; ++j)
        wait_bar(smem_u32(&m->k1_full[j % kStages]), (uint32_t)((j / kStages) & 1), m, p.status,
                 false);
      if (q_loads > 0)
        wait_bar(smem_u32(&m->q1_full), (uint32_t)((q_loads - 1) & 1), m, p.status, false);
    }
  } else if (warp == 1) {
    // ================= pass-2 producer ======================================================
    if (lane == 0) {
      int prev_head = -1, q_loads = 0;
      long long n = 0;
      for (long long idx = blockIdx.x; idx < items2; idx += gridDim.x) {
        const Item it = decode(p, idx, p.tiles2_per_head, 2);
        if (!it.valid) continue;
        if (it.head != prev_head) {
          if (!wait_bar(smem_u32(&m->q2_empty), (q_loads & 1) ^ 1, m, p.status)) break;
          const uint32_t bar = smem_u32(&m->q2_full);
          mbar_expect_tx(bar, kTileBytes);
          const int row0 = (it.b * g.n_q_heads + it.kvh * g.group) * W;
          tma_load_3d(base + kOffQ2, &map_q, 0, row0, it.layer, bar);
          tma_load_3d(base + kOffQ2 + kHalfBytes, &map_q, 64, row0, it.layer, bar);
          prev_head = it.head;
          ++q_loads;
        }
        const int st = (int)(n % kStages);
        if (!wait_bar(smem_u32(&m->k2_empty[st]), (uint32_t)((n / kStages) & 1) ^ 1, m, p.status))
          break;
        const uint32_t bar = smem_u32(&m->k2_full[st]);
        mbar_expect_tx(bar, kTileBytes);
        // the tile starts pool_radius keys before the first key it owns (halo for pooling)
        const int tok = (int)it.s.tok0 + it.tile * p.out_keys - g.pool_radius;
        tma_load_4d(base + kOffK2 + st * kTileBytes, &map_k, 0, tok, it.kvh, it.layer, bar);
        tma_load_4d(base + kOffK2 + st * kTileBytes + kHalfBytes, &map_k, 64, tok, it.kvh, it.layer,
                    bar);
        ++n;
      }
      for (long long j = (n > kStages ? n - kStages : 0); j < n; ++j)
        wait_bar(smem_u32(&m->k2_full[j % kStages]), (uint32_t)((j / kStages) & 1), m, p.status,
                 false);
      if (q_loads > 0)
        wait_bar(smem_u32(&m->q2_full), (uint32_t)((q_loads - 1) & 1), m, p.status, false);
    }
  } else if (warp == 2) {
    // ================= MMA issuer: serves both pipelines by polling =========================
    if (lane == 0) {
      long long idx1 = blockIdx.x, idx2 = blockIdx.x;
      long long n1 = 0, n2 = 0;
      int prev1 = -1, prev2 = -1, q1_uses = 0, q2_uses = 0;
      uint32_t idle = 0;
      // skip leading empty items
      while (idx1 < items1 && !decode(p, idx1, p.tiles1_per_head, 1).valid) idx1 += gridDim.x;
      while (idx2 < items2 && !decode(p, idx2, p.tiles2_per_head, 2).valid) idx2 += gridDim.x;
      while (idx1 < items1 || idx2 < items2) {
        bool progressed = false;
        if (idx1 < items1) {
          const Item it = decode(p, idx1, p.tiles1_per_head, 1);
          const int st = (int)(n1 % kStages), buf = (int)(n1 & 1);
          const bool need_q = it.head != prev1;
          if (mbar_test(smem_u32(&m->k1_full[st]), (uint32_t)((n1 / kStages) & 1)) &&
              mbar_test(smem_u32(&m->s1_empty[buf]), (uint32_t)((n1 >> 1) & 1) ^ 1) &&
              (!need_q || mbar_test(smem_u32(&m->q1_full), (uint32_t)(q1_uses & 1)))) {
            if (need_q) {
              prev1 = it.head;
              ++q1_uses;
            }
            tc_fence_after();
            const uint32_t d = tmem + (uint32_t)buf * 128u;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const uint32_t off = (uint32_t)(kk >> 2) * kHalfBytes + (uint32_t)(kk & 3) * 32u;
              umma_bf16(d, make_desc(base + kOffQ1 + off),
                        make_desc(base + kOffK1 + st * kTileBytes + off), kIdesc, kk > 0);
            }
            umma_commit(smem_u32(&m->k1_empty[st]));
            umma_commit(smem_u32(&m->s1_full[buf]));
            ++n1;
            idx1 += gridDim.x;
            while (idx1 < items1 && !decode(p, idx1, p.tiles1_per_head, 1).valid) idx1 += gridDim.x;
            // the query tile may be replaced once the MMAs of its last user have completed
            if (idx1 >= items1 || decode(p, idx1, p.tiles1_per_head, 1).head != prev1)
              umma_commit(smem_u32(&m->q1_empty));
            progressed = true;
          }
        }
        if (idx2 < items2) {
          const Item it = decode(p, idx2, p.tiles2_per_head, 2);
          const int st = (int)(n2 % kStages), buf = (int)(n2 & 1);
          const bool need_q = it.head != prev2;
          if (mbar_test(smem_u32(&m->k2_full[st]), (uint32_t)((n2 / kStages) & 1)) &&
              mbar_test(smem_u32(&m->s2_empty[buf]), (uint32_t)((n2 >> 1) & 1) ^ 1) &&
              (!need_q || mbar_test(smem_u32(&m->q2_full), (uint32_t)(q2_uses & 1)))) {
            if (need_q) {
              prev2 = it.head;
              ++q2_uses;
            }
            tc_fence_after();
            const uint32_t d = tmem + 256u + (uint32_t)buf * 128u;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const uint32_t off = (uint32_t)(kk >> 2) * kHalfBytes + (uint32_t)(kk & 3) * 32u;
              umma_bf16(d, make_desc(base + kOffK2 + st * kTileBytes + off),
                        make_desc(base + kOffQ2 + off), kIdesc, kk > 0);
            }
            umma_commit(smem_u32(&m->k2_empty[st]));
            umma_commit(smem_u32(&m->s2_full[buf]));
            ++n2;
            idx2 += gridDim.x;
            while (idx2 < items2 && !decode(p, idx2, p.tiles2_per_head, 2).valid) idx2 += gridDim.x;
            if (idx2 >= items2 || decode(p, idx2, p.tiles2_per_head, 2).head != prev2)
              umma_commit(smem_u32(&m->q2_empty));
            progressed = true;
          }
        }
        if (progressed) {
          idle = 0;
        } else {
          if (++idle > 256) {
            if (m->abort_flag) break;
            __nanosleep(32);
            if (idle > kSpinLimit) {
              m->abort_flag = 1;
              atomicOr(p.status, LAVA_DEV_WAIT_EXPIRED);
              break;
            }
          }
        }
      }
      // every MMA has completed before TMEM is released
      umma_commit(smem_u32(&m->drain));
      wait_bar(smem_u32(&m->drain), 0, m, p.status, false);
    }
  } else if (warp >= 4 && warp < 8) {
    // ================= pass-1 consumers: one thread per (query head, window query) row ======
    const int quad = warp & 3, row = quad * 32 + lane, tid = row;
    const int t_in_win = row % W;
    long long n = 0;
    for (long long idx = blockIdx.x; idx < items1; idx += gridDim.x) {
      const Item it = decode(p, idx, p.tiles1_per_head, 1);
      if (!it.valid) continue;
      const int buf = (int)(n & 1);
      const bool ok = __all_sync(
          0xffffffffu, wait_bar(smem_u32(&m->s1_full[buf]), (uint32_t)((n >> 1) & 1), m, p.status));
      tc_fence_after();
      // keys this query may see inside the tile: i < n and i <= P + t
      int limit = 0;
      if (row < rows_valid) {
        const int last = min(it.s.n, it.s.prefix + t_in_win + 1);
        limit = max(0, min(kTile, last - it.tile * kTile));
      }
      float mx = -INFINITY, z = 0.f;
      if (ok) {  // warp-uniform: the TMEM loads below are executed by whole warps
        const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)buf * 128u;
        float v[32];
#pragma unroll 1
        for (int c0 = 0; c0 < kTile; c0 += 32) {
          tmem_ld32(taddr + c0, v);
          if (c0 + 32 <= limit) {
#pragma unroll
            for (int c = 0; c < 32; ++c) mx = fmaxf(mx, v[c]);
          } else {
#pragma unroll
            for (int c = 0; c < 32; ++c)
              if (c0 + c < limit) mx = fmaxf(mx, v[c]);
          }
        }
        const float m2 = mx * g.scale_log2;
#pragma unroll 1
        for (int c0 = 0; c0 < kTile; c0 += 32) {
          tmem_ld32(taddr + c0, v);
          if (c0 + 32 <= limit) {
#pragma unroll
            for (int c = 0; c < 32; ++c) z += fast_exp2(fmaf(v[c], g.scale_log2, -m2));
          } else {
#pragma unroll
            for (int c = 0; c < 32; ++c)
              if (c0 + c < limit) z += fast_exp2(fmaf(v[c], g.scale_log2, -m2));
          }
        }
        mx = m2;
      }
      tc_fence_before();
      mbar_arrive(smem_u32(&m->s1_empty[buf]));
      ++n;
      p.part[((size_t)it.head * p.tiles1_per_head + it.tile) * 128 + row] = make_float2(mx, z);
      __threadfence();
      // the value-norm warps have pushed this tile's row norms before the head counter moves
      if (named_barrier_or(3, 256, m->abort_flag != 0)) break;
      const int expected = ceil_div(it.s.n, kTile);
      if (tid == 0) {
        const int old = atomicAdd(&p.counters[it.head], 1);
        m->last_flag = (old == expected - 1);
      }
      named_barrier(1, 128);
      const bool last = m->last_flag != 0;
      named_barrier(1, 128);
      if (last) {
        __threadfence();
        // fold the per-tile partials of this head into one log-sum-exp per window query
        const float2* pp = p.part + (size_t)it.head * p.tiles1_per_head * 128 + row;
        float big = -INFINITY, sum = 0.f;
#pragma unroll 4
        for (int j = 0; j < expected; ++j) {
          const float2 pr = __ldcg(pp + (size_t)j * 128);
          if (pr.y > 0.f) {
            if (pr.x > big) {
              sum = sum * fast_exp2(big - pr.x) + pr.y;
              big = pr.x;
            } else {
              sum += pr.y * fast_exp2(pr.x - big);
            }
          }
        }
        p.neg_lse[(size_t)it.head * 128 + row] = sum > 0.f ? -(big + log2f(sum)) : -INFINITY;
        __threadfence();
        named_barrier(1, 128);
        if (tid == 0) st_release(&p.ready[it.head], 1);
      }
    }
  } else if (warp >= 8 && warp < 12) {
    // ================= pass-2 consumers: one thread per key ==================================
    constexpr int NH = 128 / W;  // query heads that fit the 128 columns
    const int quad = warp & 3, key_lane = quad * 32 + lane, tid = key_lane;
    const int rad = g.pool_radius;
    const float inv_w = 1.0f / (float)W;
    int cur_head = -1;
    float head_scale = 0.f;
    long long n = 0;
    for (long long idx = blockIdx.x; idx < items2; idx += gridDim.x) {
      const Item it = decode(p, idx, p.tiles2_per_head, 2);
      if (!it.valid) continue;
      if (it.head != cur_head) {
        if (tid == 0) {
          m->p2_head = it.head;
          uint32_t spins = 0;
          while (ld_acquire(&p.ready[it.head]) == 0) {
            if (m->abort_flag) break;
            __nanosleep(64);
            if (++spins > kSpinLimit) {
              m->abort_flag = 1;
              atomicOr(p.status, LAVA_DEV_WAIT_EXPIRED);
              break;
            }
          }
        }
        if (named_barrier_or(2, 128, m->abort_flag != 0)) break;
        m->lse[tid] = __ldcg(p.neg_lse + (size_t)it.head * 128 + tid);
        const float vb = p.vbar_in ? p.vbar_in[it.head]
                                   : __uint_as_float(__ldcg(p.vbar_bits + it.head));
        head_scale = vb * g.c_hat;
        if (tid == 0 && p.vbar_out) p.vbar_out[it.head] = vb;
        cur_head = it.head;
        named_barrier(2, 128);
      }
      const int buf = (int)(n & 1);
      const bool ok = __all_sync(
          0xffffffffu, wait_bar(smem_u32(&m->s2_full[buf]), (uint32_t)((n >> 1) & 1), m, p.status));
      tc_fence_after();
      float acc[NH];
#pragma unroll
      for (int h = 0; h < NH; ++h) acc[h] = 0.f;
      if (ok) {
        const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + 256u + (uint32_t)buf * 128u;
        float v[32];
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 32) {
          if (c0 < rows_valid) {
            tmem_ld32(taddr + c0, v);
#pragma unroll
            for (int c4 = 0; c4 < 32; c4 += 4) {
              const float4 l4 = *reinterpret_cast<const float4*>(&m->lse[c0 + c4]);
              acc[(c0 + c4 + 0) / W] += fast_exp2(fmaf(v[c4 + 0], g.scale_log2, l4.x));
              acc[(c0 + c4 + 1) / W] += fast_exp2(fmaf(v[c4 + 1], g.scale_log2, l4.y));
              acc[(c0 + c4 + 2) / W] += fast_exp2(fmaf(v[c4 + 2], g.scale_log2, l4.z));
              acc[(c0 + c4 + 3) / W] += fast_exp2(fmaf(v[c4 + 3], g.scale_log2, l4.w));
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(smem_u32(&m->s2_empty[buf]));
      const int ab = (int)(n & 1);
      ++n;
#pragma unroll
      for (int h = 0; h < NH; ++h) m->a[ab][h][key_lane] = acc[h] * inv_w;
      if (named_barrier_or(2, 128, m->abort_flag != 0)) break;
      // lane <-> key: the tile starts pool_radius keys before the first key it owns
      const int key0 = it.tile * p.out_keys - rad;
      const int i = key0 + key_lane;
      const int own_lo = it.tile * p.out_keys, own_hi = min(it.s.prefix, own_lo + p.out_keys);
      float sc = 0.f;
      const bool mine = i >= own_lo && i < own_hi;
      if (mine) {
        const int lo = max(0, i - rad) - key0, hi = min(it.s.prefix - 1, i + rad) - key0;
        float best = 0.f;
        for (int h = 0; h < g.group; ++h) {
          const float* a = m->a[ab][h];
          float pv;
          if (g.pool_kind == LAVA_POOL_AVG) {
            pv = 0.f;
            for (int j = lo; j <= hi; ++j) pv += a[j];
            pv = pv / (float)g.pool_kernel;
          } else {
            pv = a[lo];
            for (int j = lo + 1; j <= hi; ++j) pv = fmaxf(pv, a[j]);
          }
          best = fmaxf(best, pv);
        }
        sc = best * head_scale;
        p.scores[(size_t)it.layer * g.total_scores + it.s.score_off +
                 (long long)it.kvh * it.s.prefix + i] = sc;
      }
      // entropy sums of this tile in a fixed order: lanes, then warps
      float es = 0.f, et = 0.f;
      if (mine && sc > 0.f) {
        es = sc;
        et = sc * logf(sc);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        es += __shfl_down_sync(0xffffffffu, es, o);
        et += __shfl_down_sync(0xffffffffu, et, o);
      }
      if (lane == 0) {
        m->red[0][quad] = es;
        m->red[1][quad] = et;
      }
      named_barrier(2, 128);
      if (tid == 0) {
        const double s_sum = ((double)m->red[0][0] + (double)m->red[0][1]) +
                             ((double)m->red[0][2] + (double)m->red[0][3]);
        const double t_sum = ((double)m->red[1][0] + (double)m->red[1][1]) +
                             ((double)m->red[1][2] + (double)m->red[1][3]);
        p.ent_part[(size_t)it.head * p.tiles2_per_head + it.tile] = make_double2(s_sum, t_sum);
      }
    }
    if (tid == 0) m->p2_head = 0x3fffffff;  // pass 1 is no longer held back
  } else if (warp >= 12) {
    // ================= value-norm warps: rows of V that belong to the pass-1 tile ============
    const int vt = threadIdx.x - 12 * 32;       // 0..127
    const int sub = vt >> 4, piece = vt & 15;   // 8 rows at a time, 16 x 16 B per row
    for (long long idx = blockIdx.x; idx < items1; idx += gridDim.x) {
      const Item it = decode(p, idx, p.tiles1_per_head, 1);
      if (!it.valid) continue;
      if (!p.vbar_in) {
        const int row0 = it.tile * kTile;
        const char* vb = p.v + ((size_t)it.layer * p.v_ls + (long long)it.kvh * g.v_sh) * 2;
        uint4 raw[16];
#pragma unroll
        for (int r = 0; r < 16; ++r) {
          const int row = row0 + r * 8 + sub;
          raw[r] = make_uint4(0, 0, 0, 0);
          if (row < it.s.n) {
            const uint4* src = reinterpret_cast<const uint4*>(
                vb + (it.s.tok0 + row) * g.v_st * 2 + piece * 16);
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(raw[r].x), "=r"(raw[r].y), "=r"(raw[r].z), "=r"(raw[r].w)
                         : "l"(src));
          }
        }
        float best = 0.f;
#pragma unroll
        for (int r = 0; r < 16; ++r) {
          const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw[r]);
          float sum = 0.f;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float2 f = __bfloat1622float2(h2[j]);
            sum += fabsf(f.x) + fabsf(f.y);
          }
#pragma unroll
          for (int o = 8; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
          best = fmaxf(best, sum);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
        if (lane == 0) atomicMax(&p.vbar_bits[it.head], __float_as_uint(best));
        __threadfence();
      }
      if (named_barrier_or(3, 256, m->abort_flag != 0)) break;
    }
  }

  // ---- teardown: everything this CTA started has finished before shared memory and TMEM go --
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 2) tmem_dealloc(tmem, 512);
}

// entropy of one (layer, sequence) from the per-tile sums, folded in a fixed order
__global__ void __launch_bounds__(256)
entropy_finalize_sm100_kernel(Geom g, const double2* ent_part, int tiles2_per_head, int out_keys,
                              double* entropy) {
  __shared__ double rs[8], rt[8];
  const int prob = blockIdx.x, layer = prob / g.batch, b = prob - layer * g.batch;
  const SeqInfo s = seq_info(g, b);
  const int used = ceil_div(s.prefix, out_keys);
  const int total = g.n_kv_heads * used;
  double sum_s = 0.0, sum_t = 0.0;
  for (int i = threadIdx.x; i < total; i += 256) {
    const int kvh = i / used, t = i - kvh * used;
    const double2 v = ent_part[((size_t)prob * g.n_kv_heads + kvh) * tiles2_per_head + t];
    sum_s += v.x;
    sum_t += v.y;
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

}  // namespace

bool sm100_supported(const Geom& g) {
  if (g.dtype != LAVA_BF16 || g.head_dim != 128) return false;
  if (g.window != 16 && g.window != 32 && g.window != 64 && g.window != 128) return false;
  if (g.group * g.window > 128 || g.group > 8) return false;
  if (g.pool_radius > 31) return false;
  return true;
}

Sm100Layout sm100_layout(const Geom& g, int n_layers) {
  Sm100Layout l;
  l.heads_total = n_layers * g.batch * g.n_kv_heads;
  l.tiles1 = ceil_div(g.max_seqlen, kTile);
  l.out_keys = kTile - 2 * g.pool_radius;
  l.tiles2 = ceil_div(max(1, g.max_seqlen - g.window), l.out_keys);
  size_t off = 0;
  l.off_sync = off;   // counters, ready flags, value-norm bits: zeroed before every launch
  off = up256(off + sizeof(int) * 3 * (size_t)l.heads_total);
  l.sync_bytes = off;
  l.off_part = off;
  off = up256(off + sizeof(float2) * 128 * (size_t)l.heads_total * l.tiles1);
  l.off_lse = off;
  off = up256(off + sizeof(float) * 128 * (size_t)l.heads_total);
  l.off_ent = off;
  off = up256(off + sizeof(double2) * (size_t)l.heads_total * l.tiles2);
  l.total = off;
  return l;
}

lava_status launch_score_sm100(const Geom& g, int n_layers, const void* q, const void* k,
                               const void* v, long long q_ls, long long k_ls, long long v_ls,
                               const float* vbar_in, float* scores, float* vbar_out,
                               double* entropy, char* ws_base, size_t ws_off, cudaStream_t stream) {
  char* ws = ws_base + ws_off;
  EncodeTiledFn encode = encode_fn();
  if (!encode) return fail(LAVA_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
  const Sm100Layout lay = sm100_layout(g, n_layers);

  // Q: [layer][batch*H_q*w rows][128]; K: [layer][H_kv][tokens][128]; boxes of 64 x 128 elements
  CUtensorMap map_q, map_k;
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

  Sm100Params p;
  p.g = g;
  p.n_layers = n_layers;
  p.heads_total = lay.heads_total;
  p.tiles1_per_head = lay.tiles1;
  p.tiles2_per_head = lay.tiles2;
  p.out_keys = lay.out_keys;
  // keep pass 1 within roughly 32 MiB of K+V traffic of pass 2
  const double head_bytes = 2.0 * (double)g.max_seqlen * 256.0;
  int lag = (int)(32.0 * 1024 * 1024 / head_bytes);
  p.lag_heads = lag < 1 ? 1 : (lag > 64 ? 64 : lag);
  p.vbar_in = vbar_in;
  p.scores = scores;
  p.vbar_out = vbar_out;
  p.v = (const char*)v;
  p.v_ls = v_ls;
  p.counters = reinterpret_cast<int*>(ws + lay.off_sync);
  p.ready = p.counters + lay.heads_total;
  p.vbar_bits = reinterpret_cast<unsigned*>(p.ready + lay.heads_total);
  p.part = reinterpret_cast<float2*>(ws + lay.off_part);
  p.neg_lse = reinterpret_cast<float*>(ws + lay.off_lse);
  p.ent_part = reinterpret_cast<double2*>(ws + lay.off_ent);
  p.status = reinterpret_cast<unsigned*>(ws_base);  // the status word opens the workspace

  lava_status rc = check_cuda(cudaMemsetAsync(ws + lay.off_sync, 0, lay.sync_bytes, stream),
                              "sync scratch clear");
  if (rc != LAVA_OK) return rc;

  int dev = 0, sms = 0;
  rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (rc != LAVA_OK) return rc;
  rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev), "SM count");
  if (rc != LAVA_OK) return rc;

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
  const long long items = (long long)lay.heads_total * lay.tiles1;
  const int grid = (int)(items < sms ? items : sms);
  kern<<<grid, kThreads, kSmemBytes, stream>>>(map_q, map_k, p);
  rc = check_cuda(cudaGetLastError(), "score (sm100) launch");
  if (rc != LAVA_OK) return rc;
  entropy_finalize_sm100_kernel<<<n_layers * g.batch, 256, 0, stream>>>(
      g, p.ent_part, lay.tiles2, lay.out_keys, entropy);
  count_launches(2);
  return check_cuda(cudaGetLastError(), "entropy finalize launch");
}

}  // namespace lava
