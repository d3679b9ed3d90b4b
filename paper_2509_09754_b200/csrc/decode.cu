// Decode-time attention over the packed cache (the consumer of the compressed K-hat, V-hat of
// Algorithm 1 / Algorithm 2; Sec. 5.3 reports decoding latency with it).  After the layer-wide
// selection every KV head of a (layer, sequence) holds a different number of rows, so the cache
// is ragged per head: rows of (layer l, sequence b, head g) are
//     layer_row_offset[l*batch + b] + head_offsets[l][b][g] ... + head_offsets[l][b][g+1].
// One new token's query heads attend to the rows of their KV head:
//     out[h] = softmax_i( sm_scale * q[h] . K^[g(h)][i] ) V^[g(h)]
//
// bf16, d = 128: one warp takes up to 512 rows of one (layer, sequence, KV head) for all the
// head's queries at once and keeps a running (max, sum, output) in the base-2 domain; the
// partial results of a head's warps are folded by a second small kernel.  K and V rows are
// staged per warp in shared memory with cp.async (three stages of 16 rows each, XOR-swizzled
// 16-byte pieces: two tiles are in flight while one is consumed) and read with ldmatrix for
// mma.sync m16n8k16: S = Q K^T with the queries padded to the 16 rows of the A operand, then
// O += P V with V read transposed.  The (head, chunk) pairs that have rows are listed by a small
// kernel first, and a fixed grid of warps walks that list.  Other geometries take a plain
// CUDA-core kernel.
#include "sm100_ptx.cuh"

namespace lava {
namespace {

using namespace sm100;

constexpr int kChunk = 512;  // rows per warp
constexpr int kBlk = 16;     // rows per step
constexpr int kWarps = 4;
constexpr int kStages = 3;
constexpr int kPartStride = 130;  // 128 outputs, running max, running sum

struct DecodeParams {
  Geom g;
  const void* q;            // [layers, batch, H_q, d]
  const char* k_rows;       // packed cache
  const char* v_rows;
  const int* head_offsets;  // [layers, batch, H_kv + 1]
  const long long* row_off; // [layers * batch (+1)]
  float* part;              // [layers*batch*H_kv][chunks_max][group][kPartStride]
  float* out;               // [layers, batch, H_q, d]
  int2* items;              // work list: (head = prob * H_kv + kvh, chunk) of every non-empty chunk
  int* n_items;
  int chunks_max, heads;
};

__device__ inline void cp_async16(uint32_t saddr, const void* src, bool valid) {
  const int bytes = valid ? 16 : 0;  // 0: the destination is filled with zeros
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(saddr), "l"(src), "r"(bytes)
               : "memory");
}
__device__ inline void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ inline void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ inline uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// Four 8 x 8 matrices of 16-bit elements from shared memory, as stored: thread (g = lane / 4,
// t = lane % 4) receives elements 2t, 2t+1 of row g of each matrix.
__device__ inline void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                   uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(saddr)
               : "memory");
}

constexpr int kTileBytes = kBlk * 256;              // 16 rows of K or of V
constexpr int kStageBytes = 2 * kTileBytes;         // K tile, then V tile
constexpr int kSmemBytes = kWarps * kStages * kStageBytes;

// Row counts live on the device, so the list of (head, chunk) pairs that have rows is built
// there: one block walks the heads in order (exclusive scan of their chunk counts) and writes
// the pairs; the attention kernel then runs a fixed grid over that list and no CTA is launched
// for nothing.
__global__ void __launch_bounds__(1024)
decode_plan_kernel(const DecodeParams p) {
  __shared__ int wsum[32];
  __shared__ int base;
  const Geom& g = p.g;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  for (int h0 = 0; h0 < p.heads; h0 += 1024) {
    const int h = h0 + threadIdx.x;
    int cnt = 0;
    if (h < p.heads) {
      const int prob = h / g.n_kv_heads, kvh = h - prob * g.n_kv_heads;
      const int* hoff = p.head_offsets + (size_t)prob * (g.n_kv_heads + 1);
      const int len = hoff[kvh + 1] - hoff[kvh];
      cnt = len > 0 ? min((len + kChunk - 1) / kChunk, p.chunks_max) : 0;
    }
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    int before = base;
    for (int wdx = 0; wdx < warp; ++wdx) before += wsum[wdx];
    const int start = before + incl - cnt;
    for (int c = 0; c < cnt; ++c) p.items[start + c] = make_int2(h, c);
    __syncthreads();
    if (threadIdx.x == 1023) base = start + cnt;
    __syncthreads();
  }
  if (threadIdx.x == 0) *p.n_items = base;
}

__global__ void __launch_bounds__(kWarps * 32)
decode_partial_kernel(const DecodeParams p) {
  extern __shared__ __align__(128) unsigned char stage_mem[];
  const Geom& g = p.g;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qrow = lane >> 2, t = lane & 3;  // row and column pair of the MMA fragments
  const int n_items = *p.n_items;
  for (int item = blockIdx.x * kWarps + warp; item < n_items; item += gridDim.x * kWarps) {
  const int2 it = p.items[item];
  const int prob = it.x / g.n_kv_heads, kvh = it.x - prob * g.n_kv_heads;
  const int chunk = it.y;
  const int* hoff = p.head_offsets + (size_t)prob * (g.n_kv_heads + 1);
  const int h0 = hoff[kvh], len = hoff[kvh + 1] - h0;
  const int c0 = chunk * kChunk;
  const int nkeys = min(kChunk, len - c0);
  const long long row0 = p.row_off[prob] + h0 + c0;
  const char* krow = p.k_rows + row0 * 256;
  const char* vrow = p.v_rows + row0 * 256;
  const uint32_t sbase = smem_u32(stage_mem) + warp * (kStages * kStageBytes);

  // query fragments (A operand, 16 x 16 per k-step): rows 0..G-1 hold the head's queries
  uint32_t qa[8][2];
#pragma unroll
  for (int s = 0; s < 8; ++s) qa[s][0] = qa[s][1] = 0u;
  if (qrow < g.group) {
    const char* qh = (const char*)p.q + ((size_t)prob * g.n_q_heads + kvh * g.group + qrow) * 256;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      qa[s][0] = *reinterpret_cast<const uint32_t*>(qh + (16 * s + 2 * t) * 2);
      qa[s][1] = *reinterpret_cast<const uint32_t*>(qh + (16 * s + 8 + 2 * t) * 2);
    }
  }
  const int nblk = (nkeys + kBlk - 1) / kBlk;
  // one stage = 16 K rows and 16 V rows, 16-byte pieces XOR-swizzled by the row; rows past the
  // end are filled with zeros
  auto fill = [&](int blk, int stage) {
    const uint32_t st = sbase + stage * kStageBytes;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int idx = lane + 32 * i, r = idx >> 4, pc = idx & 15;
      const int key = blk * kBlk + r;
      const bool ok = key < nkeys;
      const long long off = (long long)(ok ? key : 0) * 256 + pc * 16;
      const uint32_t dst = st + r * 256 + ((pc ^ (r & 7)) << 4);
      cp_async16(dst, krow + off, ok);
      cp_async16(dst + kTileBytes, vrow + off, ok);
    }
  };
#pragma unroll
  for (int s = 0; s < kStages - 1; ++s) {
    if (s < nblk) fill(s, s);
    cp_async_commit();
  }

  float o[16][4];
#pragma unroll
  for (int nd = 0; nd < 16; ++nd) o[nd][0] = o[nd][1] = o[nd][2] = o[nd][3] = 0.f;
  float m_run = -INFINITY, l_run = 0.f;
  const float sc2 = g.scale_log2;
  const int mi = lane >> 3, r8 = lane & 7;

  for (int blk = 0; blk < nblk; ++blk) {
    if (blk + kStages - 1 < nblk) fill(blk + kStages - 1, (blk + kStages - 1) % kStages);
    cp_async_commit();
    cp_async_wait<kStages - 1>();
    __syncwarp();
    const uint32_t st = sbase + (blk % kStages) * kStageBytes;
    // ---- S = Q K^T for 16 rows: two 8-key tiles, eight k-steps --------------------------------
    float s[2][4];
    s[0][0] = s[0][1] = s[0][2] = s[0][3] = 0.f;
    s[1][0] = s[1][1] = s[1][2] = s[1][3] = 0.f;
    {
      // matrices of one k-step: (keys 0-7, piece 2s), (keys 0-7, piece 2s+1), (keys 8-15, ...)
      const int key_l = (mi >> 1) * 8 + r8;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        uint32_t b0, b1, b2, b3;
        const int pc = 2 * ks + (mi & 1);
        ldmatrix_x4(b0, b1, b2, b3, st + key_l * 256 + ((pc ^ (key_l & 7)) << 4));
        mma_bf16_16816(s[0][0], s[0][1], s[0][2], s[0][3], qa[ks][0], 0u, qa[ks][1], 0u, b0, b1);
        mma_bf16_16816(s[1][0], s[1][1], s[1][2], s[1][3], qa[ks][0], 0u, qa[ks][1], 0u, b2, b3);
      }
    }
    // ---- running softmax of query row qrow over its keys 2t, 2t+1 (+8) --------------------------
    float x[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int key = blk * kBlk + (i >> 1) * 8 + 2 * t + (i & 1);
      x[i] = key < nkeys ? s[i >> 1][i & 1] * sc2 : -INFINITY;
    }
    float bm = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
    bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 1));
    bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 2));
    const float m_new = fmaxf(m_run, bm);  // finite: every block has at least one valid key
    const float corr = fast_exp2(m_run - m_new);
    float pr[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) pr[i] = fast_exp2(x[i] - m_new);
    l_run = l_run * corr + ((pr[0] + pr[1]) + (pr[2] + pr[3]));
    m_run = m_new;
    if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
      for (int nd = 0; nd < 16; ++nd) {
        o[nd][0] *= corr;
        o[nd][1] *= corr;
      }
    }
    const uint32_t pa0 = pack_bf16(pr[0], pr[1]), pa2 = pack_bf16(pr[2], pr[3]);
    // ---- O += P V ----------------------------------------------------------------------------
    {
      const int key_l = (mi & 1) * 8 + r8;
#pragma unroll
      for (int nd = 0; nd < 16; nd += 2) {
        uint32_t b0, b1, b2, b3;
        const int pc = nd + (mi >> 1);
        ldmatrix_x4_trans(b0, b1, b2, b3, st + kTileBytes + key_l * 256 + ((pc ^ (key_l & 7)) << 4));
        mma_bf16_16816(o[nd][0], o[nd][1], o[nd][2], o[nd][3], pa0, 0u, pa2, 0u, b0, b1);
        mma_bf16_16816(o[nd + 1][0], o[nd + 1][1], o[nd + 1][2], o[nd + 1][3], pa0, 0u, pa2, 0u, b2, b3);
      }
    }
    __syncwarp();  // the stage may be refilled by the next iteration
  }
  cp_async_wait<0>();
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  if (qrow < g.group) {
    float* dst = p.part + ((((size_t)prob * g.n_kv_heads + kvh) * p.chunks_max + chunk) * g.group + qrow) *
                              kPartStride;
#pragma unroll
    for (int nd = 0; nd < 16; ++nd)
      *reinterpret_cast<float2*>(dst + nd * 8 + 2 * t) = make_float2(o[nd][0], o[nd][1]);
    if (t == 0) {
      dst[128] = m_run;
      dst[129] = l_run;
    }
  }
  __syncwarp();  // the stages are refilled by the warp's next item
  }
}

// Fold of a head's partial results, in chunk order.
__global__ void __launch_bounds__(128)
decode_combine_kernel(const DecodeParams p) {
  const Geom& g = p.g;
  const int h = blockIdx.x, prob = blockIdx.y, kvh = h / g.group, qrow = h - kvh * g.group;
  const int* hoff = p.head_offsets + (size_t)prob * (g.n_kv_heads + 1);
  const int len = hoff[kvh + 1] - hoff[kvh];
  const int nch = (len + kChunk - 1) / kChunk;
  const float* base = p.part + (((size_t)prob * g.n_kv_heads + kvh) * p.chunks_max * g.group + qrow) * kPartStride;
  const size_t stride = (size_t)g.group * kPartStride;
  float m = -INFINITY;
  for (int c = 0; c < nch; ++c) m = fmaxf(m, base[c * stride + 128]);
  float acc = 0.f, l = 0.f;
  for (int c = 0; c < nch; ++c) {
    const float w = fast_exp2(base[c * stride + 128] - m);
    acc += w * base[c * stride + threadIdx.x];
    l += w * base[c * stride + 129];
  }
  p.out[((size_t)prob * g.n_q_heads + h) * 128 + threadIdx.x] = nch > 0 ? acc / l : 0.f;
}

// Any geometry: one block per (query head, layer*sequence), tiles of 128 rows.
__device__ inline float elem(const void* ptr, int dtype, long long i) {
  return dtype == LAVA_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(ptr)[i])
                            : reinterpret_cast<const float*>(ptr)[i];
}

__global__ void __launch_bounds__(128)
decode_generic_kernel(const DecodeParams p) {
  __shared__ float q[128], pr[128], red[4];
  const Geom& g = p.g;
  const int h = blockIdx.x, prob = blockIdx.y, kvh = h / g.group, d = g.head_dim;
  const int* hoff = p.head_offsets + (size_t)prob * (g.n_kv_heads + 1);
  const int len = hoff[kvh + 1] - hoff[kvh];
  const long long row0 = p.row_off[prob] + hoff[kvh];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid < d) q[tid] = elem(p.q, g.dtype, ((long long)prob * g.n_q_heads + h) * d + tid);
  __syncthreads();
  float m = -INFINITY, l = 0.f, acc = 0.f;
  for (int i0 = 0; i0 < len; i0 += 128) {
    const int i = i0 + tid;
    float x = -INFINITY;
    if (i < len) {
      float z = 0.f;
      for (int c = 0; c < d; ++c) z = fmaf(q[c], elem(p.k_rows, g.dtype, (row0 + i) * d + c), z);
      x = z * g.scale_log2;
    }
    float bm = x;
    for (int o = 16; o > 0; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
    if (lane == 0) red[warp] = bm;
    __syncthreads();
    const float m_new = fmaxf(m, fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3])));
    const float e = exp2f(x - m_new);
    pr[tid] = e;
    float bs = e;
    for (int o = 16; o > 0; o >>= 1) bs += __shfl_xor_sync(0xffffffffu, bs, o);
    __syncthreads();
    if (lane == 0) red[warp] = bs;
    __syncthreads();
    const float corr = exp2f(m - m_new);
    l = l * corr + ((red[0] + red[1]) + (red[2] + red[3]));
    acc *= corr;
    m = m_new;
    if (tid < d) {
      const int cnt = min(128, len - i0);
      for (int r = 0; r < cnt; ++r) acc = fmaf(pr[r], elem(p.v_rows, g.dtype, (row0 + i0 + r) * d + tid), acc);
    }
    __syncthreads();
  }
  if (tid < d) p.out[((size_t)prob * g.n_q_heads + h) * d + tid] = len > 0 ? acc / l : 0.f;
}

inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }
inline size_t part_bytes(const Geom& g, int n_layers) {
  const size_t chunks_max = (size_t)(g.max_seqlen + kChunk - 1) / kChunk;
  return up256((size_t)n_layers * g.batch * g.n_kv_heads * chunks_max * g.group * kPartStride * sizeof(float));
}
inline size_t item_bytes(const Geom& g, int n_layers) {
  const size_t chunks_max = (size_t)(g.max_seqlen + kChunk - 1) / kChunk;
  return up256((size_t)n_layers * g.batch * g.n_kv_heads * chunks_max * sizeof(int2));
}

}  // namespace
}  // namespace lava

using namespace lava;

extern "C" {

size_t lava_decode_workspace_bytes(const lava_layer_desc* desc, int32_t n_layers) {
  Geom g;
  if (n_layers < 1 || make_geom(desc, &g) != LAVA_OK) return 0;
  return part_bytes(g, n_layers) + item_bytes(g, n_layers) + 256;
}

lava_status lava_decode_attention_layers(const lava_layer_desc* desc, int32_t n_layers, const void* q,
                                         const void* k_packed, const void* v_packed,
                                         const int32_t* head_offsets,
                                         const int64_t* layer_row_offset, float* out,
                                         void* workspace, size_t workspace_bytes, void* stream) {
  Geom g;
  lava_status rc = make_geom(desc, &g);
  if (rc != LAVA_OK) return rc;
  if (n_layers < 1) return fail(LAVA_ERR_INVALID_ARG, "n_layers must be >= 1");
  if (!q || !k_packed || !v_packed || !head_offsets || !layer_row_offset || !out)
    return fail(LAVA_ERR_INVALID_ARG, "NULL argument");
  if (!aligned16(q) || !aligned16(k_packed) || !aligned16(v_packed) || !aligned16(out))
    return fail(LAVA_ERR_INVALID_ARG, "q, k_packed, v_packed and out must be 16-byte aligned");
  if ((long long)n_layers * g.batch > 65535)
    return fail(LAVA_ERR_UNSUPPORTED, "n_layers*batch must be <= 65535");
  DecodeParams p;
  p.g = g;
  p.q = q;
  p.k_rows = (const char*)k_packed;
  p.v_rows = (const char*)v_packed;
  p.head_offsets = head_offsets;
  p.row_off = (const long long*)layer_row_offset;
  p.out = out;
  p.part = nullptr;
  p.items = nullptr;
  p.n_items = nullptr;
  p.chunks_max = (g.max_seqlen + kChunk - 1) / kChunk;
  p.heads = n_layers * g.batch * g.n_kv_heads;
  cudaStream_t st = (cudaStream_t)stream;
  const bool tensor_path = g.dtype == LAVA_BF16 && g.head_dim == 128 && g.group <= 8;
  if (!tensor_path) {
    decode_generic_kernel<<<dim3(g.n_q_heads, n_layers * g.batch), 128, 0, st>>>(p);
    count_launches(1);
    return check_cuda(cudaGetLastError(), "decode attention launch");
  }
  const size_t need = part_bytes(g, n_layers) + item_bytes(g, n_layers) + 256;
  if (!workspace || workspace_bytes < need)
    return fail(LAVA_ERR_WORKSPACE, "workspace too small: %zu < %zu bytes", workspace_bytes, need);
  if (!aligned16(workspace)) return fail(LAVA_ERR_INVALID_ARG, "workspace must be 16-byte aligned");
  p.part = (float*)workspace;
  p.items = (int2*)((char*)workspace + part_bytes(g, n_layers));
  p.n_items = (int*)((char*)workspace + part_bytes(g, n_layers) + item_bytes(g, n_layers));
  decode_plan_kernel<<<1, 1024, 0, st>>>(p);
  // two CTAs fit an SM (shared memory); a few CTAs per slot even out items of unequal length
  const long long slots = (long long)(sm_count() > 0 ? sm_count() : 1) * 2;
  const long long max_items = (long long)p.heads * p.chunks_max;
  const int grid = (int)std::max<long long>(1, std::min(slots, (max_items + kWarps - 1) / kWarps));
  {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
      rc = check_cuda(cudaFuncSetAttribute(decode_partial_kernel,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes),
                      "decode attention attribute");
      if (rc != LAVA_OK) return rc;
      configured[dev] = true;
    }
  }
  decode_partial_kernel<<<grid, kWarps * 32, kSmemBytes, st>>>(p);
  decode_combine_kernel<<<dim3(g.n_q_heads, n_layers * g.batch), 128, 0, st>>>(p);
  count_launches(3);
  return check_cuda(cudaGetLastError(), "decode attention launch");
}

lava_status lava_decode_attention(const lava_layer_desc* desc, const void* q, const void* k_packed,
                                  const void* v_packed, const int32_t* head_offsets,
                                  const int64_t* layer_row_offset, float* out, void* workspace,
                                  size_t workspace_bytes, void* stream) {
  return lava_decode_attention_layers(desc, 1, q, k_packed, v_packed, head_offsets,
                                      layer_row_offset, out, workspace, workspace_bytes, stream);
}

}  // extern "C"
