// LAVa score, generic CUDA-core path: any dtype (fp32 / bf16), head_dim 64 or 128, any window
// and group size.  fp32 inputs always take this path (tf32 tensor cores would not hold the
// 1e-3 relative tolerance on peaked softmax rows).
//
// Passes over one layer (every kernel also batches over layers and sequences in grid.z):
//   1. value_norm_partial : per (KV head, row slice) the largest row L1 norm of V      (Theorem 1)
//   2. stats_partial      : per (query head, key slice, window query) max and sum-exp of the
//                           base-2 logits over the keys the query may see               (Sec. 2)
//   3. combine            : log-sum-exp per window query; Vbar per KV head
//   4. score              : a_h[i] = (1/w) sum_t softmax_t[i]; pool; * Vbar; group max;
//                           entropy partial sums                      (Definition 1, Sec. 4.2-4.3)
//   5. entropy_finalize   : e = (ln S - T/S) / (H_kv n) from ordered fp64 partial sums
// All reductions run in a fixed order, so results are bitwise reproducible.
#include <math.h>

#include "lava_internal.cuh"

namespace lava {
namespace {

constexpr int kTK = 64;        // keys per shared-memory tile
constexpr int kThreads = 256;  // 64 keys x 4 query sub-groups
constexpr int kSlice = Workspace::kSlice;
constexpr int kVSlice = Workspace::kVSlice;
constexpr int kMaxRadius = 31;

__device__ inline float load_elem(const void* p, long long idx, int dtype) {
  if (dtype == LAVA_BF16) return __bfloat162float(((const __nv_bfloat16*)p)[idx]);
  return ((const float*)p)[idx];
}

// Shared-memory carve-up used by the stats and score kernels.
struct Tiles {
  float* qs;   // [w_pad][d]      queries of one head, pre-multiplied by scale*log2(e)
  float* ks;   // [kTK][d + 4]    key tile
  float* zs;   // [w_pad][kTK+1]  base-2 logits of the tile
  int d, kstride;
};

__device__ inline Tiles carve(float* smem, const Geom& g) {
  Tiles t;
  t.d = g.head_dim;
  t.kstride = g.head_dim + 4;
  t.qs = smem;
  t.ks = t.qs + (size_t)g.w_pad * g.head_dim;
  t.zs = t.ks + (size_t)kTK * t.kstride;
  return t;
}

size_t tiles_bytes(const Geom& g) {
  return sizeof(float) * ((size_t)g.w_pad * g.head_dim + (size_t)kTK * (g.head_dim + 4) +
                          (size_t)g.w_pad * (kTK + 1));
}

__device__ inline void load_q(const Tiles& t, const Geom& g, const void* q, int b, int h) {
  const long long base = ((long long)b * g.n_q_heads + h) * g.window * g.head_dim;
  const int total = g.w_pad * g.head_dim;
  for (int i = threadIdx.x; i < total; i += blockDim.x) {
    const int row = i / g.head_dim;
    float x = 0.f;
    if (row < g.window) x = load_elem(q, base + i, g.dtype) * g.scale_log2;
    t.qs[i] = x;
  }
}

// Rows [key0, key0 + count) of KV head `kvh` of the sequence starting at token tok0.
__device__ inline void load_k_tile(const Tiles& t, const Geom& g, const void* k, int kvh,
                                   long long tok0, int key0, int count) {
  const int d = g.head_dim;
  for (int i = threadIdx.x; i < kTK * d; i += blockDim.x) {
    const int row = i / d, c = i - row * d;
    float x = 0.f;
    if (row < count)
      x = load_elem(k, (long long)kvh * g.k_sh + (tok0 + key0 + row) * g.k_st + c, g.dtype);
    t.ks[row * t.kstride + c] = x;
  }
}

// Thread (key = tid % 64, sub = tid / 64) computes logits for rows sub*rows_per .. in groups of 4.
template <typename F>
__device__ inline void for_each_logit(const Tiles& t, const Geom& g, F&& f) {
  const int key = threadIdx.x & (kTK - 1);
  const int sub = threadIdx.x / kTK;
  const int rows_per = g.w_pad / 4;
  const float4* k4 = reinterpret_cast<const float4*>(t.ks + key * t.kstride);
  for (int r0 = sub * rows_per; r0 < (sub + 1) * rows_per; r0 += 4) {
    float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
    const float4* q0 = reinterpret_cast<const float4*>(t.qs + (size_t)(r0 + 0) * t.d);
    const float4* q1 = reinterpret_cast<const float4*>(t.qs + (size_t)(r0 + 1) * t.d);
    const float4* q2 = reinterpret_cast<const float4*>(t.qs + (size_t)(r0 + 2) * t.d);
    const float4* q3 = reinterpret_cast<const float4*>(t.qs + (size_t)(r0 + 3) * t.d);
    for (int c = 0; c < t.d / 4; ++c) {
      const float4 kk = k4[c];
      float4 qq = q0[c];
      acc0 = fmaf(kk.x, qq.x, acc0); acc0 = fmaf(kk.y, qq.y, acc0);
      acc0 = fmaf(kk.z, qq.z, acc0); acc0 = fmaf(kk.w, qq.w, acc0);
      qq = q1[c];
      acc1 = fmaf(kk.x, qq.x, acc1); acc1 = fmaf(kk.y, qq.y, acc1);
      acc1 = fmaf(kk.z, qq.z, acc1); acc1 = fmaf(kk.w, qq.w, acc1);
      qq = q2[c];
      acc2 = fmaf(kk.x, qq.x, acc2); acc2 = fmaf(kk.y, qq.y, acc2);
      acc2 = fmaf(kk.z, qq.z, acc2); acc2 = fmaf(kk.w, qq.w, acc2);
      qq = q3[c];
      acc3 = fmaf(kk.x, qq.x, acc3); acc3 = fmaf(kk.y, qq.y, acc3);
      acc3 = fmaf(kk.z, qq.z, acc3); acc3 = fmaf(kk.w, qq.w, acc3);
    }
    f(r0 + 0, key, acc0);
    f(r0 + 1, key, acc1);
    f(r0 + 2, key, acc2);
    f(r0 + 3, key, acc3);
  }
}

// ------------------------------------------------------------------------------------------
// 1. value-norm partials
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
value_norm_partial_kernel(Geom g, const char* v, long long v_ls, float* vpart, int n_vslices) {
  const int prob = blockIdx.z, layer = prob / g.batch, b = prob - layer * g.batch;
  const int kvh = blockIdx.y, slice = blockIdx.x;
  const SeqInfo s = seq_info(g, b);
  const int row0 = slice * kVSlice;
  float best = 0.f;
  if (row0 < s.n) {
    const int row1 = min(s.n, row0 + kVSlice);
    const int es = g.dtype == LAVA_BF16 ? 2 : 4;
    const char* base = v + (size_t)layer * v_ls * es;
    const int chunks = g.head_dim * es / 16;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int row = row0 + warp; row < row1; row += 8) {
      const char* rp = base + ((long long)kvh * g.v_sh + (s.tok0 + row) * g.v_st) * es;
      float sum = 0.f;
      for (int c = lane; c < chunks; c += 32) {
        const uint4 raw = *reinterpret_cast<const uint4*>(rp + c * 16);
        if (g.dtype == LAVA_BF16) {
          const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float2 f = __bfloat1622float2(p[j]);
            sum += fabsf(f.x) + fabsf(f.y);
          }
        } else {
          const float* p = reinterpret_cast<const float*>(&raw);
          sum += fabsf(p[0]) + fabsf(p[1]) + fabsf(p[2]) + fabsf(p[3]);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      best = fmaxf(best, sum);
    }
  }
  __shared__ float red[8];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = red[0];
    for (int i = 1; i < 8; ++i) m = fmaxf(m, red[i]);
    vpart[((size_t)prob * g.n_kv_heads + kvh) * n_vslices + slice] = m;
  }
}

// ------------------------------------------------------------------------------------------
// 2. softmax statistics per (query head, key slice)
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
stats_partial_kernel(Geom g, const char* q, const char* k, long long q_ls, long long k_ls,
                     float2* stats, int n_slices) {
  extern __shared__ float smem[];
  const Tiles t = carve(smem, g);
  __shared__ float run_m[128], run_z[128];
  const int prob = blockIdx.z, layer = prob / g.batch, b = prob - layer * g.batch;
  const int h = blockIdx.y, slice = blockIdx.x, kvh = h / g.group;
  const SeqInfo s = seq_info(g, b);
  const int key_lo = slice * kSlice;
  if (key_lo >= s.n) return;
  const int key_hi = min(s.n, key_lo + kSlice);
  const int es = g.dtype == LAVA_BF16 ? 2 : 4;
  const void* ql = q + (size_t)layer * q_ls * es;
  const void* kl = k + (size_t)layer * k_ls * es;

  load_q(t, g, ql, b, h);
  for (int i = threadIdx.x; i < g.w_pad; i += blockDim.x) {
    run_m[i] = -INFINITY;
    run_z[i] = 0.f;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int key0 = key_lo; key0 < key_hi; key0 += kTK) {
    const int count = min(kTK, key_hi - key0);
    __syncthreads();
    load_k_tile(t, g, kl, kvh, s.tok0, key0, count);
    __syncthreads();
    for_each_logit(t, g, [&](int row, int key, float z) { t.zs[row * (kTK + 1) + key] = z; });
    __syncthreads();
    // window query `row` sits at position prefix + row and sees keys <= that position
    for (int row = warp; row < g.window; row += kThreads / 32) {
      const int last = s.prefix + row;  // last visible key
      float z0 = -INFINITY, z1 = -INFINITY;
      if (lane < count && key0 + lane <= last) z0 = t.zs[row * (kTK + 1) + lane];
      if (lane + 32 < count && key0 + lane + 32 <= last) z1 = t.zs[row * (kTK + 1) + lane + 32];
      float m = fmaxf(z0, z1);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (m == -INFINITY) continue;  // whole tile masked for this query (warp-uniform)
      float e = exp2f(z0 - m) + exp2f(z1 - m);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
      if (lane == 0) {
        const float om = run_m[row], oz = run_z[row];
        const float nm = fmaxf(om, m);
        run_z[row] = oz * exp2f(om - nm) + e * exp2f(m - nm);
        run_m[row] = nm;
      }
    }
  }
  __syncthreads();
  float2* out = stats + (((size_t)prob * g.n_q_heads + h) * n_slices + slice) * g.window;
  for (int i = threadIdx.x; i < g.window; i += blockDim.x) out[i] = make_float2(run_m[i], run_z[i]);
}

// ------------------------------------------------------------------------------------------
// 3. combine: log-sum-exp per window query and Vbar per KV head
// ------------------------------------------------------------------------------------------
__global__ void combine_kernel(Geom g, const float2* stats, int n_slices, const float* vpart,
                               int n_vslices, const float* vbar_in, float* neg_lse, float* vbar,
                               float* vbar_out, unsigned* status) {
  const int prob = blockIdx.y, layer = prob / g.batch, b = prob - layer * g.batch;
  const SeqInfo s = seq_info(g, b);
  const int used = ceil_div(s.n, kSlice);
  const int h = blockIdx.x;
  if (s.n < g.window && threadIdx.x == 0 && h == 0) atomicOr(status, LAVA_DEV_SHORT_SEQUENCE);
  if (h < g.n_q_heads) {
    for (int t = threadIdx.x; t < g.window; t += blockDim.x) {
      const float2* p = stats + (((size_t)prob * g.n_q_heads + h) * n_slices) * g.window + t;
      float m = -INFINITY;
      for (int sl = 0; sl < used; ++sl) m = fmaxf(m, p[(size_t)sl * g.window].x);
      float z = 0.f;
      for (int sl = 0; sl < used; ++sl) {
        const float2 v = p[(size_t)sl * g.window];
        if (v.y > 0.f) z += v.y * exp2f(v.x - m);
      }
      neg_lse[((size_t)prob * g.n_q_heads + h) * g.window + t] = -(m + log2f(z));
    }
  } else if (threadIdx.x < g.n_kv_heads) {
    // one extra block per problem folds the value-norm partials, one thread per KV head
    const int vused = ceil_div(s.n, kVSlice);
    const int kvh = threadIdx.x;
    float m = 0.f;
    if (vbar_in) {
      m = vbar_in[(size_t)prob * g.n_kv_heads + kvh];
    } else {
      const float* p = vpart + ((size_t)prob * g.n_kv_heads + kvh) * n_vslices;
      for (int sl = 0; sl < vused; ++sl) m = fmaxf(m, p[sl]);
    }
    vbar[(size_t)prob * g.n_kv_heads + kvh] = m;
    if (vbar_out) vbar_out[(size_t)prob * g.n_kv_heads + kvh] = m;
  }
}

// ------------------------------------------------------------------------------------------
// 4. scores of one (KV head, key slice): window mean, pooling, Vbar scale, group max, entropy
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
score_kernel(Geom g, const char* q, const char* k, long long q_ls, long long k_ls,
             const float* neg_lse, const float* vbar, float* scores, double2* ent_part,
             int n_slices) {
  extern __shared__ float smem[];
  const Tiles t = carve(smem, g);
  // a[h_local][i - a_lo], window-mean attention of every head of the group on the slice + halo
  float* a_buf = t.zs + (size_t)g.w_pad * (kTK + 1);
  const int a_stride = kSlice + 2 * kMaxRadius + 2;
  __shared__ float nl[128];
  __shared__ double red_s[kThreads / 32], red_t[kThreads / 32];

  if (batch_has_short_sequence(g)) return;  // reported by the combine kernel
  const int prob = blockIdx.z, layer = prob / g.batch, b = prob - layer * g.batch;
  const int kvh = blockIdx.y, slice = blockIdx.x;
  const SeqInfo s = seq_info(g, b);
  const int s0 = slice * kSlice;
  if (s0 >= s.prefix) return;
  const int s1 = min(s.prefix, s0 + kSlice);
  const int r = g.pool_kind == LAVA_POOL_NONE ? 0 : g.pool_radius;
  const int a_lo = max(0, s0 - r), a_hi = min(s.prefix, s1 + r);
  const int es = g.dtype == LAVA_BF16 ? 2 : 4;
  const void* ql = q + (size_t)layer * q_ls * es;
  const void* kl = k + (size_t)layer * k_ls * es;
  const float inv_w = 1.0f / (float)g.window;

  for (int hl = 0; hl < g.group; ++hl) {
    const int h = kvh * g.group + hl;
    __syncthreads();
    load_q(t, g, ql, b, h);
    for (int i = threadIdx.x; i < g.w_pad; i += blockDim.x)
      nl[i] = i < g.window ? neg_lse[((size_t)prob * g.n_q_heads + h) * g.window + i] : -INFINITY;
    for (int key0 = a_lo; key0 < a_hi; key0 += kTK) {
      const int count = min(kTK, a_hi - key0);
      __syncthreads();
      load_k_tile(t, g, kl, kvh, s.tok0, key0, count);
      __syncthreads();
      float psum = 0.f;  // this thread's rows of the window sum for its key
      for_each_logit(t, g, [&](int row, int key, float z) { psum += exp2f(z + nl[row]); });
      const int key = threadIdx.x & (kTK - 1), sub = threadIdx.x / kTK;
      t.zs[sub * (kTK + 1) + key] = psum;
      __syncthreads();
      if (threadIdx.x < count) {
        const float sum = ((t.zs[0 * (kTK + 1) + key] + t.zs[1 * (kTK + 1) + key]) +
                           t.zs[2 * (kTK + 1) + key]) + t.zs[3 * (kTK + 1) + key];
        a_buf[hl * a_stride + (key0 - a_lo) + key] = sum * inv_w;
      }
    }
  }
  __syncthreads();

  const float scale = vbar[(size_t)prob * g.n_kv_heads + kvh] * g.c_hat;
  float* out = scores + (size_t)layer * g.total_scores + s.score_off + (long long)kvh * s.prefix;
  double ls = 0.0, lt = 0.0;
  for (int i = s0 + threadIdx.x; i < s1; i += blockDim.x) {
    const int lo = max(a_lo, i - r), hi = min(a_hi - 1, i + r);
    float best = 0.f;
    for (int hl = 0; hl < g.group; ++hl) {
      const float* a = a_buf + hl * a_stride - a_lo;
      float p;
      if (g.pool_kind == LAVA_POOL_AVG) {
        p = 0.f;
        for (int j = lo; j <= hi; ++j) p += a[j];
        p = p / (float)g.pool_kernel;
      } else {
        p = a[lo];
        for (int j = lo + 1; j <= hi; ++j) p = fmaxf(p, a[j]);
      }
      best = fmaxf(best, p);
    }
    const float sc = best * scale;
    out[i] = sc;
    if (sc > 0.f) {
      ls += (double)sc;
      lt += (double)(sc * logf(sc));
    }
  }
  // ordered block reduction of the entropy sums
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ls += __shfl_down_sync(0xffffffffu, ls, o);
    lt += __shfl_down_sync(0xffffffffu, lt, o);
  }
  if ((threadIdx.x & 31) == 0) {
    red_s[threadIdx.x >> 5] = ls;
    red_t[threadIdx.x >> 5] = lt;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0, c = 0.0;
    for (int i = 0; i < kThreads / 32; ++i) {
      a += red_s[i];
      c += red_t[i];
    }
    ent_part[((size_t)prob * g.n_kv_heads + kvh) * n_slices + slice] = make_double2(a, c);
  }
}

// ------------------------------------------------------------------------------------------
// 5. entropy of one (layer, sequence): e = (ln S - T/S) / (H_kv * n)
// ------------------------------------------------------------------------------------------
__global__ void entropy_finalize_kernel(Geom g, const double2* ent_part, int n_slices,
                                        double* entropy) {
  const int prob = blockIdx.x, layer = prob / g.batch, b = prob - layer * g.batch;
  const SeqInfo s = seq_info(g, b);
  const int used = ceil_div(s.prefix, kSlice);
  // lane j adds entries j, j+32, ... in ascending order; lanes are then folded pairwise
  double sum_s = 0.0, sum_t = 0.0;
  const int total = g.n_kv_heads * used;
  for (int i = threadIdx.x; i < total; i += 32) {
    const int kvh = i / used, sl = i - kvh * used;
    const double2 p = ent_part[((size_t)prob * g.n_kv_heads + kvh) * n_slices + sl];
    sum_s += p.x;
    sum_t += p.y;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    sum_s += __shfl_down_sync(0xffffffffu, sum_s, o);
    sum_t += __shfl_down_sync(0xffffffffu, sum_t, o);
  }
  if (threadIdx.x != 0) return;
  double e = 0.0;
  if (sum_s > 0.0) e = (log(sum_s) - sum_t / sum_s) / ((double)g.n_kv_heads * (double)s.n);
  entropy[(size_t)layer * g.batch + b] = e;
}

}  // namespace

lava_status launch_score_generic(const Geom& g, int n_layers, const void* q, const void* k,
                                 const void* v, long long q_ls, long long k_ls, long long v_ls,
                                 const float* vbar_in, float* scores, float* vbar_out,
                                 double* entropy, char* ws, const Workspace& lay,
                                 cudaStream_t stream) {
  const int problems = n_layers * g.batch;
  float* vpart = reinterpret_cast<float*>(ws + lay.off_vpart);
  float2* stats = reinterpret_cast<float2*>(ws + lay.off_stats);
  float* neg_lse = reinterpret_cast<float*>(ws + lay.off_lse);
  float* vbar = reinterpret_cast<float*>(ws + lay.off_vbar);
  double2* ent_part = reinterpret_cast<double2*>(ws + lay.off_ent);
  unsigned* status = reinterpret_cast<unsigned*>(ws);

  if (!vbar_in) {
    dim3 grid(lay.n_vslices, g.n_kv_heads, problems);
    value_norm_partial_kernel<<<grid, 256, 0, stream>>>(g, (const char*)v, v_ls, vpart,
                                                        lay.n_vslices);
  }
  const size_t tile_bytes = tiles_bytes(g);
  const size_t score_bytes =
      tile_bytes + sizeof(float) * (size_t)g.group * (kSlice + 2 * kMaxRadius + 2);
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(stats_partial_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               200 * 1024);
    if (e != cudaSuccess) return check_cuda(e, "cudaFuncSetAttribute(score kernels)");
    attr_set = true;
  }
  if (score_bytes > 200 * 1024)
    return fail(LAVA_ERR_UNSUPPORTED, "window/group too large for the generic score kernel");
  {
    dim3 grid(lay.n_slices, g.n_q_heads, problems);
    stats_partial_kernel<<<grid, kThreads, tile_bytes, stream>>>(
        g, (const char*)q, (const char*)k, q_ls, k_ls, stats, lay.n_slices);
  }
  {
    dim3 grid(g.n_q_heads + 1, problems);
    combine_kernel<<<grid, 128, 0, stream>>>(g, stats, lay.n_slices, vpart, lay.n_vslices, vbar_in,
                                            neg_lse, vbar, vbar_out, status);
  }
  {
    dim3 grid(lay.n_slices, g.n_kv_heads, problems);
    score_kernel<<<grid, kThreads, score_bytes, stream>>>(g, (const char*)q, (const char*)k, q_ls,
                                                         k_ls, neg_lse, vbar, scores, ent_part,
                                                         lay.n_slices);
  }
  entropy_finalize_kernel<<<problems, 32, 0, stream>>>(g, ent_part, lay.n_slices, entropy);
  count_launches(vbar_in ? 4 : 5);
  return check_cuda(cudaGetLastError(), "score (generic) launch");
}

// ------------------------------------------------------------------------------------------
// C-hat = largest absolute row sum of W_O (Theorem 1)
// ------------------------------------------------------------------------------------------
namespace {
__global__ void wo_norm_kernel(const void* w_o, int dtype, long long rows, long long cols,
                               float* out) {
  __shared__ float red[32];
  float best = 0.f;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  for (long long r = warp; r < rows; r += nwarps) {
    float sum = 0.f;
    for (long long c = lane; c < cols; c += 32) sum += fabsf(load_elem(w_o, r * cols + c, dtype));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    best = fmaxf(best, sum);
  }
  if (lane == 0) red[warp] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = 0.f;
    for (int i = 0; i < nwarps; ++i) m = fmaxf(m, red[i]);
    *out = m;
  }
}
}  // namespace

lava_status launch_wo_norm(const void* w_o, int dtype, long long rows, long long cols, float* out,
                           cudaStream_t stream) {
  wo_norm_kernel<<<1, 1024, 0, stream>>>(w_o, dtype, rows, cols, out);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "wo_norm launch");
}

}  // namespace lava
