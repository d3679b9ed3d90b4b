// Score variants of the methods the paper compares LAVa with (its table of score functions and
// the related-work paragraph on VATP), as thin steps around the score kernels:
//
//   unit value term     SnapKV / AdaKV: the pooled window-mean attention alone.  The score kernels
//                       run with a caller-style value-norm array of ones and never read V.
//   per-token value     VATP: s_g[i] = c_hat * ||V_g[i]||_1 * max_h pool(a_h)[i].  The norm of a
//     norms             position is common to the query heads of its KV head, so it multiplies the
//                       unit-term score after the group maximum: one streaming pass over V scales
//                       the score array in place, and the layer entropy (Sec. 4.2) is then taken
//                       from the final scores.
#include "lava_internal.cuh"

namespace lava {
namespace {

__global__ void fill_ones_kernel(float* dst, long long count) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) dst[i] = 1.0f;
}

// One warp per prefix position of one KV head: the row's L1 norm times the position's score.
__global__ void __launch_bounds__(256)
token_norm_scale_kernel(Geom g, const char* v, long long v_ls, float* scores) {
  if (batch_has_short_sequence(g)) return;  // the score layout has no room for such a batch
  const int prob = blockIdx.z, layer = prob / g.batch, b = prob - layer * g.batch;
  const int kvh = blockIdx.y;
  const SeqInfo s = seq_info(g, b);
  const int es = g.dtype == LAVA_BF16 ? 2 : 4;
  const int chunks = g.head_dim * es / 16;  // 16-byte pieces per row
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const char* base = v + ((size_t)layer * v_ls + (long long)kvh * g.v_sh) * es;
  float* sc = scores + (size_t)layer * g.total_scores + s.score_off + (long long)kvh * s.prefix;
  for (int i = blockIdx.x * 8 + warp; i < s.prefix; i += gridDim.x * 8) {
    const char* rp = base + (s.tok0 + i) * g.v_st * es;
    float sum = 0.f;
    for (int c = lane; c < chunks; c += 32) {
      const uint4 raw = *reinterpret_cast<const uint4*>(rp + c * 16);
      if (g.dtype == LAVA_BF16) {
        const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 f = __bfloat1622float2(p2[j]);
          sum += fabsf(f.x) + fabsf(f.y);
        }
      } else {
        const float* pf = reinterpret_cast<const float*>(&raw);
        sum += fabsf(pf[0]) + fabsf(pf[1]) + fabsf(pf[2]) + fabsf(pf[3]);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) sc[i] *= sum;
  }
}

}  // namespace

lava_status launch_fill_ones(float* dst, long long count, cudaStream_t stream) {
  if (count <= 0) return LAVA_OK;
  fill_ones_kernel<<<(unsigned)((count + 255) / 256), 256, 0, stream>>>(dst, count);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "fill launch");
}

lava_status launch_token_norm_scale(const Geom& g, int n_layers, const void* v, long long v_ls,
                                    float* scores, cudaStream_t stream) {
  int blocks = (g.max_seqlen + 63) / 64;  // eight positions per block and pass
  if (blocks < 1) blocks = 1;
  if (blocks > 512) blocks = 512;
  dim3 grid(blocks, g.n_kv_heads, n_layers * g.batch);
  token_norm_scale_kernel<<<grid, 256, 0, stream>>>(g, (const char*)v, v_ls, scores);
  count_launches(1);
  return check_cuda(cudaGetLastError(), "token-norm launch");
}

}  // namespace lava
