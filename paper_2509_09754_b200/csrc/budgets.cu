// Layer budgets from layer uncertainties (Algorithm 2: B_l = e_l / sum_l e_l * B), integral.
//
// One block per sequence, one thread per layer, fp64 with explicitly rounded operations (no
// fused multiply-add) and layer-ordered sums, so the integers depend only on the entropies
// given.  Rule:
//   * active layers share the remaining budget R in proportion to e_l (equally when the sum of
//     their e is zero / not finite, or in uniform mode; in pyramid mode e_l is replaced by the
//     PyramidKV line quoted in the paper's layer-allocation comparison);
//   * shares become integers by largest remainder: floors first, then +1 in order of
//     decreasing fractional part, ties to the lower layer;
//   * if some active layer falls below the floor or above the cap, the total shortfall and
//     the total excess are compared, the larger side (shortfall on a tie) is clamped and
//     leaves the active set, and the round repeats.  One-sided clamping keeps the remaining
//     problem feasible whenever L*floor <= B <= L*cap.
#include "lava_internal.cuh"

namespace lava {
namespace {

constexpr int kMaxLayers = 256;

// One block per sequence, one thread per layer.  Sums that decide integers are taken by
// thread 0 in layer order so they do not depend on the launch shape.
__global__ void __launch_bounds__(kMaxLayers)
budgets_kernel(int n_layers, int batch, const double* entropy, const long long* total,
               const long long* lo_in, const long long* hi_in, int mode, long long* budget,
               unsigned* status) {
  __shared__ double sh_e[kMaxLayers], sh_frac[kMaxLayers];
  __shared__ long long sh_val[kMaxLayers];
  __shared__ int sh_active[kMaxLayers];
  __shared__ double sh_esum;
  __shared__ long long sh_remaining, sh_rest, sh_short, sh_excess;
  __shared__ int sh_nactive, sh_uniform, sh_done;

  const int b = blockIdx.x, l = threadIdx.x;
  long long lo = lo_in[b], hi = hi_in[b], tot = total[b];
  if (hi < lo) hi = lo;
  if (tot < (long long)n_layers * lo || tot > (long long)n_layers * hi) {
    if (status && l == 0) atomicOr(status, LAVA_DEV_BUDGET_INFEASIBLE);
    tot = tot < (long long)n_layers * lo ? (long long)n_layers * lo : (long long)n_layers * hi;
  }
  const int kind = mode & 0xff;
  if (l < n_layers) {
    double e = entropy[(size_t)l * batch + b];
    if (kind == LAVA_BUDGET_PYRAMID) {
      // the PyramidKV line the paper quotes, for a total of 1: last = 1 / (beta L),
      // first = 2 / L - last, straight in between (same operations, same order, as double)
      const double beta = (mode >> 8) > 0 ? (double)(mode >> 8) : 20.0;
      const double nl = (double)n_layers;
      const double last = __ddiv_rn(1.0, __dmul_rn(beta, nl));
      const double first = __dsub_rn(__ddiv_rn(2.0, nl), last);
      e = n_layers == 1 ? 1.0
                        : __dadd_rn(first, __ddiv_rn(__dmul_rn(__dsub_rn(last, first), (double)l),
                                                     (double)(n_layers - 1)));
    }
    sh_e[l] = e;
    sh_active[l] = 1;
    sh_val[l] = 0;
  }
  if (l == 0) {
    sh_remaining = tot;
    sh_nactive = n_layers;
    sh_done = 0;
  }
  __syncthreads();

  for (int round = 0; round <= n_layers; ++round) {
    if (l == 0) {
      double esum = 0.0;
      for (int m = 0; m < n_layers; ++m)
        if (sh_active[m]) esum = __dadd_rn(esum, sh_e[m]);
      sh_esum = esum;
      sh_uniform = (kind == LAVA_BUDGET_UNIFORM) || !(esum > 0.0) || isinf(esum) || isnan(esum);
    }
    __syncthreads();
    const bool active = l < n_layers && sh_active[l];
    double fl = 0.0;
    if (active) {
      double share;
      if (sh_uniform) share = __ddiv_rn((double)sh_remaining, (double)sh_nactive);
      else share = __ddiv_rn(__dmul_rn((double)sh_remaining, sh_e[l]), sh_esum);
      fl = floor(share);
      sh_frac[l] = __dsub_rn(share, fl);
      sh_val[l] = (long long)fl;
    }
    __syncthreads();
    if (l == 0) {
      long long floors = 0;
      for (int m = 0; m < n_layers; ++m)
        if (sh_active[m]) floors += sh_val[m];
      sh_rest = sh_remaining - floors;
    }
    __syncthreads();
    // Largest remainder: the first |rest| layers in the order (fraction descending, layer
    // ascending) gain one; a negative rest (rounding noise only) is taken from the other end.
    long long val = 0;
    if (active) {
      int rank = 0;
      const double fr = sh_frac[l];
      for (int m = 0; m < n_layers; ++m) {
        if (m == l || !sh_active[m]) continue;
        const double frm = sh_frac[m];
        if (frm > fr || (frm == fr && m < l)) ++rank;
      }
      const long long rest = sh_rest;
      const int na = sh_nactive;
      const long long mag = rest >= 0 ? rest : -rest;
      const long long cycles = mag / na, part = mag % na;
      val = (long long)fl;
      if (rest >= 0) val += cycles + (rank < part ? 1 : 0);
      else val -= cycles + ((na - 1 - rank) < part ? 1 : 0);
    }
    __syncthreads();
    if (active) sh_val[l] = val;
    __syncthreads();
    if (l == 0) {
      long long short_sum = 0, excess_sum = 0;
      for (int m = 0; m < n_layers; ++m) {
        if (!sh_active[m]) continue;
        if (sh_val[m] < lo) short_sum += lo - sh_val[m];
        if (sh_val[m] > hi) excess_sum += sh_val[m] - hi;
      }
      sh_short = short_sum;
      sh_excess = excess_sum;
      sh_done = (short_sum == 0 && excess_sum == 0);
    }
    __syncthreads();
    if (sh_done) break;
    const bool clamp_low = sh_short >= sh_excess;
    if (active) {
      if (clamp_low && val < lo) {
        sh_val[l] = lo;
        sh_active[l] = 0;
      } else if (!clamp_low && val > hi) {
        sh_val[l] = hi;
        sh_active[l] = 0;
      }
    }
    __syncthreads();
    if (l == 0) {
      long long rem = tot;
      int na = 0;
      for (int m = 0; m < n_layers; ++m) {
        if (sh_active[m]) ++na;
        else rem -= sh_val[m];
      }
      sh_remaining = rem;
      sh_nactive = na;
    }
    __syncthreads();
    if (sh_nactive == 0) break;
  }
  if (l < n_layers) budget[(size_t)l * batch + b] = sh_val[l];
}

// Exclusive prefix sums of the budgets in (layer, sequence) order: first packed row of each.
__global__ void __launch_bounds__(256)
row_offsets_kernel(int count, const long long* budget, long long* row_off) {
  __shared__ long long warp_tot[8];
  __shared__ long long carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int base = 0; base < count; base += 256) {
    const int i = base + threadIdx.x;
    const long long x = i < count ? budget[i] : 0;
    long long incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    long long before = carry;
    for (int wdx = 0; wdx < warp; ++wdx) before += warp_tot[wdx];
    if (i < count) row_off[i] = before + incl - x;
    __syncthreads();
    if (threadIdx.x == 255) carry = before + incl;
    __syncthreads();
  }
  if (threadIdx.x == 0) row_off[count] = carry;
}

}  // namespace

lava_status launch_budgets(int n_layers, int batch, const double* entropy, const long long* total,
                           const long long* lo, const long long* hi, int mode, long long* budget,
                           long long* row_off, unsigned* status, cudaStream_t stream) {
  const int threads = ((n_layers + 31) / 32) * 32;
  budgets_kernel<<<batch, threads, 0, stream>>>(n_layers, batch, entropy, total, lo, hi, mode,
                                                budget, status);
  row_offsets_kernel<<<1, 256, 0, stream>>>(n_layers * batch, budget, row_off);
  count_launches(2);
  return check_cuda(cudaGetLastError(), "layer_budgets launch");
}

}  // namespace lava
