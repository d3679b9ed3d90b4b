// lava_score_layer_static: the score step for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside another framework's
// memory pool with no allocator hook exposed to them, in a plugin whose host forbids driver
// allocations after start-up, or in a latency-critical serving loop where an allocation (and the
// implicit synchronisation it can bring) is unacceptable.  They can hand over inputs and outputs
// but have no buffer to give as workspace.  For them the scratch of one layer lives in a fixed
// array inside the library image: every GPU that loads the library holds those bytes until the
// process exits, whether or not this entry point is ever called.
#include <mutex>

#include "lava_internal.cuh"

namespace {

// 8 MiB: enough for one layer of a Llama-3-8B-shaped cache up to about 128K tokens.
constexpr size_t kStaticScratchBytes = 8u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of the array, per device.  The array's name is only a host-side handle here;
// kernels need the address cudaGetSymbolAddress returns for the current device.
std::mutex g_setup_mutex;
void* g_scratch_addr[64] = {};

}  // namespace

using namespace lava;

extern "C" lava_status lava_score_layer_static(const lava_layer_desc* desc, const void* q_win,
                                               const void* k, const void* v, const float* vbar_in,
                                               float* scores, float* vbar_out, double* entropy,
                                               uint32_t* device_status_out, void* stream) {
  Geom geom;
  lava_status rc = make_geom(desc, &geom);
  if (rc != LAVA_OK) return rc;
  const size_t need = workspace_layout(desc, 1).total;
  if (need > kStaticScratchBytes)
    return fail(LAVA_ERR_WORKSPACE,
                "this layer needs %zu bytes of scratch; the built-in scratch of "
                "lava_score_layer_static holds %zu bytes: use lava_score_layer with a workspace",
                need, kStaticScratchBytes);
  int dev = 0;
  rc = check_cuda(cudaGetDevice(&dev), "cudaGetDevice");
  if (rc != LAVA_OK) return rc;
  if (dev < 0 || dev >= 64) return fail(LAVA_ERR_UNSUPPORTED, "device index out of range");
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
      void* addr = nullptr;
      rc = check_cuda(cudaGetSymbolAddress(&addr, g_static_scratch), "cudaGetSymbolAddress");
      if (rc != LAVA_OK) return rc;
      g_scratch_addr[dev] = addr;
    }
    scratch = g_scratch_addr[dev];
  }
  cudaStream_t st = (cudaStream_t)stream;
  // The array keeps whatever the previous call left: the status word must start at zero (the
  // score kernels clear the rest of what they rely on themselves).
  rc = check_cuda(cudaMemsetAsync(scratch, 0, Workspace::kStatusBytes, st), "status clear");
  if (rc != LAVA_OK) return rc;
  rc = lava_score_layer(desc, q_win, k, v, vbar_in, scores, vbar_out, entropy, scratch,
                        kStaticScratchBytes, stream);
  if (rc != LAVA_OK) return rc;
  if (device_status_out)
    rc = check_cuda(cudaMemcpyAsync(device_status_out, scratch, sizeof(uint32_t),
                                    cudaMemcpyDeviceToDevice, st), "status copy");
  return rc;
}
