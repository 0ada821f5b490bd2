// lory_route_noalloc: the routing step (pool -> router softmax -> causal shift) for callers that
// cannot hand this library a workspace.  Its scratch lives in a fixed device array owned by the
// library image instead of in caller memory.
#include "common.cuh"
#include "routing.cuh"

namespace lory {

// Scratch of the routing step: h_bar [S, d] followed by p [S, E], both float.
// Every GPU that loads this library carries these 4 MiB until the process exits.
static __device__ __align__(256) float g_route_scratch[LORY_NOALLOC_SCRATCH_BYTES / sizeof(float)];

// In host code the array's name only stands in for the symbol; the address a kernel can use comes from
// cudaGetSymbolAddress, asked for while the device is current.  It is asked for on every call and never kept:
// the address belongs to the device's primary context, and a remembered copy would dangle once that context
// has been destroyed and created again (cudaDeviceReset).  The lookup allocates nothing.
static int scratch_for_current_device(float** out) {
  void* ptr = nullptr;
  LORY_CUDA_OK(cudaGetSymbolAddress(&ptr, g_route_scratch));
  *out = static_cast<float*>(ptr);
  return LORY_OK;
}

}  // namespace lory

using namespace lory;

extern "C" int lory_route_noalloc(const lory_dims* dims, const void* x, const void* w_r, float* route_w,
                                  float* route_p, void* cuda_stream) {
  if (!dims || !x || !w_r || !route_w) return LORY_ERR_NULL;
  if (dims->dtype != LORY_FP32 && dims->dtype != LORY_BF16) return LORY_ERR_DTYPE;
  if (dims->B < 1 || dims->L < 1 || dims->T < 1 || dims->d < 1 || dims->E < 1 || dims->L % dims->T != 0 ||
      dims->E > 4096)
    return LORY_ERR_SHAPE;
  const long N = dims->L / dims->T, S = (long)dims->B * N;
  if (S > 65535) return LORY_ERR_SHAPE;
  const size_t need = ((size_t)S * dims->d + (size_t)S * dims->E) * sizeof(float);
  if (need > LORY_NOALLOC_SCRATCH_BYTES) return LORY_ERR_TOO_LARGE;
  int dev = 0, major = 0;
  LORY_CUDA_OK(cudaGetDevice(&dev));
  LORY_CUDA_OK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10) return LORY_ERR_ARCH;
  float* scratch = nullptr;
  LORY_TRY(scratch_for_current_device(&scratch));
  float* h_bar = scratch;
  float* p_ws = scratch + (size_t)S * dims->d;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  call_state().launches = 0;
  // Nothing in the scratch has to start at zero: both kernels overwrite every element they later read.
  if (dims->dtype == LORY_FP32)
    return launch_pool_router<float>((const float*)x, (const float*)w_r, h_bar, p_ws, route_p, route_w, dims->B,
                                     (int)N, dims->T, dims->d, dims->E, (dims->flags & LORY_FLAG_PREFIX_ROUTING) ? 1 : 0, st);
  return launch_pool_router<bf16>((const bf16*)x, (const bf16*)w_r, h_bar, p_ws, route_p, route_w, dims->B, (int)N,
                                  dims->T, dims->d, dims->E, (dims->flags & LORY_FLAG_PREFIX_ROUTING) ? 1 : 0, st);
}
