// Diagnostic: how fast, and up to what footprint, does the L2 cache hand data written by one pass to the pass
// that follows it?  This is the question behind keeping the per-segment merged weights (or their gradients)
// out of HBM between the kernel that produces them and the kernel that consumes them.
//
// A ring of `slots` regions of `slot_bytes` each.  Every CTA owns one contiguous slice of every slot.  In
// iteration i it writes its slice of slot (i mod slots) and reads a slice of slot ((i - lag) mod slots), written
// `lag` iterations earlier: its own (shift = 0) or that of the CTA `shift` positions further (another SM; the
// CTAs are not synchronised, so such a read may see the previous round's data, which is all the same to a
// bandwidth measurement).  Loads and stores bypass L1 (.cg), so a read is served by L2 when the line is
// still there and by HBM otherwise.  The footprint the cache has to hold for reads to hit is
// (lag + 1) * slot_bytes.
#include "common.cuh"

namespace lory {

// mode: bit 0 = write, bit 1 = read
__global__ void __launch_bounds__(512) l2_ring_kernel(uint4* __restrict__ buf, size_t slot_vec, size_t slice_vec,
                                                      int slots, int lag, int iters, int mode, int shift,
                                                      unsigned int* __restrict__ sink) {
  uint4 acc = make_uint4(0u, 0u, 0u, 0u);
  const size_t base = (size_t)blockIdx.x * slice_vec;
  const size_t rbase = (size_t)((blockIdx.x + shift) % gridDim.x) * slice_vec;  // whose slice this CTA reads
  for (int it = 0; it < iters; ++it) {
    if (mode & 1) {
      uint4* dst = buf + (size_t)(it % slots) * slot_vec + base;
      const uint4 v = make_uint4((unsigned)it, threadIdx.x, blockIdx.x, 0x9e3779b9u);
      for (size_t i = threadIdx.x; i < slice_vec; i += blockDim.x) __stcg(dst + i, v);
    }
    if (mode & 2) {
      const uint4* src = buf + (size_t)(((it - lag) % slots + slots) % slots) * slot_vec + rbase;
      size_t i = threadIdx.x;
      for (; i + 3 * (size_t)blockDim.x < slice_vec; i += 4 * (size_t)blockDim.x) {
        const uint4 a = __ldcg(src + i), b = __ldcg(src + i + blockDim.x), c = __ldcg(src + i + 2 * blockDim.x),
                    d = __ldcg(src + i + 3 * blockDim.x);
        acc.x ^= a.x ^ b.x ^ c.x ^ d.x;
        acc.y ^= a.y ^ b.y ^ c.y ^ d.y;
        acc.z ^= a.z ^ b.z ^ c.z ^ d.z;
        acc.w ^= a.w ^ b.w ^ c.w ^ d.w;
      }
      for (; i < slice_vec; i += blockDim.x) {
        const uint4 a = __ldcg(src + i);
        acc.x ^= a.x; acc.y ^= a.y; acc.z ^= a.z; acc.w ^= a.w;
      }
    }
  }
  // keeps the loads alive; the condition never holds for the values written above
  if ((acc.x ^ acc.y ^ acc.z ^ acc.w) == 0x12345u) atomicAdd(sink, 1u);
}

}  // namespace lory

using namespace lory;

extern "C" int lory_probe_l2_ring(void* buf, size_t buf_bytes, size_t slot_bytes, int slots, int lag, int iters,
                                  int mode, int shift, float* ms_out, void* cuda_stream) {
  if (!buf || !ms_out) return LORY_ERR_NULL;
  if (slots < 1 || lag < 0 || lag > slots || iters < 1 || (mode & 3) == 0 || (mode & ~3) || shift < 0)
    return LORY_ERR_SHAPE;
  if (((uintptr_t)buf & 255) != 0) return LORY_ERR_WORKSPACE;
  int dev = 0, sms = 0;
  LORY_CUDA_OK(cudaGetDevice(&dev));
  LORY_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int grid = 2 * sms;
  // every CTA's slice: a multiple of 512 threads x 16 bytes
  const size_t slice_vec = slot_bytes / 16 / grid / 512 * 512;
  if (slice_vec == 0) return LORY_ERR_SHAPE;
  const size_t slot_vec = slice_vec * grid;
  if ((size_t)slots * slot_vec * 16 + 256 > buf_bytes) return LORY_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  unsigned int* sink = (unsigned int*)((char*)buf + (size_t)slots * slot_vec * 16);
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  LORY_CUDA_OK(cudaEventCreate(&e0));
  LORY_CUDA_OK(cudaEventCreate(&e1));
  // one untimed pass first: the timed pass then starts with the ring written and the caches warm
  l2_ring_kernel<<<grid, 512, 0, st>>>((uint4*)buf, slot_vec, slice_vec, slots, lag, slots + lag, mode | 1, shift, sink);
  cudaEventRecord(e0, st);
  l2_ring_kernel<<<grid, 512, 0, st>>>((uint4*)buf, slot_vec, slice_vec, slots, lag, iters, mode, shift, sink);
  cudaEventRecord(e1, st);
  cudaError_t e = cudaEventSynchronize(e1);
  if (e == cudaSuccess) e = cudaGetLastError();
  float ms = 0.f;
  if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (e != cudaSuccess) {
    note_cuda_error(e, "lory_probe_l2_ring");
    return LORY_ERR_CUDA;
  }
  *ms_out = ms;
  return LORY_OK;
}
