// Shared host/device helpers for the Lory MoE kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lory.h"

namespace lory {

typedef __nv_bfloat16 bf16;

// ---- per-thread call bookkeeping (host) -----------------------------------------------
struct CallState {
  int launches;
  char cuda_error[256];
};
CallState& call_state();
void note_cuda_error(cudaError_t e, const char* what);

#define LORY_CUDA_OK(expr)                              \
  do {                                                  \
    cudaError_t _e = (expr);                            \
    if (_e != cudaSuccess) {                            \
      ::lory::note_cuda_error(_e, #expr);               \
      return LORY_ERR_CUDA;                             \
    }                                                   \
  } while (0)

// Call after every kernel launch: counts it and turns a launch error into a status.
#define LORY_AFTER_LAUNCH()                             \
  do {                                                  \
    ::lory::call_state().launches++;                    \
    cudaError_t _e = cudaGetLastError();                \
    if (_e != cudaSuccess) {                            \
      ::lory::note_cuda_error(_e, "kernel launch");     \
      return LORY_ERR_CUDA;                             \
    }                                                   \
  } while (0)

#define LORY_TRY(expr)             \
  do {                             \
    int _s = (expr);               \
    if (_s != LORY_OK) return _s;  \
  } while (0)

// ---- optional per-launch timing (host) ---------------------------------------------------
// When enabled through lory_profile_enable, every labelled launch is bracketed by two CUDA
// events on its stream; lory_profile_read returns label and milliseconds per record.
void prof_begin(const char* label, cudaStream_t st);
void prof_end(cudaStream_t st);
struct ProfScope {
  cudaStream_t st;
  ProfScope(const char* label, cudaStream_t s) : st(s) { prof_begin(label, s); }
  ~ProfScope() { prof_end(st); }
};

// ---- storage conversion ---------------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T>
__device__ __forceinline__ T from_f32(float v);
template <>
__device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

__host__ __device__ __forceinline__ long ceil_div(long a, long b) { return (a + b - 1) / b; }
__host__ __device__ __forceinline__ size_t align_up(size_t a, size_t b) { return (a + b - 1) / b * b; }

// logistic function, fp32
__device__ __forceinline__ float sigmoidf_(float g) { return 1.0f / (1.0f + __expf(-g)); }

// branch-free logistic for the tensor-core epilogues: ex2.approx and rcp.approx (about 2 ulp)
__device__ __forceinline__ float sigmoid_fast(float g) {
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-1.4426950408889634f * g));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
  return r;
}

// ---- device status word -----------------------------------------------------------------
// Kernels with bounded waits OR a non-zero code into this word when a wait gives up.
enum : uint32_t { STATUS_OK = 0, STATUS_TIMEOUT_TMA = 1, STATUS_TIMEOUT_MMA = 2, STATUS_TIMEOUT_EPI = 4,
                  STATUS_DEBUG_BOUNDS = 8 };

// ---- bounds checks of the debug build (-DLORY_DEBUG) ---------------------------------------------
// The tensor-core kernels address memory through TMA boxes, shared-memory stages and TMEM columns whose
// coordinates come from tile arithmetic.  In a debug build every such coordinate is checked before it is used:
// a violated bound raises STATUS_DEBUG_BOUNDS in the status word and the access is skipped (a store) or
// redirected to coordinate zero (a load, so that the barrier waiting for its bytes still completes) instead of
// being issued.  In a release build the checks compile to nothing.
namespace dbg {
#ifdef LORY_DEBUG
constexpr bool kOn = true;
#else
constexpr bool kOn = false;
#endif

// Returns ok; in a debug build a false `ok` is recorded in the status word first.
__device__ __forceinline__ bool check(bool ok, uint32_t* status) {
  if (!kOn) return true;
  if (!ok) atomicOr(status, STATUS_DEBUG_BOUNDS);
  return ok;
}
// [p, p + bytes) lies inside this CTA's dynamic shared memory
__device__ __forceinline__ bool smem_ok(const void* p, uint32_t bytes) {
  if (!kOn) return true;
  extern __shared__ uint8_t dyn_smem_[];
  uint32_t size;
  asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(size));
  const uint32_t lo = static_cast<uint32_t>(__cvta_generic_to_shared(dyn_smem_));
  const uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(p));
  return a >= lo && a + bytes <= lo + size;
}
// TMEM address taddr (lane in bits 16.., column in bits 0..15): `cols` columns starting there stay inside the
// `alloc_cols` columns allocated at `base`, and the 32 lanes starting at its lane stay below 128
__device__ __forceinline__ bool tmem_ok(uint32_t taddr, uint32_t base, uint32_t alloc_cols, uint32_t cols) {
  if (!kOn) return true;
  const uint32_t col = (taddr & 0xFFFFu) - (base & 0xFFFFu), lane = (taddr >> 16) - (base >> 16);
  return col + cols <= alloc_cols && lane + 32u <= 128u;
}
// a TMA coordinate: inside [0, extent) and, for the innermost one, on a 16-byte boundary (8 bf16 elements)
__device__ __forceinline__ bool coord_ok(int c, int extent) { return !kOn || (c >= 0 && c < extent); }
__device__ __forceinline__ bool inner_ok(int c, int extent) { return !kOn || (c >= 0 && c < extent && (c & 7) == 0); }
}  // namespace dbg

}  // namespace lory
