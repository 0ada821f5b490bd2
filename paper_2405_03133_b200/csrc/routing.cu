// Segment-mean pooling, router softmax, causal shift, and their backward
// (Eq. 3 and Algorithm 1 of the Lory paper).  All arithmetic in fp32.
#include "routing.cuh"

namespace lory {

// ---------------------------------------------------------------------------------------
// h_bar[s, :] = (1/T) sum_t x[s*T + t, :]
// grid (S, ceil(d / (32*VEC))), block 256 = 8 warps; warp w sums rows w, w+8, ...;
// a lane owns VEC consecutive columns (one 16-byte load per row).
// ---------------------------------------------------------------------------------------
template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&v)[4]) {
    float4 q = *reinterpret_cast<const float4*>(p);
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  }
};
template <>
struct Vec16<bf16> {
  static constexpr int N = 8;
  __device__ static void load(const bf16* p, float (&v)[8]) {
    uint4 q = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(h[i]);
      v[2 * i] = f.x; v[2 * i + 1] = f.y;
    }
  }
};

template <typename T>
__global__ void __launch_bounds__(256) pool_kernel(const T* __restrict__ x, float* __restrict__ h_bar,
                                                    int Tseg, int d) {
  constexpr int VEC = Vec16<T>::N;
  const int s = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int col = (blockIdx.y * 32 + lane) * VEC;
  __shared__ float red[8][32 * VEC];
  float acc[VEC];
#pragma unroll
  for (int i = 0; i < VEC; ++i) acc[i] = 0.f;
  const bool vec_ok = (col + VEC <= d) && (d % VEC == 0);
  const T* base = x + (size_t)s * Tseg * d;
  if (vec_ok) {
    // four independent 16-byte loads in flight per lane
    int t = warp;
    for (; t + 24 < Tseg; t += 32) {
      float v0[VEC], v1[VEC], v2[VEC], v3[VEC];
      Vec16<T>::load(base + (size_t)t * d + col, v0);
      Vec16<T>::load(base + (size_t)(t + 8) * d + col, v1);
      Vec16<T>::load(base + (size_t)(t + 16) * d + col, v2);
      Vec16<T>::load(base + (size_t)(t + 24) * d + col, v3);
#pragma unroll
      for (int i = 0; i < VEC; ++i) acc[i] += (v0[i] + v1[i]) + (v2[i] + v3[i]);
    }
    for (; t < Tseg; t += 8) {
      float v[VEC];
      Vec16<T>::load(base + (size_t)t * d + col, v);
#pragma unroll
      for (int i = 0; i < VEC; ++i) acc[i] += v[i];
    }
  } else {
    for (int t = warp; t < Tseg; t += 8) {
      const T* row = base + (size_t)t * d;
#pragma unroll
      for (int i = 0; i < VEC; ++i)
        if (col + i < d) acc[i] += to_f32(row[col + i]);
    }
  }
#pragma unroll
  for (int i = 0; i < VEC; ++i) red[warp][lane * VEC + i] = acc[i];
  __syncthreads();
  for (int c = threadIdx.x; c < 32 * VEC; c += 256) {
    float sum = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) sum += red[w][c];
    int gc = blockIdx.y * 32 * VEC + c;
    if (gc < d) h_bar[(size_t)s * d + gc] = sum / (float)Tseg;
  }
}

// ---------------------------------------------------------------------------------------
// p_s = softmax(W_r h_bar_s); w_{b,0} = p_{b,0}; w_{b,n} = p_{b,n-1}.
// One block per segment; its warps (one per expert when E <= 32) take the experts in turn.
// ---------------------------------------------------------------------------------------
// One routing-weight row: fp32 (workspace and, if asked, the caller's copy) and the bf16 hi + lo tables.
__device__ __forceinline__ void write_weight_row(const float* p_sm, size_t row, int E, int lane, float* w_out,
                                                 const RouteExtra& ex) {
  for (int e = lane; e < E; e += 32) {
    w_out[row * E + e] = p_sm[e];
    if (ex.w_copy) ex.w_copy[row * E + e] = p_sm[e];
  }
  if (ex.hi) {
    for (int e = lane; e < ex.Epad; e += 32) {
      const float v = e < E ? p_sm[e] : 0.f;
      const bf16 h = __float2bfloat16_rn(v);
      ex.hi[row * ex.Epad + e] = h;
      ex.lo[row * ex.Epad + e] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
  }
  if (ex.comb) {
    // [hi | lo | hi | hi | lo | lo], 32 columns each
    for (int c = lane; c < 192; c += 32) {
      const int e = c & 31, part = c >> 5;
      const float v = e < E ? p_sm[e] : 0.f;
      const bf16 h = __float2bfloat16_rn(v);
      const bool is_hi = part == 0 || part == 2 || part == 3;
      ex.comb[row * 192 + c] = is_hi ? h : __float2bfloat16_rn(v - __bfloat162float(h));
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(1024) router_kernel(const float* __restrict__ h_bar,
                                                     const T* __restrict__ w_r, float* __restrict__ p_ws,
                                                     float* __restrict__ route_p, float* __restrict__ w_out,
                                                     int N, int d, int E, int prefix, const RouteExtra ex) {
  extern __shared__ float sm[];  // z[E]
  const int s = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float* h = h_bar + (size_t)s * d;
  const int nwarps = blockDim.x >> 5;
  for (int e = warp; e < E; e += nwarps) {
    const T* wr = w_r + (size_t)e * d;
    float acc = 0.f;
    constexpr int VEC = Vec16<T>::N;
    if (d % VEC == 0) {
      for (int j = lane * VEC; j < d; j += 32 * VEC) {
        float wv[VEC];
        Vec16<T>::load(wr + j, wv);
#pragma unroll
        for (int i = 0; i < VEC; i += 4) {
          float4 hv = *reinterpret_cast<const float4*>(h + j + i);
          acc += wv[i] * hv.x + wv[i + 1] * hv.y + wv[i + 2] * hv.z + wv[i + 3] * hv.w;
        }
      }
    } else {
      for (int j = lane; j < d; j += 32) acc += to_f32(wr[j]) * h[j];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) sm[e] = acc;
  }
  __syncthreads();
  if (warp == 0) {
    float m = -INFINITY;
    for (int e = lane; e < E; e += 32) m = fmaxf(m, sm[e]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float sum = 0.f;
    for (int e = lane; e < E; e += 32) {
      float ez = expf(sm[e] - m);
      sm[e] = ez;
      sum += ez;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float inv = 1.0f / sum;
    const int n = s % N;
    for (int e = lane; e < E; e += 32) {
      float p = sm[e] * inv;
      sm[e] = p;
      p_ws[(size_t)s * E + e] = p;
      if (route_p) route_p[(size_t)s * E + e] = p;
    }
    __syncwarp();
    if (prefix) {
      // prefix routing: the first segment's probabilities route every segment of its sequence
      if (n == 0)
        for (int m2 = 0; m2 < N; ++m2) write_weight_row(sm, (size_t)(s + m2), E, lane, w_out, ex);
    } else {
      if (n == 0) write_weight_row(sm, (size_t)s, E, lane, w_out, ex);          // first segment routes itself
      if (n < N - 1) write_weight_row(sm, (size_t)(s + 1), E, lane, w_out, ex);  // and every segment routes the next
    }
  }
}

// ---------------------------------------------------------------------------------------
// Backward of the router path.
// ---------------------------------------------------------------------------------------
// dw[s,:] = sum of the partial slabs; dz_s = p_s * (dp_s - <dp_s, p_s>) with dp_{b,n} = dw_{b,n+1} (0 for the
// last segment); dh_bar_s = W_r^T dz_s.  One block per segment; the block sums the slab rows it needs itself
// (its own row for the dw output, the next segment's row for dp).
template <typename T>
__global__ void __launch_bounds__(256) router_bwd_kernel(const float* __restrict__ partial, int n_slabs,
                                                         const float* __restrict__ p,
                                                         const T* __restrict__ w_r, float* __restrict__ dw,
                                                         float* __restrict__ d_route_w, float* __restrict__ dz,
                                                         float* __restrict__ dh_bar, int S, int N, int d, int E,
                                                         int prefix) {
  __shared__ float red[8][128];
  extern __shared__ float sm[];  // dp[E], dz[E]
  float* dp_sm = sm;
  float* dz_sm = sm + E;
  const int s = blockIdx.x;
  const int n = s % N;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const size_t SE = (size_t)S * E;
  // Sums one [E] row over the slabs, 128 experts at a time (every thread of the block calls this).
  // mode 0: the row is this segment's dw (written out); 1: dp = row; 2: dp += row.
  auto reduce_row = [&](size_t row, int mode) {
    for (int e0 = 0; e0 < E; e0 += 128) {
      for (int e = e0 + lane; e < min(E, e0 + 128); e += 32) {
        // four independent partial sums: the loads of four slabs are in flight together
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        const float* src = partial + row * E + e;
        int c = warp;
        for (; c + 24 < n_slabs; c += 32) {
          a0 += src[(size_t)c * SE];
          a1 += src[(size_t)(c + 8) * SE];
          a2 += src[(size_t)(c + 16) * SE];
          a3 += src[(size_t)(c + 24) * SE];
        }
        for (; c < n_slabs; c += 8) a0 += src[(size_t)c * SE];
        red[warp][e - e0] = (a0 + a1) + (a2 + a3);
      }
      __syncthreads();
      for (int e = e0 + threadIdx.x; e < min(E, e0 + 128); e += 256) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) t += red[w][e - e0];
        if (mode == 0) {
          dw[row * E + e] = t;
          if (d_route_w) d_route_w[row * E + e] = t;
        } else if (mode == 1) {
          dp_sm[e] = t;
        } else {
          dp_sm[e] += t;
        }
      }
      __syncthreads();
    }
  };
  reduce_row((size_t)s, 0);
  for (int e = threadIdx.x; e < E; e += 256) dp_sm[e] = 0.f;
  __syncthreads();
  // gradient reaching p_s: from the next segment's weights, or (prefix routing) from segments 1..N-1 if s is the
  // first segment of its sequence; the first segment's own use of p_s carries no gradient (stop-gradient)
  const bool prefix_mode = (prefix & 1) != 0, first_grad = (prefix & 2) != 0;
  if (!prefix_mode) {
    if (n < N - 1) reduce_row((size_t)s + 1, 1);
  } else if (n == 0) {
    for (int m = 1; m < N; ++m) reduce_row((size_t)s + m, 2);
  }
  // without the stop-gradient the first segment's own weights also feed p_s
  if (first_grad && n == 0) reduce_row((size_t)s, 2);
  if (warp == 0) {
    float dot = 0.f;
    for (int e = lane; e < E; e += 32) dot += dp_sm[e] * p[(size_t)s * E + e];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    for (int e = lane; e < E; e += 32) {
      float v = p[(size_t)s * E + e] * (dp_sm[e] - dot);
      dz_sm[e] = v;
      dz[(size_t)s * E + e] = v;
    }
  }
  __syncthreads();
  // dh_bar_s = W_r^T dz_s.  A thread takes VEC consecutive columns (one 16-byte load per expert row) and one
  // half of the experts; the two halves of the block meet in shared memory.  All loads of a thread are independent.
  constexpr int VEC = Vec16<T>::N;
  if (d % VEC == 0) {
    float* xch = &red[0][0];  // 128 threads x VEC <= 1024 floats
    const int nvec = d / VEC, half = threadIdx.x >> 7, vt = threadIdx.x & 127;
    const int eh = (E + 1) / 2, e_begin = half * eh, e_end = min(E, e_begin + eh);
    for (int v0 = 0; v0 < nvec; v0 += 128) {
      const int v = v0 + vt;
      float acc[VEC];
#pragma unroll
      for (int i = 0; i < VEC; ++i) acc[i] = 0.f;
      if (v < nvec) {
#pragma unroll 8
        for (int e = e_begin; e < e_end; ++e) {
          float wv[VEC];
          Vec16<T>::load(w_r + (size_t)e * d + (size_t)v * VEC, wv);
          const float z = dz_sm[e];
#pragma unroll
          for (int i = 0; i < VEC; ++i) acc[i] += z * wv[i];
        }
      }
      if (half == 1) {
#pragma unroll
        for (int i = 0; i < VEC; ++i) xch[i * 128 + vt] = acc[i];
      }
      __syncthreads();
      if (half == 0 && v < nvec) {
#pragma unroll
        for (int i = 0; i < VEC; i += 4) {
          float4 o = make_float4(acc[i] + xch[i * 128 + vt], acc[i + 1] + xch[(i + 1) * 128 + vt],
                                 acc[i + 2] + xch[(i + 2) * 128 + vt], acc[i + 3] + xch[(i + 3) * 128 + vt]);
          *reinterpret_cast<float4*>(dh_bar + (size_t)s * d + (size_t)v * VEC + i) = o;
        }
      }
      __syncthreads();
    }
  } else {
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
      float a0 = 0.f;
      for (int e = 0; e < E; ++e) a0 += dz_sm[e] * to_f32(w_r[(size_t)e * d + j]);
      dh_bar[(size_t)s * d + j] = a0;
    }
  }
}

// dW_r[e, j] = sum_s dz[s,e] h_bar[s,j].  grid (ceil(d/64), ceil(E/4)), block 512 = 64 columns x 8 runs of
// segments: a thread sums its run for one column and four experts (each h_bar element it loads serves the four),
// then the eight runs are added in a fixed order through shared memory.
template <typename T>
__global__ void __launch_bounds__(512) dwr_kernel(const float* __restrict__ dz, const float* __restrict__ h_bar,
                                                  T* __restrict__ dw_r, int S, int d, int E, int accumulate) {
  __shared__ float red[8][4][64];
  const int jj = threadIdx.x & 63, part = threadIdx.x >> 6;
  const int j = blockIdx.x * 64 + jj, e0 = blockIdx.y * 4;
  const int run = (S + 7) / 8;
  const int s_begin = part * run, s_end = min(S, s_begin + run);
  float a[4] = {0.f, 0.f, 0.f, 0.f};
  if (j < d) {
#pragma unroll 4
    for (int s = s_begin; s < s_end; ++s) {
      const float h = h_bar[(size_t)s * d + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (e0 + i < E) a[i] += dz[(size_t)s * E + e0 + i] * h;
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) red[part][i][jj] = a[i];
  __syncthreads();
  if (threadIdx.x < 256) {
    const int i = threadIdx.x >> 6, e = e0 + i;
    if (j < d && e < E) {
      float out = 0.f;
#pragma unroll
      for (int q = 0; q < 8; ++q) out += red[q][i][jj];
      if (accumulate) out += to_f32(dw_r[(size_t)e * d + j]);
      dw_r[(size_t)e * d + j] = from_f32<T>(out);
    }
  }
}

// dx[t, j] += dh_bar[s(t), j] / T   (mean-pool backward), fp32 add then round to storage.
template <typename T>
__global__ void add_pool_grad_kernel(T* __restrict__ dx, const float* __restrict__ dh_bar, int Tseg, int d,
                                     size_t total) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  size_t t = i / d;
  int j = (int)(i - t * d);
  size_t s = t / Tseg;
  dx[i] = from_f32<T>(to_f32(dx[i]) + dh_bar[s * d + j] / (float)Tseg);
}

// ---------------------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------------------
template <typename T>
int launch_pool_router(const T* x, const T* w_r, float* h_bar, float* p_ws, float* route_p, float* w_out,
                       int B, int N, int Tseg, int d, int E, int prefix, cudaStream_t st, RouteExtra extra) {
  const int S = B * N;
  constexpr int VEC = Vec16<T>::N;
  dim3 grid(S, (unsigned)ceil_div(d, 32 * VEC));
  pool_kernel<T><<<grid, 256, 0, st>>>(x, h_bar, Tseg, d);
  LORY_AFTER_LAUNCH();
  const int router_threads = E >= 32 ? 1024 : (E > 8 ? 32 * E : 256);  // one warp per expert, 8 to 32 warps
  router_kernel<T><<<S, router_threads, E * sizeof(float), st>>>(h_bar, w_r, p_ws, route_p, w_out, N, d, E, prefix, extra);
  LORY_AFTER_LAUNCH();
  return LORY_OK;
}

template <typename T>
int launch_router_backward(const float* dw_partial, int n_slabs, const float* p_ws, const float* h_bar,
                           const T* w_r, float* dw, float* d_route_w, float* dz, float* dh_bar, T* dw_r,
                           int B, int N, int d, int E, int prefix, cudaStream_t st) {
  const int S = B * N;
  router_bwd_kernel<T><<<S, 256, 2 * E * sizeof(float), st>>>(dw_partial, n_slabs, p_ws, w_r, dw, d_route_w, dz, dh_bar, S, N, d, E, prefix);
  LORY_AFTER_LAUNCH();
  dwr_kernel<T><<<dim3((unsigned)ceil_div(d, 64), (unsigned)ceil_div(E, 4)), 512, 0, st>>>(dz, h_bar, dw_r, S, d, E, (prefix & 4) ? 1 : 0);
  LORY_AFTER_LAUNCH();
  return LORY_OK;
}

template <typename T>
int launch_add_pool_grad(T* dx, const float* dh_bar, int tokens, int Tseg, int d, cudaStream_t st) {
  size_t total = (size_t)tokens * d;
  add_pool_grad_kernel<T><<<(unsigned)ceil_div((long)total, 256), 256, 0, st>>>(dx, dh_bar, Tseg, d, total);
  LORY_AFTER_LAUNCH();
  return LORY_OK;
}

// one thread per expert; the S weights of an expert are E floats apart
__global__ void expert_utilization_kernel(const float* __restrict__ route_w, int S, int E, int* __restrict__ counts) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= E) return;
  const float thr = 2.0f / (float)E;
  int n = 0;
  for (int s = 0; s < S; ++s) n += route_w[(size_t)s * E + e] > thr ? 1 : 0;
  counts[e] = n;
}

int launch_expert_utilization(const float* route_w, int S, int E, int* counts, cudaStream_t st) {
  expert_utilization_kernel<<<(unsigned)ceil_div(E, 128), 128, 0, st>>>(route_w, S, E, counts);
  LORY_AFTER_LAUNCH();
  return LORY_OK;
}

#define INST(T)                                                                                              \
  template int launch_pool_router<T>(const T*, const T*, float*, float*, float*, float*, int, int, int, int, \
                                     int, int, cudaStream_t, RouteExtra);                                    \
  template int launch_router_backward<T>(const float*, int, const float*, const float*, const T*, float*,    \
                                         float*, float*, float*, T*, int, int, int, int, int, cudaStream_t); \
  template int launch_add_pool_grad<T>(T*, const float*, int, int, int, cudaStream_t);
INST(float)
INST(bf16)
#undef INST

}  // namespace lory
