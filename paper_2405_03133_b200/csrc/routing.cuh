// Pooling / router / shift kernels and their backward (Eq. 3, Algorithm 1).
#pragma once
#include "common.cuh"

namespace lory {

// x [S*T, d] -> h_bar [S, d]; p = softmax(W_r h_bar); w_out = shifted p (Algorithm 1).
// p_ws is the workspace copy of p kept for the backward; route_p may be NULL.
// prefix != 0: prefix routing (every segment of a sequence uses its first segment's p).
// Optional extra outputs of the routing step, written by the router kernel itself:
// a second copy of the routing weights (the caller's route_w), and the bf16 hi + lo tables of the weights that
// the tensor-core merge reads: hi, lo [S, Epad]; comb [S, 192] = [hi | lo | hi | hi | lo | lo] in groups of 32 columns (E <= 32 only).
struct RouteExtra {
  float* w_copy = nullptr;
  bf16* hi = nullptr;
  bf16* lo = nullptr;
  bf16* comb = nullptr;
  int Epad = 0;
};
template <typename T>
int launch_pool_router(const T* x, const T* w_r, float* h_bar, float* p_ws, float* route_p, float* w_out,
                       int B, int N, int Tseg, int d, int E, int prefix, cudaStream_t st,
                       RouteExtra extra = RouteExtra());

// dw = sum of n_slabs partial [S,E] slabs; dz, dh_bar, dW_r from it (stop-gradient on segment 0).
// prefix: bit 0 = prefix routing, bit 1 = keep the first segment's own gradient (no stop-gradient),
// bit 2 = add to the dW_r already stored (gradient accumulation).
template <typename T>
int launch_router_backward(const float* dw_partial, int n_slabs, const float* p_ws, const float* h_bar,
                           const T* w_r, float* dw, float* d_route_w, float* dz, float* dh_bar, T* dw_r,
                           int B, int N, int d, int E, int prefix, cudaStream_t st);

// dx[t,:] += dh_bar[segment(t),:] / T
template <typename T>
int launch_add_pool_grad(T* dx, const float* dh_bar, int tokens, int Tseg, int d, cudaStream_t st);

// counts[e] = number of segments whose routing weight for expert e exceeds 2/E
// (the activation criterion of the paper's expert-utilisation analysis).
int launch_expert_utilization(const float* route_w, int S, int E, int* counts, cudaStream_t st);

}  // namespace lory
