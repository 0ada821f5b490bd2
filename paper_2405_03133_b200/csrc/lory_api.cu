// C ABI of the Lory MoE layer: argument checks, workspace layout, and the order in which the
// kernels run.  See lory.h for the contract.
#include <stdio.h>
#include <string.h>

#include "common.cuh"
#include "layout.cuh"
#include "routing.cuh"
#include "simt.cuh"
#include "block.cuh"
#include "tc.cuh"

namespace lory {

CallState& call_state() {
  static thread_local CallState s = {0, {0}};
  return s;
}

void note_cuda_error(cudaError_t e, const char* what) {
  CallState& s = call_state();
  snprintf(s.cuda_error, sizeof(s.cuda_error), "%s: %s (%s)", what, cudaGetErrorName(e), cudaGetErrorString(e));
}

static const int kMaxDevices = 64;  // per-device host state (streams, events) is kept per device ordinal

// ---- per-launch timing ---------------------------------------------------------------------
static const int PROF_MAX = 8192;
struct Prof {
  bool on;
  int n;
  bool open;
  cudaEvent_t ev[2 * PROF_MAX];
  bool created[2 * PROF_MAX];
  const char* label[PROF_MAX];
};
static Prof g_prof;

void prof_begin(const char* label, cudaStream_t st) {
  Prof& P = g_prof;
  if (!P.on || P.n >= PROF_MAX) return;
  for (int j = 0; j < 2; ++j) {
    int i = 2 * P.n + j;
    if (!P.created[i]) {
      if (cudaEventCreate(&P.ev[i]) != cudaSuccess) return;
      P.created[i] = true;
    }
  }
  P.label[P.n] = label;
  cudaEventRecord(P.ev[2 * P.n], st);
  P.open = true;
}

void prof_end(cudaStream_t st) {
  Prof& P = g_prof;
  if (!P.on || !P.open) return;
  cudaEventRecord(P.ev[2 * P.n + 1], st);
  P.open = false;
  P.n++;
}

static bool use_tc(const lory_dims& D) {
  return D.dtype == LORY_BF16 && !(D.flags & LORY_FLAG_SIMT) && tc_supported(D);
}

static Layout make_layout(const lory_dims& D) {
  Layout Lo;
  const size_t S = (size_t)D.B * (D.L / D.T), tok = (size_t)D.B * D.L;
  const size_t es = D.dtype == LORY_BF16 ? 2 : 4;
  const size_t P1 = (size_t)D.f * D.d;
  // plain-FMA pipeline: [S, f*d] row-major; tensor-core pipeline: blocked [rb][cb][S][64][64]
  const size_t PS = P1;
  Lo.seg_stride = (long)PS;
  const bool blk = use_tc(D);
  const size_t n13 = blk ? tc_blocked_elems(D, D.f, D.d) : S * PS;
  const size_t n2 = blk ? tc_blocked_elems(D, D.d, D.f) : S * PS;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  Lo.status = take(256);
  Lo.h_bar = take(S * D.d * 4);
  Lo.p = take(S * D.E * 4);
  Lo.w = take(S * D.E * 4);
  Lo.w_split = take(D.dtype == LORY_BF16 ? tc_w_split_bytes(D) : 0);
  Lo.wbar1 = take(n13 * es);
  Lo.wbar3 = take(n13 * es);
  Lo.wbar2 = take(n2 * es);
  Lo.G = take(tok * D.f * es);
  Lo.U = take(tok * D.f * es);
  Lo.H = take(tok * D.f * es);
  Lo.fwd_end = off;
  Lo.dG = take(tok * D.f * es);
  Lo.dU = take(tok * D.f * es);
  if (blk && (D.flags & LORY_FLAG_CHUNKED_ADJOINT)) {
    // one L2-sized buffer for a rectangle of per-segment weight gradients at a time
    Lo.dwbar1 = take(tc_adjoint_ring_elems(D) * es);
    Lo.dwbar3 = Lo.dwbar2 = Lo.dwbar1;
  } else {
    Lo.dwbar1 = take(n13 * es);
    Lo.dwbar3 = take(n13 * es);
    Lo.dwbar2 = take(n2 * es);
  }
  Lo.k_chunk = 8192;
  int simt_slabs = 3 * (int)ceil_div((long)P1, Lo.k_chunk);
  Lo.n_slabs = use_tc(D) ? tc_dw_slabs(D) : simt_slabs;
  Lo.dw_partial = take((size_t)Lo.n_slabs * S * D.E * 4);
  Lo.dw = take(S * D.E * 4);
  Lo.dz = take(S * D.E * 4);
  Lo.dh_bar = take(S * D.d * 4);
  Lo.bwd_end = off;
  return Lo;
}

static int check_dims(const lory_dims* D) {
  if (!D) return LORY_ERR_NULL;
  if (D->dtype != LORY_FP32 && D->dtype != LORY_BF16) return LORY_ERR_DTYPE;
  if (D->B < 1 || D->L < 1 || D->T < 1 || D->d < 1 || D->f < 1 || D->E < 1) return LORY_ERR_SHAPE;
  if (D->L % D->T != 0) return LORY_ERR_SHAPE;
  if (D->E > 4096) return LORY_ERR_SHAPE;
  if (D->dtype == LORY_BF16) {
    if (D->d % 8 != 0 || D->f % 8 != 0 || D->E > 128) return LORY_ERR_SHAPE;
  }
  if ((long)D->f * D->d > 0x7fffffffL) return LORY_ERR_SHAPE;
  if ((long)D->B * D->L >= (1L << 30)) return LORY_ERR_SHAPE;
  if ((long)D->B * (D->L / D->T) > 65535) return LORY_ERR_SHAPE;
  return LORY_OK;
}

static int check_device() {
  int dev = 0;
  LORY_CUDA_OK(cudaGetDevice(&dev));
  int major = 0;
  LORY_CUDA_OK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10) return LORY_ERR_ARCH;
  return LORY_OK;
}

// ---------------------------------------------------------------------------------------
// Plain-FMA pipeline (fp32 mode, and bf16 with LORY_FLAG_SIMT).
// ---------------------------------------------------------------------------------------
template <typename T>
struct Simt {
  static int g_wTT(const SimtGemm& g, cudaStream_t st) { return launch_simt_gemm<float, T, T>(g, st); }
  static int g_TTT(const SimtGemm& g, cudaStream_t st) { return launch_simt_gemm<T, T, T>(g, st); }
  static int g_TTf(const SimtGemm& g, cudaStream_t st) { return launch_simt_gemm<T, T, float>(g, st); }
};

// Field order of SimtGemm: A B C | M N K groups | a_m a_k a_g | b_k b_n b_g | c_m c_n c_g | k_chunk accumulate
template <typename T>
static int simt_ffn_forward(const lory_dims& D, const Layout& Lo, char* ws, const T* x, const T* w1, const T* w2,
                            const T* w3, T* y, cudaStream_t st) {
  const int S = D.B * (D.L / D.T), Tn = D.T, d = D.d, f = D.f, E = D.E;
  const long P1 = (long)f * d, PS = Lo.seg_stride;
  const float* w = (const float*)(ws + Lo.w);
  T* wbar1 = (T*)(ws + Lo.wbar1);
  T* wbar3 = (T*)(ws + Lo.wbar3);
  T* wbar2 = (T*)(ws + Lo.wbar2);
  T* G = (T*)(ws + Lo.G);
  T* U = (T*)(ws + Lo.U);
  T* H = (T*)(ws + Lo.H);
  // merge: Wbar_k[S, P1] = w[S, E] . W_k[E, P1]   (Eq. 2)
  const T* src[3] = {w1, w3, w2};
  T* dst[3] = {wbar1, wbar3, wbar2};
  for (int k = 0; k < 3 && !(D.flags & LORY_FLAG_REUSE_MERGED); ++k) {
    SimtGemm g = {w, src[k], dst[k], S, (int)P1, E, 1, E, 1, 0, P1, 1, 0, PS, 1, 0, 0, 0};
    LORY_TRY(Simt<T>::g_wTT(g, st));
  }
  // G = X Wbar1^T, U = X Wbar3^T, per segment
  {
    SimtGemm g = {x, wbar1, G, Tn, f, d, S, d, 1, (long)Tn * d, 1, d, PS, f, 1, (long)Tn * f, 0, 0};
    LORY_TRY(Simt<T>::g_TTT(g, st));
    g.B = wbar3;
    g.C = U;
    LORY_TRY(Simt<T>::g_TTT(g, st));
  }
  LORY_TRY(launch_swiglu_fwd<T>(G, U, H, (size_t)S * Tn * f, st));
  // Y = H Wbar2^T
  {
    SimtGemm g = {H, wbar2, y, Tn, d, f, S, f, 1, (long)Tn * f, 1, f, PS, d, 1, (long)Tn * d, 0, 0};
    LORY_TRY(Simt<T>::g_TTT(g, st));
  }
  return LORY_OK;
}

template <typename T>
static int simt_ffn_backward(const lory_dims& D, const Layout& Lo, char* ws, const T* x, const T* w1, const T* w2,
                             const T* w3, const T* dy, T* dx, T* dw1, T* dw2, T* dw3, cudaStream_t st) {
  const int S = D.B * (D.L / D.T), Tn = D.T, d = D.d, f = D.f, E = D.E;
  const long P1 = (long)f * d, PS = Lo.seg_stride;
  const float* w = (const float*)(ws + Lo.w);
  T* wbar1 = (T*)(ws + Lo.wbar1);
  T* wbar3 = (T*)(ws + Lo.wbar3);
  T* wbar2 = (T*)(ws + Lo.wbar2);
  T* G = (T*)(ws + Lo.G);
  T* U = (T*)(ws + Lo.U);
  T* H = (T*)(ws + Lo.H);
  T* dG = (T*)(ws + Lo.dG);
  T* dU = (T*)(ws + Lo.dU);
  T* dwbar1 = (T*)(ws + Lo.dwbar1);
  T* dwbar3 = (T*)(ws + Lo.dwbar3);
  T* dwbar2 = (T*)(ws + Lo.dwbar2);
  float* dw_partial = (float*)(ws + Lo.dw_partial);
  // dH = dY Wbar2 (into dG), then the SwiGLU backward in place
  {
    SimtGemm g = {dy, wbar2, dG, Tn, f, d, S, d, 1, (long)Tn * d, f, 1, PS, f, 1, (long)Tn * f, 0, 0};
    LORY_TRY(Simt<T>::g_TTT(g, st));
  }
  LORY_TRY(launch_swiglu_bwd<T>(G, U, dG, dU, (size_t)S * Tn * f, st));
  // dWbar2 = dY^T H  [d, f]
  {
    SimtGemm g = {dy, H, dwbar2, d, f, Tn, S, 1, d, (long)Tn * d, f, 1, (long)Tn * f, f, 1, PS, 0, 0};
    LORY_TRY(Simt<T>::g_TTT(g, st));
  }
  // dWbar1 = dG^T X, dWbar3 = dU^T X  [f, d]
  {
    SimtGemm g = {dG, x, dwbar1, f, d, Tn, S, 1, f, (long)Tn * f, d, 1, (long)Tn * d, d, 1, PS, 0, 0};
    LORY_TRY(Simt<T>::g_TTT(g, st));
    g.A = dU;
    g.C = dwbar3;
    LORY_TRY(Simt<T>::g_TTT(g, st));
  }
  // dX = dG Wbar1 + dU Wbar3
  {
    SimtGemm g = {dG, wbar1, dx, Tn, d, f, S, f, 1, (long)Tn * f, d, 1, PS, d, 1, (long)Tn * d, 0, 0};
    LORY_TRY(Simt<T>::g_TTT(g, st));
    g.A = dU;
    g.B = wbar3;
    g.accumulate = 1;
    LORY_TRY(Simt<T>::g_TTT(g, st));
  }
  // adjoint of the merge: dW_k[E, P1] = w^T[E, S] . dWbar_k[S, P1]
  // and dw[S, E] += dWbar_k[S, P1] . W_k^T[P1, E]  (K split into slabs)
  const T* dsrc[3] = {dwbar1, dwbar3, dwbar2};
  const T* wsrc[3] = {w1, w3, w2};
  T* ddst[3] = {dw1, dw3, dw2};
  const int slabs_per = (int)ceil_div(P1, Lo.k_chunk);
  for (int k = 0; k < 3; ++k) {
    SimtGemm g = {w, dsrc[k], ddst[k], E, (int)P1, S, 1, 1, E, 0, PS, 1, 0, P1, 1, 0, 0,
                  (D.flags & LORY_FLAG_ACCUMULATE_GRADS) ? 1 : 0};
    LORY_TRY(Simt<T>::g_wTT(g, st));
    SimtGemm h = {dsrc[k], wsrc[k], dw_partial + (size_t)k * slabs_per * S * E, S, E, (int)P1, slabs_per,
                  PS, 1, 0, 1, P1, 0, E, 1, (long)S * E, Lo.k_chunk, 0};
    LORY_TRY(Simt<T>::g_TTf(h, st));
  }
  return LORY_OK;
}

// ---------------------------------------------------------------------------------------
// Whole-layer drivers
// ---------------------------------------------------------------------------------------
// residual (optional): y = residual + layer output.  The tensor-core pipeline adds it in its last GEMM's epilogue,
// the plain-FMA pipeline with a separate kernel.
static int run_ffn_forward(const lory_dims& D, const Layout& Lo, char* ws, const float* x, const float* w1,
                           const float* w2, const float* w3, float* y, cudaStream_t st, bool, const float* residual) {
  {
    ProfScope ps("simt_forward", st);
    LORY_TRY(simt_ffn_forward<float>(D, Lo, ws, x, w1, w2, w3, y, st));
  }
  if (!residual) return LORY_OK;
  ProfScope ps("residual_add", st);
  return launch_residual_add<float>(y, residual, (size_t)D.B * D.L * D.d, st);
}
static int run_ffn_forward(const lory_dims& D, const Layout& Lo, char* ws, const bf16* x, const bf16* w1,
                           const bf16* w2, const bf16* w3, bf16* y, cudaStream_t st, bool w_is_split,
                           const bf16* residual) {
  if (use_tc(D)) return tc_ffn_forward(D, Lo, ws, x, w1, w2, w3, y, st, w_is_split, residual);
  {
    ProfScope ps("simt_forward", st);
    LORY_TRY(simt_ffn_forward<bf16>(D, Lo, ws, x, w1, w2, w3, y, st));
  }
  if (!residual) return LORY_OK;
  ProfScope ps("residual_add", st);
  return launch_residual_add<bf16>(y, residual, (size_t)D.B * D.L * D.d, st);
}
static int run_ffn_backward(const lory_dims& D, const Layout& Lo, char* ws, const float* x, const float* w1,
                            const float* w2, const float* w3, const float* dy, float* dx, float* dw1, float* dw2,
                            float* dw3, cudaStream_t st) {
  ProfScope ps("simt_backward", st);
  return simt_ffn_backward<float>(D, Lo, ws, x, w1, w2, w3, dy, dx, dw1, dw2, dw3, st);
}
static int run_ffn_backward(const lory_dims& D, const Layout& Lo, char* ws, const bf16* x, const bf16* w1,
                            const bf16* w2, const bf16* w3, const bf16* dy, bf16* dx, bf16* dw1, bf16* dw2,
                            bf16* dw3, cudaStream_t st) {
  if (use_tc(D)) return tc_ffn_backward(D, Lo, ws, x, w1, w2, w3, dy, dw1, dw2, dw3, st);
  ProfScope ps("simt_backward", st);
  return simt_ffn_backward<bf16>(D, Lo, ws, x, w1, w2, w3, dy, dx, dw1, dw2, dw3, st);
}

template <typename T>
static int forward_impl(const lory_dims& D, const Layout& Lo, const T* x, const T* w_r, const T* w1, const T* w2,
                        const T* w3, T* y, float* route_w, float* route_p, const float* injected_w, char* ws,
                        cudaStream_t st, const T* residual = nullptr) {
  const int N = D.L / D.T, S = D.B * N;
  LORY_CUDA_OK(cudaMemsetAsync(ws + Lo.status, 0, 256, st));
  float* w = (float*)(ws + Lo.w);
  bool w_is_split = false;
  if (D.flags & LORY_FLAG_REUSE_MERGED) {
    // the merged weights of an earlier call are still in the workspace: nothing to route or merge
  } else if (injected_w) {
    LORY_CUDA_OK(cudaMemcpyAsync(w, injected_w, (size_t)S * D.E * 4, cudaMemcpyDeviceToDevice, st));
  } else {
    // the router kernel also writes the caller's copy of the weights and, for the tensor-core pipeline, their
    // bf16 hi / lo tables
    ProfScope ps("pool_router", st);
    RouteExtra extra;
    extra.w_copy = route_w;
    if (D.dtype == LORY_BF16 && use_tc(D)) {
      tc_split_tables(D, Lo, ws, &extra.hi, &extra.lo, &extra.comb, &extra.Epad);
      w_is_split = true;
    }
    LORY_TRY(launch_pool_router<T>(x, w_r, (float*)(ws + Lo.h_bar), (float*)(ws + Lo.p), route_p, w, D.B, N, D.T,
                                   D.d, D.E, (D.flags & LORY_FLAG_PREFIX_ROUTING) ? 1 : 0, st, extra));
  }
  return run_ffn_forward(D, Lo, ws, x, w1, w2, w3, y, st, w_is_split, residual);
}

template <typename T>
static int backward_impl(const lory_dims& D, const Layout& Lo, const T* x, const T* w_r, const T* w1, const T* w2,
                         const T* w3, const T* dy, T* dx, T* dw_r, T* dw1, T* dw2, T* dw3, float* d_route_w,
                         char* ws, cudaStream_t st) {
  const int N = D.L / D.T;
  LORY_TRY(run_ffn_backward(D, Lo, ws, x, w1, w2, w3, dy, dx, dw1, dw2, dw3, st));
  ProfScope ps("router_backward", st);
  LORY_TRY(launch_router_backward<T>((const float*)(ws + Lo.dw_partial), Lo.n_slabs, (const float*)(ws + Lo.p),
                                     (const float*)(ws + Lo.h_bar), w_r, (float*)(ws + Lo.dw), d_route_w,
                                     (float*)(ws + Lo.dz), (float*)(ws + Lo.dh_bar), dw_r, D.B, N, D.d, D.E,
                                     ((D.flags & LORY_FLAG_PREFIX_ROUTING) ? 1 : 0) |
                                         ((D.flags & LORY_FLAG_FIRST_SEGMENT_GRAD) ? 2 : 0) |
                                         ((D.flags & LORY_FLAG_ACCUMULATE_GRADS) ? 4 : 0),
                                     st));
  prof_end(st);
  if (use_tc(D)) return tc_ffn_backward_dx(D, Lo, ws, (const float*)(ws + Lo.dh_bar), (bf16*)dx, st);
  prof_begin("add_pool_grad", st);
  LORY_TRY(launch_add_pool_grad<T>(dx, (const float*)(ws + Lo.dh_bar), D.B * D.L, D.T, D.d, st));
  return LORY_OK;
}

}  // namespace lory

using namespace lory;

extern "C" {

const char* lory_status_string(int status) {
  switch (status) {
    case LORY_OK: return "LORY_OK";
    case LORY_ERR_NULL: return "LORY_ERR_NULL: a required pointer is NULL";
    case LORY_ERR_SHAPE: return "LORY_ERR_SHAPE: bad dimension (need all >= 1, L % T == 0; bf16: d, f % 8 == 0, E <= 128)";
    case LORY_ERR_DTYPE: return "LORY_ERR_DTYPE: dtype must be LORY_FP32 or LORY_BF16";
    case LORY_ERR_WORKSPACE: return "LORY_ERR_WORKSPACE: workspace too small or misaligned";
    case LORY_ERR_ARCH: return "LORY_ERR_ARCH: device is not compute capability 10.x";
    case LORY_ERR_CUDA: return "LORY_ERR_CUDA: a CUDA call failed";
    case LORY_ERR_DEVICE_TIMEOUT: return "LORY_ERR_DEVICE_TIMEOUT: a bounded device-side wait expired";
    case LORY_ERR_TOO_LARGE: return "LORY_ERR_TOO_LARGE: problem exceeds the fixed scratch array of lory_route_noalloc";
    case LORY_ERR_DEBUG_BOUNDS: return "LORY_ERR_DEBUG_BOUNDS: a bounds check of the debug build fired";
    default: return "unknown lory_status";
  }
}

const char* lory_last_cuda_error(void) { return call_state().cuda_error; }

int lory_last_launch_count(void) { return call_state().launches; }

int lory_profile_enable(int on) {
  g_prof.on = on != 0;
  g_prof.n = 0;
  g_prof.open = false;
  return LORY_OK;
}

int lory_profile_read(int max_records, const char** labels, float* ms) {
  Prof& P = g_prof;
  int n = P.n < max_records ? P.n : max_records;
  for (int i = 0; i < n; ++i) {
    if (cudaEventSynchronize(P.ev[2 * i + 1]) != cudaSuccess) return LORY_ERR_CUDA;
    float t = 0.f;
    if (cudaEventElapsedTime(&t, P.ev[2 * i], P.ev[2 * i + 1]) != cudaSuccess) return LORY_ERR_CUDA;
    if (labels) labels[i] = P.label[i];
    if (ms) ms[i] = t;
  }
  return n;
}

int lory_moe_workspace_bytes(const lory_dims* dims, size_t* fwd_bytes, size_t* bwd_bytes) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  Layout Lo = make_layout(*dims);
  if (fwd_bytes) *fwd_bytes = Lo.fwd_end;
  if (bwd_bytes) *bwd_bytes = Lo.bwd_end;
  return LORY_OK;
}

static int check_ws(void* ws, size_t have, size_t need) {
  if (!ws) return LORY_ERR_NULL;
  if (((uintptr_t)ws & 255) != 0 || have < need) return LORY_ERR_WORKSPACE;
  return LORY_OK;
}

int lory_moe_forward(const lory_dims* dims, const void* x, const void* w_r, const void* w1, const void* w2,
                     const void* w3, void* y, float* route_w, float* route_p, void* workspace,
                     size_t workspace_bytes, void* cuda_stream) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  if (!x || !w_r || !w1 || !w2 || !w3 || !y || !route_w) return LORY_ERR_NULL;
  if (dims->flags & LORY_FLAG_REUSE_MERGED) return LORY_ERR_SHAPE;  // only lory_moe_ffn can reuse merged weights
  Layout Lo = make_layout(*dims);
  s = check_ws(workspace, workspace_bytes, Lo.fwd_end);
  if (s != LORY_OK) return s;
  s = check_device();
  if (s != LORY_OK) return s;
  call_state().launches = 0;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* ws = (char*)workspace;
  if (dims->dtype == LORY_FP32)
    return forward_impl<float>(*dims, Lo, (const float*)x, (const float*)w_r, (const float*)w1, (const float*)w2,
                               (const float*)w3, (float*)y, route_w, route_p, nullptr, ws, st);
  return forward_impl<bf16>(*dims, Lo, (const bf16*)x, (const bf16*)w_r, (const bf16*)w1, (const bf16*)w2,
                            (const bf16*)w3, (bf16*)y, route_w, route_p, nullptr, ws, st);
}

int lory_moe_ffn(const lory_dims* dims, const void* x, const float* route_w, const void* w1, const void* w2,
                 const void* w3, void* y, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  const bool reuse = (dims->flags & LORY_FLAG_REUSE_MERGED) != 0;
  if (!x || (!route_w && !reuse) || !w1 || !w2 || !w3 || !y) return LORY_ERR_NULL;
  Layout Lo = make_layout(*dims);
  s = check_ws(workspace, workspace_bytes, Lo.fwd_end);
  if (s != LORY_OK) return s;
  s = check_device();
  if (s != LORY_OK) return s;
  call_state().launches = 0;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* ws = (char*)workspace;
  if (dims->dtype == LORY_FP32)
    return forward_impl<float>(*dims, Lo, (const float*)x, nullptr, (const float*)w1, (const float*)w2,
                               (const float*)w3, (float*)y, nullptr, nullptr, route_w, ws, st);
  return forward_impl<bf16>(*dims, Lo, (const bf16*)x, nullptr, (const bf16*)w1, (const bf16*)w2, (const bf16*)w3,
                            (bf16*)y, nullptr, nullptr, route_w, ws, st);
}

int lory_moe_backward(const lory_dims* dims, const void* x, const void* w_r, const void* w1, const void* w2,
                      const void* w3, const void* dy, void* dx, void* dw_r, void* dw1, void* dw2, void* dw3,
                      float* d_route_w, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  if (!x || !w_r || !w1 || !w2 || !w3 || !dy || !dx || !dw_r || !dw1 || !dw2 || !dw3) return LORY_ERR_NULL;
  Layout Lo = make_layout(*dims);
  s = check_ws(workspace, workspace_bytes, Lo.bwd_end);
  if (s != LORY_OK) return s;
  s = check_device();
  if (s != LORY_OK) return s;
  call_state().launches = 0;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* ws = (char*)workspace;
  if (dims->dtype == LORY_FP32)
    return backward_impl<float>(*dims, Lo, (const float*)x, (const float*)w_r, (const float*)w1, (const float*)w2,
                                (const float*)w3, (const float*)dy, (float*)dx, (float*)dw_r, (float*)dw1,
                                (float*)dw2, (float*)dw3, d_route_w, ws, st);
  return backward_impl<bf16>(*dims, Lo, (const bf16*)x, (const bf16*)w_r, (const bf16*)w1, (const bf16*)w2,
                             (const bf16*)w3, (const bf16*)dy, (bf16*)dx, (bf16*)dw_r, (bf16*)dw1, (bf16*)dw2,
                             (bf16*)dw3, d_route_w, ws, st);
}

int lory_expert_utilization(const float* route_w, int S, int E, int* counts, void* cuda_stream) {
  if (!route_w || !counts) return LORY_ERR_NULL;
  if (S < 1 || E < 1 || E > 4096) return LORY_ERR_SHAPE;
  call_state().launches = 0;
  return launch_expert_utilization(route_w, S, E, counts, (cudaStream_t)cuda_stream);
}

int lory_moe_step_host_bytes(const lory_dims* dims, size_t* arena_bytes) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  if (!arena_bytes) return LORY_ERR_NULL;
  Layout Lo = make_layout(*dims);
  const size_t es = dims->dtype == LORY_BF16 ? 2 : 4;
  const size_t act = align_up((size_t)dims->B * dims->L * dims->d * es, 256);
  const size_t rw = align_up((size_t)dims->B * (dims->L / dims->T) * dims->E * 4, 256);
  *arena_bytes = 4 * act + rw + Lo.bwd_end;
  return LORY_OK;
}

int lory_moe_step_host(const lory_dims* dims, const void* x_host, const void* dy_host, const void* w_r,
                       const void* w1, const void* w2, const void* w3, void* y_host, void* dx_host,
                       float* route_w_host, void* dw_r, void* dw1, void* dw2, void* dw3, void* arena,
                       size_t arena_bytes, void* cuda_stream) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  if (!x_host || !dy_host || !y_host || !dx_host || !route_w_host) return LORY_ERR_NULL;
  size_t need = 0;
  lory_moe_step_host_bytes(dims, &need);
  s = check_ws(arena, arena_bytes, need);
  if (s != LORY_OK) return s;
  Layout Lo = make_layout(*dims);
  const size_t es = dims->dtype == LORY_BF16 ? 2 : 4;
  const size_t act_bytes = (size_t)dims->B * dims->L * dims->d * es;
  const size_t act = align_up(act_bytes, 256);
  const size_t rw_bytes = (size_t)dims->B * (dims->L / dims->T) * dims->E * 4;
  const size_t rw = align_up(rw_bytes, 256);
  char* a = (char*)arena;
  char* x_d = a;
  char* dy_d = a + act;
  char* y_d = a + 2 * act;
  char* dx_d = a + 3 * act;
  float* rw_d = (float*)(a + 4 * act);
  char* ws = a + 4 * act + rw;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // A second stream carries dY in while the forward runs and y out while the backward runs (one per host thread
  // and device: streams and events belong to the device that was current when they were created).
  struct Side {
    cudaStream_t side;
    cudaEvent_t ev_x, ev_dy, ev_fwd, ev_y;
  };
  static thread_local Side sides[kMaxDevices] = {};
  int dev = 0;
  LORY_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return LORY_ERR_CUDA;
  cudaStream_t& side = sides[dev].side;
  cudaEvent_t &ev_x = sides[dev].ev_x, &ev_dy = sides[dev].ev_dy, &ev_fwd = sides[dev].ev_fwd, &ev_y = sides[dev].ev_y;
  if (!side) {
    LORY_CUDA_OK(cudaStreamCreateWithFlags(&side, cudaStreamNonBlocking));
    LORY_CUDA_OK(cudaEventCreateWithFlags(&ev_x, cudaEventDisableTiming));
    LORY_CUDA_OK(cudaEventCreateWithFlags(&ev_dy, cudaEventDisableTiming));
    LORY_CUDA_OK(cudaEventCreateWithFlags(&ev_fwd, cudaEventDisableTiming));
    LORY_CUDA_OK(cudaEventCreateWithFlags(&ev_y, cudaEventDisableTiming));
  }
  LORY_CUDA_OK(cudaMemcpyAsync(x_d, x_host, act_bytes, cudaMemcpyHostToDevice, st));
  LORY_CUDA_OK(cudaEventRecord(ev_x, st));
  LORY_CUDA_OK(cudaStreamWaitEvent(side, ev_x, 0));  // also orders the side stream after earlier work on st
  LORY_CUDA_OK(cudaMemcpyAsync(dy_d, dy_host, act_bytes, cudaMemcpyHostToDevice, side));
  LORY_CUDA_OK(cudaEventRecord(ev_dy, side));
  s = lory_moe_forward(dims, x_d, w_r, w1, w2, w3, y_d, rw_d, nullptr, ws, Lo.bwd_end, cuda_stream);
  if (s != LORY_OK) return s;
  int fwd_launches = call_state().launches;
  LORY_CUDA_OK(cudaEventRecord(ev_fwd, st));
  LORY_CUDA_OK(cudaStreamWaitEvent(side, ev_fwd, 0));
  LORY_CUDA_OK(cudaMemcpyAsync(y_host, y_d, act_bytes, cudaMemcpyDeviceToHost, side));
  LORY_CUDA_OK(cudaMemcpyAsync(route_w_host, rw_d, rw_bytes, cudaMemcpyDeviceToHost, side));
  LORY_CUDA_OK(cudaEventRecord(ev_y, side));
  LORY_CUDA_OK(cudaStreamWaitEvent(st, ev_dy, 0));
  s = lory_moe_backward(dims, x_d, w_r, w1, w2, w3, dy_d, dx_d, dw_r, dw1, dw2, dw3, nullptr, ws, Lo.bwd_end,
                        cuda_stream);
  if (s != LORY_OK) return s;
  call_state().launches += fwd_launches;
  LORY_CUDA_OK(cudaMemcpyAsync(dx_host, dx_d, act_bytes, cudaMemcpyDeviceToHost, st));
  LORY_CUDA_OK(cudaStreamWaitEvent(st, ev_y, 0));
  LORY_CUDA_OK(cudaStreamSynchronize(st));
  return LORY_OK;
}

// ---- the layer inside a pre-norm residual block ---------------------------------------------------
namespace {
struct BlockLayout {
  size_t x_hat, inv, layer, dxh, slab, fwd_end, bwd_end;
  int n_slabs;
};
BlockLayout make_block_layout(const lory_dims& D, const Layout& Lo) {
  BlockLayout b;
  const size_t tok = (size_t)D.B * D.L, es = D.dtype == LORY_BF16 ? 2 : 4;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  b.x_hat = take(tok * D.d * es);
  b.inv = take(tok * 4);
  b.layer = off;
  b.fwd_end = off + Lo.fwd_end;
  off += Lo.bwd_end;
  b.n_slabs = block_norm_slabs((long)tok);
  b.dxh = take(tok * D.d * es);
  b.slab = take((size_t)b.n_slabs * D.d * 4);
  b.bwd_end = off;
  return b;
}
}  // namespace

int lory_block_workspace_bytes(const lory_dims* dims, size_t* forward_bytes, size_t* backward_bytes) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  Layout Lo = make_layout(*dims);
  BlockLayout b = make_block_layout(*dims, Lo);
  if (forward_bytes) *forward_bytes = b.fwd_end;
  if (backward_bytes) *backward_bytes = b.bwd_end;
  return LORY_OK;
}

int lory_block_forward(const lory_dims* dims, const void* x, const void* gamma, float eps, const void* w_r,
                       const void* w1, const void* w2, const void* w3, void* y, float* route_w, float* route_p,
                       void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  if (!x || !gamma || !w_r || !w1 || !w2 || !w3 || !y || !route_w) return LORY_ERR_NULL;
  if (dims->flags & LORY_FLAG_REUSE_MERGED) return LORY_ERR_SHAPE;
  if (!(eps >= 0.f)) return LORY_ERR_SHAPE;
  Layout Lo = make_layout(*dims);
  BlockLayout b = make_block_layout(*dims, Lo);
  s = check_ws(workspace, workspace_bytes, b.fwd_end);
  if (s != LORY_OK) return s;
  s = check_device();
  if (s != LORY_OK) return s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* ws = (char*)workspace;
  const long tok = (long)dims->B * dims->L;
  call_state().launches = 0;
  {
    ProfScope ps("rmsnorm", st);
    if (dims->dtype == LORY_FP32)
      LORY_TRY(launch_rmsnorm<float>((const float*)x, (const float*)gamma, (float*)(ws + b.x_hat),
                                     (float*)(ws + b.inv), tok, dims->d, eps, st));
    else
      LORY_TRY(launch_rmsnorm<bf16>((const bf16*)x, (const bf16*)gamma, (bf16*)(ws + b.x_hat), (float*)(ws + b.inv),
                                    tok, dims->d, eps, st));
  }
  // the layer on x_hat, with the block's input as the residual of its output
  char* lws = ws + b.layer;
  if (dims->dtype == LORY_FP32)
    return forward_impl<float>(*dims, Lo, (const float*)(ws + b.x_hat), (const float*)w_r, (const float*)w1,
                               (const float*)w2, (const float*)w3, (float*)y, route_w, route_p, nullptr, lws, st,
                               (const float*)x);
  return forward_impl<bf16>(*dims, Lo, (const bf16*)(ws + b.x_hat), (const bf16*)w_r, (const bf16*)w1, (const bf16*)w2,
                            (const bf16*)w3, (bf16*)y, route_w, route_p, nullptr, lws, st, (const bf16*)x);
}

int lory_block_backward(const lory_dims* dims, const void* x, const void* gamma, const void* w_r, const void* w1,
                        const void* w2, const void* w3, const void* dy, void* dx, void* dgamma, void* dw_r,
                        void* dw1, void* dw2, void* dw3, float* d_route_w, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  if (!x || !gamma || !w_r || !w1 || !w2 || !w3 || !dy || !dx || !dgamma || !dw_r || !dw1 || !dw2 || !dw3)
    return LORY_ERR_NULL;
  Layout Lo = make_layout(*dims);
  BlockLayout b = make_block_layout(*dims, Lo);
  s = check_ws(workspace, workspace_bytes, b.bwd_end);
  if (s != LORY_OK) return s;
  s = check_device();
  if (s != LORY_OK) return s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char* ws = (char*)workspace;
  const long tok = (long)dims->B * dims->L;
  s = lory_moe_backward(dims, ws + b.x_hat, w_r, w1, w2, w3, dy, ws + b.dxh, dw_r, dw1, dw2, dw3, d_route_w,
                        ws + b.layer, Lo.bwd_end, cuda_stream);
  if (s != LORY_OK) return s;
  const int acc = (dims->flags & LORY_FLAG_ACCUMULATE_GRADS) ? 1 : 0;
  {
    ProfScope ps("rmsnorm_backward", st);
    if (dims->dtype == LORY_FP32)
      LORY_TRY(launch_rmsnorm_backward<float>((const float*)x, (const float*)gamma, (const float*)(ws + b.inv),
                                              (const float*)(ws + b.dxh), (const float*)dy, (float*)dx,
                                              (float*)dgamma, (float*)(ws + b.slab), tok, dims->d, acc, st));
    else
      LORY_TRY(launch_rmsnorm_backward<bf16>((const bf16*)x, (const bf16*)gamma, (const float*)(ws + b.inv),
                                             (const bf16*)(ws + b.dxh), (const bf16*)dy, (bf16*)dx, (bf16*)dgamma,
                                             (float*)(ws + b.slab), tok, dims->d, acc, st));
  }
  return LORY_OK;
}

// ---- two-slot host pipeline ---------------------------------------------------------------------
namespace {
struct HostPipe {
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t x_in[2] = {}, dy_in[2] = {}, fwd[2] = {}, bwd[2] = {}, landed[2] = {};
  bool used[2] = {false, false};
};
// One pipeline per host thread and device.
HostPipe* host_pipe() {
  static thread_local HostPipe hp[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  return &hp[dev];
}
int host_pipe_init(HostPipe& hp) {
  if (hp.in) return LORY_OK;
  LORY_CUDA_OK(cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking));
  LORY_CUDA_OK(cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking));
  for (int i = 0; i < 2; ++i) {
    LORY_CUDA_OK(cudaEventCreateWithFlags(&hp.x_in[i], cudaEventDisableTiming));
    LORY_CUDA_OK(cudaEventCreateWithFlags(&hp.dy_in[i], cudaEventDisableTiming));
    LORY_CUDA_OK(cudaEventCreateWithFlags(&hp.fwd[i], cudaEventDisableTiming));
    LORY_CUDA_OK(cudaEventCreateWithFlags(&hp.bwd[i], cudaEventDisableTiming));
    LORY_CUDA_OK(cudaEventCreateWithFlags(&hp.landed[i], cudaEventDisableTiming));
  }
  return LORY_OK;
}
}  // namespace

int lory_moe_step_host_pipeline_bytes(const lory_dims* dims, size_t* arena_bytes) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  if (!arena_bytes) return LORY_ERR_NULL;
  Layout Lo = make_layout(*dims);
  const size_t es = dims->dtype == LORY_BF16 ? 2 : 4;
  const size_t act = align_up((size_t)dims->B * dims->L * dims->d * es, 256);
  const size_t rw = align_up((size_t)dims->B * (dims->L / dims->T) * dims->E * 4, 256);
  *arena_bytes = 2 * (4 * act + rw) + Lo.bwd_end;  // per slot: x, dY, y, dX, routing weights; one workspace
  return LORY_OK;
}

int lory_moe_step_host_enqueue(const lory_dims* dims, int slot, const void* x_host, const void* dy_host,
                               const void* w_r, const void* w1, const void* w2, const void* w3, void* y_host,
                               void* dx_host, float* route_w_host, void* dw_r, void* dw1, void* dw2, void* dw3,
                               void* arena, size_t arena_bytes, void* cuda_stream) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  if (slot != 0 && slot != 1) return LORY_ERR_SHAPE;
  if (!x_host || !dy_host || !y_host || !dx_host || !route_w_host) return LORY_ERR_NULL;
  size_t need = 0;
  lory_moe_step_host_pipeline_bytes(dims, &need);
  s = check_ws(arena, arena_bytes, need);
  if (s != LORY_OK) return s;
  HostPipe* hpp = host_pipe();
  if (!hpp) return LORY_ERR_CUDA;
  HostPipe& hp = *hpp;
  s = host_pipe_init(hp);
  if (s != LORY_OK) return s;
  Layout Lo = make_layout(*dims);
  const size_t es = dims->dtype == LORY_BF16 ? 2 : 4;
  const size_t act_bytes = (size_t)dims->B * dims->L * dims->d * es;
  const size_t act = align_up(act_bytes, 256);
  const size_t rw_bytes = (size_t)dims->B * (dims->L / dims->T) * dims->E * 4;
  const size_t rw = align_up(rw_bytes, 256);
  char* a = (char*)arena + (size_t)slot * (4 * act + rw);
  char* x_d = a;
  char* dy_d = a + act;
  char* y_d = a + 2 * act;
  char* dx_d = a + 3 * act;
  float* rw_d = (float*)(a + 4 * act);
  char* ws = (char*)arena + 2 * (4 * act + rw);
  cudaStream_t st = (cudaStream_t)cuda_stream;

  // copy-in stream: this slot's inputs may be overwritten once the backward that read them has finished
  if (hp.used[slot]) LORY_CUDA_OK(cudaStreamWaitEvent(hp.in, hp.bwd[slot], 0));
  LORY_CUDA_OK(cudaMemcpyAsync(x_d, x_host, act_bytes, cudaMemcpyHostToDevice, hp.in));
  LORY_CUDA_OK(cudaEventRecord(hp.x_in[slot], hp.in));
  LORY_CUDA_OK(cudaMemcpyAsync(dy_d, dy_host, act_bytes, cudaMemcpyHostToDevice, hp.in));
  LORY_CUDA_OK(cudaEventRecord(hp.dy_in[slot], hp.in));

  // compute stream: needs x; must not overwrite this slot's outputs before their last copy-out has read them
  LORY_CUDA_OK(cudaStreamWaitEvent(st, hp.x_in[slot], 0));
  if (hp.used[slot]) LORY_CUDA_OK(cudaStreamWaitEvent(st, hp.landed[slot], 0));
  s = lory_moe_forward(dims, x_d, w_r, w1, w2, w3, y_d, rw_d, nullptr, ws, Lo.bwd_end, cuda_stream);
  if (s != LORY_OK) return s;
  const int fwd_launches = call_state().launches;
  LORY_CUDA_OK(cudaEventRecord(hp.fwd[slot], st));
  LORY_CUDA_OK(cudaStreamWaitEvent(st, hp.dy_in[slot], 0));
  s = lory_moe_backward(dims, x_d, w_r, w1, w2, w3, dy_d, dx_d, dw_r, dw1, dw2, dw3, nullptr, ws, Lo.bwd_end,
                        cuda_stream);
  if (s != LORY_OK) return s;
  call_state().launches += fwd_launches;
  LORY_CUDA_OK(cudaEventRecord(hp.bwd[slot], st));

  // copy-out stream: y and the routing weights after the forward, dX after the backward
  LORY_CUDA_OK(cudaStreamWaitEvent(hp.out, hp.fwd[slot], 0));
  LORY_CUDA_OK(cudaMemcpyAsync(y_host, y_d, act_bytes, cudaMemcpyDeviceToHost, hp.out));
  LORY_CUDA_OK(cudaMemcpyAsync(route_w_host, rw_d, rw_bytes, cudaMemcpyDeviceToHost, hp.out));
  LORY_CUDA_OK(cudaStreamWaitEvent(hp.out, hp.bwd[slot], 0));
  LORY_CUDA_OK(cudaMemcpyAsync(dx_host, dx_d, act_bytes, cudaMemcpyDeviceToHost, hp.out));
  LORY_CUDA_OK(cudaEventRecord(hp.landed[slot], hp.out));
  hp.used[slot] = true;
  return LORY_OK;
}

int lory_moe_step_host_wait(int slot) {
  if (slot != 0 && slot != 1) return LORY_ERR_SHAPE;
  HostPipe* hpp = host_pipe();
  if (!hpp) return LORY_ERR_CUDA;
  HostPipe& hp = *hpp;
  if (!hp.in || !hp.used[slot]) return LORY_OK;  // nothing was enqueued on this slot
  LORY_CUDA_OK(cudaEventSynchronize(hp.landed[slot]));
  return LORY_OK;
}

int lory_selftest_bounded_wait(const lory_dims* dims, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  Layout Lo = make_layout(*dims);
  s = check_ws(workspace, workspace_bytes, Lo.fwd_end);
  if (s != LORY_OK) return s;
  s = check_device();
  if (s != LORY_OK) return s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  LORY_CUDA_OK(cudaMemsetAsync((char*)workspace + Lo.status, 0, 256, st));
  return tc_bounded_wait_selftest((uint32_t*)((char*)workspace + Lo.status), st);
}

int lory_check_status(const lory_dims* dims, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  Layout Lo = make_layout(*dims);
  s = check_ws(workspace, workspace_bytes, Lo.fwd_end);
  if (s != LORY_OK) return s;
  uint32_t word = 0;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  LORY_CUDA_OK(cudaMemcpyAsync(&word, (char*)workspace + Lo.status, 4, cudaMemcpyDeviceToHost, st));
  LORY_CUDA_OK(cudaStreamSynchronize(st));
  if (word & STATUS_DEBUG_BOUNDS) return LORY_ERR_DEBUG_BOUNDS;
  return word == 0 ? LORY_OK : LORY_ERR_DEVICE_TIMEOUT;
}

int lory_debug_build(void) { return dbg::kOn ? 1 : 0; }

int lory_selftest_debug_bounds(const lory_dims* dims, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int s = check_dims(dims);
  if (s != LORY_OK) return s;
  Layout Lo = make_layout(*dims);
  s = check_ws(workspace, workspace_bytes, Lo.fwd_end);
  if (s != LORY_OK) return s;
  s = check_device();
  if (s != LORY_OK) return s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  LORY_CUDA_OK(cudaMemsetAsync((char*)workspace + Lo.status, 0, 256, st));
  return tc_debug_bounds_selftest((uint32_t*)((char*)workspace + Lo.status), st);
}

}  // extern "C"
