// Host side of the tensor-core pipeline (bf16 mode): tensor maps and the order of the GEMMs.
//
//   forward : split w into bf16 hi+lo  ->  merge  ->  G,U,H = SwiGLU(X Wbar1^T, X Wbar3^T)  ->  Y = H Wbar2^T
//   backward: dH = dY Wbar2 (+ SwiGLU backward in the epilogue)  ->  dWbar2 = dY^T H, dWbar1 = dG^T X,
//             dWbar3 = dU^T X  ->  dW_e = w^T dWbar and dw partials (one pass)  ->  [router backward]  ->
//             dX = dG Wbar1 + dU Wbar3 + dh_bar / T
//
// The merged weights Wbar_k and their gradients dWbar_k are kept in a blocked layout: a per-segment
// matrix [R, C] is stored as [ceil(R/64)][ceil(C/64)][S][64][64], so that (a) every 64 x 64 block a GEMM
// needs from one segment is one contiguous 8 KB piece and (b) the kernels that sweep all segments at a
// fixed parameter position (merge, merge adjoint) touch one contiguous S x 8 KB region per block instead
// of S rows that are megabytes apart.
#include "tc.cuh"

#include <cuda.h>
#include <stdio.h>
#include <stdlib.h>

#include "gemm_tc.cuh"
#include "merge_tc.cuh"
#include "stage2_tc.cuh"
#include "wgrad_tc.cuh"

namespace lory {

// ---------------------------------------------------------------------------------------
// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda).
// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !p) {
      note_cuda_error(e != cudaSuccess ? e : cudaErrorUnknown, "cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)");
      return nullptr;
    }
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 3-D bf16 tensor map: dims (inner, rows, groups), strides in elements, box (64, box_rows, 1),
// 128-byte swizzle, out-of-bounds elements read as zero.
static int make_map(CUtensorMap* m, const void* base, uint64_t inner, uint64_t rows, uint64_t groups,
                    uint64_t row_stride, uint64_t group_stride, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return LORY_ERR_CUDA;
  cuuint64_t dims[3] = {inner, rows, groups};
  cuuint64_t strides[2] = {row_stride * 2, (groups > 1 ? group_stride : rows * row_stride) * 2};
  cuuint32_t box[3] = {64, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    CallState& s = call_state();
    snprintf(s.cuda_error, sizeof(s.cuda_error),
             "cuTensorMapEncodeTiled failed with CUresult %d (inner %llu rows %llu groups %llu)", (int)r,
             (unsigned long long)inner, (unsigned long long)rows, (unsigned long long)groups);
    return LORY_ERR_CUDA;
  }
  return LORY_OK;
}

// Generic tiled bf16 tensor map with the 128-byte swizzle; strides in elements for dims 1..rank-1.
static int make_map_nd(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_el,
                       const uint32_t* box) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return LORY_ERR_CUDA;
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], es[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) st[i] = strides_el[i] * 2;
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    CallState& s = call_state();
    snprintf(s.cuda_error, sizeof(s.cuda_error), "cuTensorMapEncodeTiled (rank %d) failed with CUresult %d", rank, (int)r);
    return LORY_ERR_CUDA;
  }
  return LORY_OK;
}

// Blocked per-segment matrix [R, C] of S segments: dims (col in block, row in block, segment, col block, row block).
static int make_blocked_map(CUtensorMap* m, const void* base, int R, int C, int S, uint32_t box_rin, uint32_t box_seg,
                            uint32_t box_cb, uint32_t box_rb) {
  const uint64_t Rb = (R + 63) / 64, Cb = (C + 63) / 64;
  const uint64_t dims[5] = {64, 64, (uint64_t)S, Cb, Rb};
  const uint64_t strides[4] = {64, 4096, (uint64_t)S * 4096, Cb * S * 4096};
  const uint32_t box[5] = {64, box_rin, box_seg, box_cb, box_rb};
  return make_map_nd(m, base, 5, dims, strides, box);
}

// Expert matrix W_k [E, R, C] seen as (C, E, R): a box is 64 columns x box_e experts of one row.
// e_stride / row_stride (elements) describe a sub-rectangle of a larger [E, R0, C0] tensor; 0 = dense [E, R, C].
static int make_expert_map(CUtensorMap* m, const void* base, int R, int C, int E, uint32_t box_e, uint64_t e_stride = 0,
                           uint64_t row_stride = 0) {
  const uint64_t dims[3] = {(uint64_t)C, (uint64_t)E, (uint64_t)R};
  const uint64_t strides[2] = {e_stride ? e_stride : (uint64_t)R * C, row_stride ? row_stride : (uint64_t)C};
  const uint32_t box[3] = {64, box_e, 1};
  return make_map_nd(m, base, 3, dims, strides, box);
}

// Per-device state is kept per device ordinal: a process may drive several GPUs.
static const int kMaxDevices = 64;
static int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
  return dev;
}

static int sm_count() {
  static int n[kMaxDevices];
  const int dev = current_device();
  if (!n[dev]) {
    if (cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n[dev] <= 0)
      n[dev] = 148;
  }
  return n[dev];
}

// cudaFuncAttributeMaxDynamicSharedMemorySize belongs to the (function, device) pair: set it once on every
// device that launches the kernel.
template <typename K>
static int allow_dynamic_smem(K kern, int bytes, bool (&done)[kMaxDevices]) {
  const int dev = current_device();
  if (!done[dev]) {
    LORY_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    done[dev] = true;
  }
  return LORY_OK;
}

static const int kMaxSmem = 227 * 1024 - 512;  // dynamic shared memory we may ask for (static use is < 512 B)

template <bool A_MN, bool B_MN, int BN, int MODE, int EPI, bool B_BLK = false, bool C_BLK = false, int CTAS = 1,
          int AROWS = 128>
static int launch_tc(const char* label, const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& b0,
                     const CUtensorMap& b1, const CUtensorMap& c0, const CUtensorMap& c1, const CUtensorMap& c2,
                     TcGemmParams p, cudaStream_t st, const CUtensorMap* e0 = nullptr,
                     const CUtensorMap* e1 = nullptr) {
  constexpr int TILE_N = (MODE == MODE_DUALB) ? BN / 2 : BN;
  using Tile = TcTile<BN, EPI, CTAS, AROWS>;
  p.m_tiles = (int)ceil_div(p.M, 128 * CTAS);
  p.n_tiles = (int)ceil_div(p.N, TILE_N);
  const long tiles = (long)p.m_tiles * p.n_tiles * p.groups;
  if (tiles <= 0) return LORY_OK;
  if (tiles > 0x7fffffffL) return LORY_ERR_SHAPE;
  auto kern = tc_gemm_kernel<A_MN, B_MN, BN, MODE, EPI, B_BLK, C_BLK, CTAS, AROWS>;
  static bool attr_set[kMaxDevices];
  LORY_TRY(allow_dynamic_smem(kern, Tile::SMEM_BYTES, attr_set));
  const int slots = sm_count() / CTAS;  // persistent CTAs (or CTA pairs)
  const int grid = CTAS * (int)(tiles < slots ? tiles : slots);
  const CUtensorMap& me0 = e0 ? *e0 : c0;
  const CUtensorMap& me1 = e1 ? *e1 : c0;
  ProfScope ps(label, st);
  if (CTAS == 1) {
    kern<<<grid, 192, Tile::SMEM_BYTES, st>>>(a0, a1, b0, b1, c0, c1, c2, me0, me1, p);
  } else {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(192);
    cfg.dynamicSmemBytes = Tile::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    LORY_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, a0, a1, b0, b1, c0, c1, c2, me0, me1, p));
  }
  LORY_AFTER_LAUNCH();
  return LORY_OK;
}

// One per-segment weight gradient C_g = A_g^T B_g (K = T): the resident-operand kernel for CTA-pair tiles with short
// segments (its strips run along the dimension with more tiles), else the grouped GEMM.  Measured on one GPU
// (d = 2048, f = 5504, E = 32; three launches): T = 64: 3.69 -> 3.53 ms, T = 128: 1.99 -> 1.82 ms; at T = 256 the two
// kernels tie (d = 1024, f = 2752: 0.591 vs 0.600 ms; d = 2048: 1.14 vs 1.11 ms) and the grouped GEMM stays.
static int launch_wgrad(const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& c, int M, int N, int K, int groups,
                        bool pairs, uint32_t* status, cudaStream_t st) {
  if (pairs && K <= 128) {
    WgradParams p = {};
    p.M = M; p.N = N; p.K = K; p.groups = groups; p.status = status;
    p.m_tiles = (int)ceil_div(M, 256);
    p.n_tiles = (int)ceil_div(N, 256);
    const bool res_a = p.n_tiles >= p.m_tiles;
    const long strips = (long)(res_a ? p.m_tiles : p.n_tiles) * groups;
    if (strips <= 0) return LORY_OK;
    if (strips > 0x7fffffffL) return LORY_ERR_SHAPE;
    static bool attr_set[2][kMaxDevices];
    LORY_TRY(allow_dynamic_smem(wgrad_kernel<false>, WgradTile::SMEM_BYTES, attr_set[0]));
    LORY_TRY(allow_dynamic_smem(wgrad_kernel<true>, WgradTile::SMEM_BYTES, attr_set[1]));
    const int slots = sm_count() / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)(strips < slots ? strips : slots));
    cfg.blockDim = dim3(192);
    cfg.dynamicSmemBytes = WgradTile::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    ProfScope ps("wgrad", st);
    if (res_a) LORY_CUDA_OK(cudaLaunchKernelEx(&cfg, wgrad_kernel<true>, a, b, c, p));
    else LORY_CUDA_OK(cudaLaunchKernelEx(&cfg, wgrad_kernel<false>, a, b, c, p));
    LORY_AFTER_LAUNCH();
    return LORY_OK;
  }
  TcGemmParams p = {};
  p.groups = groups; p.K = K; p.M = M; p.N = N; p.status = status;
  if (pairs) return launch_tc<true, true, 256, MODE_PLAIN, EPI_BF16, false, true, 2>("wgrad", a, a, b, b, c, c, c, p, st);
  return launch_tc<true, true, 256, MODE_PLAIN, EPI_BF16, false, true>("wgrad", a, a, b, b, c, c, c, p, st);
}

// ---------------------------------------------------------------------------------------
// w (float [S, E]) -> hi, lo (bf16 [S, Epad]) with hi + lo == w to ~16 bits; padding columns zero.
// ---------------------------------------------------------------------------------------
static int e_pad(const lory_dims& D) { return (D.E + 7) / 8 * 8; }
static int e_pad16(const lory_dims& D) { return (D.E + 15) / 16 * 16; }

// Routing weights as bf16 hi + lo tables [S, Epad].  With E <= 32 also one [S, 192] table `comb` holding, in groups
// of 32 columns, [hi | lo | hi | hi | lo | lo] (zero where e >= E): the merge adjoint reads columns 0..63 or
// 64..191 of it; the grid then covers S x 192.
__global__ void split_w_kernel(const float* __restrict__ w, bf16* __restrict__ hi, bf16* __restrict__ lo,
                               bf16* __restrict__ comb, int S, int E, int Epad) {
  const int width = E <= 32 ? 192 : Epad;
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= S * width) return;
  const int s = i / width, c = i - s * width;
  const int e = E <= 32 ? (c & 31) : c;
  const float v = e < E ? w[(size_t)s * E + e] : 0.f;
  const bf16 h = __float2bfloat16_rn(v);
  const bf16 l = __float2bfloat16_rn(v - __bfloat162float(h));
  if (E <= 32) {
    const int part = c >> 5;
    comb[i] = (part == 0 || part == 2 || part == 3) ? h : l;
    if (c >= Epad) return;
  }
  hi[(size_t)s * Epad + e] = h;
  lo[(size_t)s * Epad + e] = l;
}

size_t tc_w_split_bytes(const lory_dims& D) {
  const size_t S = (size_t)D.B * (D.L / D.T);
  return 2 * align_up(S * e_pad(D) * 2, 256) + align_up(S * 192 * 2, 256);
}

// The merge and merge-adjoint kernels keep the routing weights of the segments they work on resident in shared
// memory: at most 256 segments per launch (more segments take more launches) and at most 64 experts (more
// experts run on the plain-FMA path).
bool tc_supported(const lory_dims& D) {
  return D.E <= 64;
}

size_t tc_blocked_elems(const lory_dims& D, int R, int C) {
  const size_t S = (size_t)D.B * (D.L / D.T);
  return (size_t)((R + 63) / 64) * ((C + 63) / 64) * S * 4096;
}

// Two-row tiles (64 columns of rows r, r + 1) pay off only with very few segments, where the expert traffic dominates
// (S = 16: 1.67 -> 1.56 ms at d = 2048, f = 5504, E = 32); at S >= 64 they measure the same as 128 columns of one row,
// and at S = 32 the three-block tiles below are better (1.42 -> 1.34 ms).
static int stage2_rpt_shift(const lory_dims& D) {
  return D.B * (D.L / D.T) <= 16 ? 1 : 0;
}
// One of the (up to three) parameter rectangles a launch of the merge adjoint covers: a whole expert matrix, or a
// sub-rectangle of one whose per-segment gradients sit in a buffer of their own.  R == 0: not part of the launch.
struct AdjPiece {
  const bf16* dsrc;  // blocked per-segment gradients of the rectangle [R, C]
  const bf16* wsrc;  // experts: first element of the rectangle inside W_k
  bf16* ddst;        // expert gradients: first element of the rectangle inside dW_k
  int R, C;
  uint64_t e_stride, row_stride;  // elements between experts / rows of W_k and dW_k
};
// Tiles of three 64-column blocks instead of two where both weight halves go through the tensor core (E <= 32,
// 17..64 segments): the first product then needs its MMAs once per 192 columns instead of once per 128, and the MMA
// count is what a tile waits for there (d = 2048, f = 5504: E = 16, S = 64: 1.54 -> 1.34 ms; E = 32, S = 64: 1.64 -> 1.58;
// S = 32: 1.42 -> 1.34).  Four blocks would not fit TMEM beside the double buffering.
static int stage2_ncb(const lory_dims& D) {
  const int S = D.B * (D.L / D.T);
  return (D.E <= 32 && S > 16 && S <= 64) ? 3 : 2;
}
static void stage2_tiles(const lory_dims& D, const int R[3], const int C[3], int ctiles[3], int tile_end[3]) {
  const int rsh = stage2_rpt_shift(D);
  const int width = rsh ? 64 : stage2_ncb(D) * 64;   // columns per tile
  int acc = 0;
  for (int k = 0; k < 3; ++k) {
    ctiles[k] = C[k] > 0 ? (C[k] + width - 1) / width : 1;
    acc += (((R[k] + 63) / 64 * 64) >> rsh) * ctiles[k];  // whole row blocks: the rows past R[k] read zeros and store nothing
    tile_end[k] = acc;
  }
}
static int stage2_grid(const lory_dims& D) {
  const int R[3] = {D.f, D.f, D.d}, C[3] = {D.d, D.d, D.f};
  int ct[3], te[3];
  stage2_tiles(D, R, C, ct, te);
  return te[2] < sm_count() ? te[2] : sm_count();
}

int tc_dw_slabs(const lory_dims& D) { return stage2_grid(D); }

// ---------------------------------------------------------------------------------------
// Chunked adjoint (LORY_FLAG_CHUNKED_ADJOINT): the per-segment weight gradients of one rectangle of one expert
// matrix at a time (all segments), written by the weight-gradient GEMM into a buffer small enough to stay in L2
// and consumed from there by the merge adjoint before the next rectangle overwrites it.
// ---------------------------------------------------------------------------------------
static size_t adjoint_budget_bytes() {
  // read on every call: the workspace query and the backward must see the same value, nothing else is assumed
  if (const char* ev = getenv("LORY_ADJOINT_CHUNK_MB")) {
    const long mb = atol(ev);
    if (mb > 0) return (size_t)mb << 20;
  }
  static size_t bytes[kMaxDevices];
  const int dev = current_device();
  if (!bytes[dev]) {
    int l2 = 0;
    if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess || l2 <= 0) l2 = 64 << 20;
    bytes[dev] = (size_t)l2 / 2;  // what a producer can leave in L2 for the consumer that follows it
  }
  return bytes[dev];
}
struct AdjChunks {
  int rows;     // rows of a rectangle (256: one row of CTA-pair tiles; fewer for small matrices)
  int cols[3];  // columns of a rectangle of W1 / W3 / W2, a multiple of 256 (or the whole width)
};
static AdjChunks adjoint_chunks(const lory_dims& D) {
  const size_t S = (size_t)D.B * (D.L / D.T);
  const int R[3] = {D.f, D.f, D.d}, C[3] = {D.d, D.d, D.f};
  AdjChunks a;
  a.rows = 256;
  const size_t per_col = (size_t)a.rows * S * 2;  // bytes of one column of a rectangle over all segments
  long cmax = (long)(adjoint_budget_bytes() / per_col) / 256 * 256;
  if (cmax < 256) cmax = 256;
  for (int k = 0; k < 3; ++k) {
    (void)R;
    const long n = ceil_div(C[k], cmax);
    a.cols[k] = (int)(ceil_div(ceil_div(C[k], n), 256) * 256);
  }
  return a;
}
size_t tc_adjoint_ring_elems(const lory_dims& D) {
  const AdjChunks a = adjoint_chunks(D);
  const size_t S = (size_t)D.B * (D.L / D.T);
  size_t best = 0;
  for (int k = 0; k < 3; ++k) {
    const size_t e = (size_t)(a.rows / 64) * (size_t)((a.cols[k] + 63) / 64) * S * 4096;
    if (e > best) best = e;
  }
  return best;
}

// CTA pairs (256-row tiles) pay off when a segment fills them.
static bool use_pairs(int rows) { return rows % 256 == 0; }

struct WsPtrs {
  uint32_t* status;
  const float* w;
  bf16 *w_hi, *w_lo, *w_comb, *wbar1, *wbar3, *wbar2, *G, *U, *H, *dG, *dU, *dwbar1, *dwbar3, *dwbar2;
  float* dw_partial;
};
static WsPtrs ws_ptrs(const lory_dims& D, const Layout& Lo, char* ws) {
  const int S = D.B * (D.L / D.T);
  WsPtrs q;
  q.status = (uint32_t*)(ws + Lo.status);
  q.w = (const float*)(ws + Lo.w);
  q.w_hi = (bf16*)(ws + Lo.w_split);
  q.w_lo = (bf16*)(ws + Lo.w_split + align_up((size_t)S * e_pad(D) * 2, 256));
  q.w_comb = (bf16*)(ws + Lo.w_split + 2 * align_up((size_t)S * e_pad(D) * 2, 256));
  q.wbar1 = (bf16*)(ws + Lo.wbar1); q.wbar3 = (bf16*)(ws + Lo.wbar3); q.wbar2 = (bf16*)(ws + Lo.wbar2);
  q.G = (bf16*)(ws + Lo.G); q.U = (bf16*)(ws + Lo.U); q.H = (bf16*)(ws + Lo.H);
  q.dG = (bf16*)(ws + Lo.dG); q.dU = (bf16*)(ws + Lo.dU);
  q.dwbar1 = (bf16*)(ws + Lo.dwbar1); q.dwbar3 = (bf16*)(ws + Lo.dwbar3); q.dwbar2 = (bf16*)(ws + Lo.dwbar2);
  q.dw_partial = (float*)(ws + Lo.dw_partial);
  return q;
}

// Wbar_k (blocked) = (w_hi + w_lo) . W_k for the three matrices in one launch      (Eq. 2)
static int launch_merge(const lory_dims& D, const WsPtrs& q, const bf16* const src[3], bf16* const dst[3],
                        cudaStream_t st) {
  const int S = D.B * (D.L / D.T), E = D.E, Ep = e_pad(D);
  const int R[3] = {D.f, D.f, D.d}, C[3] = {D.d, D.d, D.f};
  MergeMaps maps;
  MergeParams p = {};
  const int S_launch = S < 256 ? S : 256;  // the routing weights of at most 256 segments stay in shared memory
  p.S = S_launch; p.E = E; p.Epad16 = e_pad16(D); p.s_tiles = (S_launch + 127) / 128; p.status = q.status;
  p.dup = S <= 32 ? 2 : (S <= 64 ? 1 : 0);
  // Tiles of 4 rows x 64 columns: a segment's four 128-byte output pieces of one tile are neighbours in its 64 x 64
  // block (512 contiguous bytes).  Measured against 1 x 256 and 2 x 128: C3 0.546 / 0.520 / 0.524 ms (1, 2, 4 rows),
  // C4 1.064 / 1.036 / 0.996 ms.
  p.rpt_shift = 2;
  const uint32_t w_box = p.dup == 2 ? 32u : (p.dup ? 64u : 128u);
  LORY_TRY(make_map(&maps.w_hi, q.w_hi, Ep, S, 1, Ep, 0, w_box));
  LORY_TRY(make_map(&maps.w_lo, q.w_lo, Ep, S, 1, Ep, 0, w_box));
  int acc = 0;
  for (int k = 0; k < 3; ++k) {
    LORY_TRY(make_expert_map(&maps.theta[k], src[k], R[k], C[k], E, p.Epad16));
    LORY_TRY(make_blocked_map(&maps.out[k], dst[k], R[k], C[k], S, 1, S < 32 ? (uint32_t)S : 32u, 1, 1));  // no box rows past the segments
    p.ctiles[k] = (C[k] + (256 >> p.rpt_shift) - 1) / (256 >> p.rpt_shift);
    acc += (((R[k] + 63) / 64 * 64) >> p.rpt_shift) * p.ctiles[k];  // padded rows are written too (as zeros)
    p.tile_end[k] = acc;
  }
  p.stage_bytes = 4 * p.Epad16 * 128;
  const int fixed = p.s_tiles * 32768 + 32768 + 1024;
  p.stages = (kMaxSmem - fixed) / p.stage_bytes;
  if (p.stages > 8) p.stages = 8;
  if (p.stages < 2) return LORY_ERR_SHAPE;
  const int smem = fixed + p.stages * p.stage_bytes;
  static bool attr_set[kMaxDevices];
  LORY_TRY(allow_dynamic_smem(merge_kernel, kMaxSmem, attr_set));
  const int grid = p.tile_end[2] < sm_count() ? p.tile_end[2] : sm_count();
  // one launch per 256 segments (each re-reads the experts once: the same ratio as one launch at S = 256)
  for (int base = 0; base < S; base += 256) {
    p.seg_base = base;
    p.S = S - base < 256 ? S - base : 256;
    p.s_tiles = (p.S + 127) / 128;
    ProfScope ps("merge", st);
    merge_kernel<<<grid, 192, smem, st>>>(maps, p);
    LORY_AFTER_LAUNCH();
  }
  return LORY_OK;
}

// dW_k = w^T dWbar_k and the dw partial slabs, one pass over the blocked dWbar_k of every piece.
// slab_add: the launch covers only part of the parameters, so its dw sums are added to the slabs.
static int launch_stage2(const lory_dims& D, const WsPtrs& q, const AdjPiece pc[3], bool slab_add, cudaStream_t st) {
  const int S = D.B * (D.L / D.T), E = D.E, Ep = e_pad(D);
  int R[3], C[3], first = -1;
  for (int k = 0; k < 3; ++k) {
    R[k] = pc[k].R;
    C[k] = pc[k].R > 0 ? pc[k].C : 0;
    if (R[k] > 0 && first < 0) first = k;
  }
  if (first < 0) return LORY_OK;
  Stage2Maps maps;
  Stage2Params p = {};
  const int S_launch = S < 256 ? S : 256;
  p.S = S_launch; p.S_total = S; p.E = E; p.Epad16 = e_pad16(D); p.s_tiles = (S_launch + 127) / 128;
  p.dw_partial = q.dw_partial; p.status = q.status;
  p.slab_add = slab_add ? 1 : 0;
  p.rpt_shift = stage2_rpt_shift(D);
  p.ncb = stage2_ncb(D);
  stage2_tiles(D, R, C, p.ctiles, p.tile_end);
  for (int k = 0; k < 3; ++k)
    p.cmagic[k] = p.ctiles[k] == 1 ? 0u : (uint32_t)(((1ull << 32) + p.ctiles[k] - 1) / p.ctiles[k]);
  if ((uint64_t)p.tile_end[2] * 64 >= (1ull << 32)) return LORY_ERR_SHAPE;  // keeps the reciprocal division exact
  // A box of fewer than 128 segments when S < 128: TMA would otherwise zero-fill the missing rows piece by piece.
  // A multiple of 16, so that the K steps of the first product stay inside the box (rows S.. of it are zero-filled).
  const uint32_t seg_box = S >= 128 ? 128u : (uint32_t)((S + 15) / 16 * 16);
  p.cb_stride = (int)seg_box * 128;
  p.dup = E <= 32 ? 1 : 0;
  // E <= 32 and at most 64 segments: both weight halves go through the tensor core into the same accumulator,
  // every 32-lane quarter of it holds the finished sums, and the epilogue warps take whole tiles in turn
  p.fast = (p.dup && S <= 64) ? 1 : 0;
  p.split = (S > 64 && E > 16) ? 0 : 1;   // measured: see the kernel's header
  if (p.dup) {
    LORY_TRY(make_map(&maps.w_hi, q.w_comb, 192, S, 1, 192, 0, 128));
    maps.w_lo = maps.w_hi;
  } else {
    LORY_TRY(make_map(&maps.w_hi, q.w_hi, Ep, S, 1, Ep, 0, 128));
    LORY_TRY(make_map(&maps.w_lo, q.w_lo, Ep, S, 1, Ep, 0, 128));
  }
  for (int k = 0; k < 3; ++k) {
    const AdjPiece& a = pc[R[k] > 0 ? k : first];  // an absent piece has no tiles; its maps repeat a present one
    LORY_TRY(make_blocked_map(&maps.dwbar[k], a.dsrc, a.R, a.C, S, 1, seg_box, p.rpt_shift ? 1 : p.ncb, 1));
    LORY_TRY(make_expert_map(&maps.theta[k], a.wsrc, a.R, a.C, E, p.Epad16, a.e_stride, a.row_stride));
    LORY_TRY(make_expert_map(&maps.out[k], a.ddst, a.R, a.C, E, E < 32 ? (uint32_t)E : 32u, a.e_stride, a.row_stride));  // no box rows past the experts
    p.acc_base[k] = a.ddst;
    p.rows[k] = a.R;
    p.cols[k] = a.C;
    p.e_stride[k] = (long)a.e_stride;
    p.row_stride[k] = (long)a.row_stride;
  }
  p.stage_bytes = p.ncb * (p.cb_stride + p.Epad16 * 128);  // dWbar tile (ncb 64-column blocks) + expert tile
  p.tx_bytes = p.stage_bytes;
  p.xch_bytes = p.dup ? 4096 : 8192;
  // w tiles, output staging, lo/hi exchange; and, when the box has fewer than 128 segments, room behind the last
  // stage for the 128-row operand reads of the second product (rows past the box are read and never used)
  p.w_bytes = p.fast ? 65536 : p.s_tiles * 32768;
  const int fixed = p.w_bytes + 16384 + 4 * p.xch_bytes + 1024 + (16384 - p.cb_stride);
  p.stages = (kMaxSmem - fixed) / p.stage_bytes;
  if (p.stages > 8) p.stages = 8;
  if (p.stages < 2) return LORY_ERR_SHAPE;
  const int smem = fixed + p.stages * p.stage_bytes;
  static bool attr_set[2][kMaxDevices];
  LORY_TRY(allow_dynamic_smem(stage2_kernel<false>, kMaxSmem, attr_set[0]));
  LORY_TRY(allow_dynamic_smem(stage2_kernel<true>, kMaxSmem, attr_set[1]));
  const int grid = p.tile_end[2] < sm_count() ? p.tile_end[2] : sm_count();
  // One launch per 256 segments; launches after the first add to the expert gradients the earlier ones stored
  // (the same read-add-store as gradient accumulation), and each writes its own rows of the dw slabs.
  for (int base = 0; base < S; base += 256) {
    p.seg_base = base;
    p.S = S - base < 256 ? S - base : 256;
    p.s_tiles = (p.S + 127) / 128;
    ProfScope ps("stage2", st);
    if (base > 0 || (D.flags & LORY_FLAG_ACCUMULATE_GRADS)) stage2_kernel<true><<<grid, 224, smem, st>>>(maps, p);
    else stage2_kernel<false><<<grid, 224, smem, st>>>(maps, p);
    LORY_AFTER_LAUNCH();
  }
  return LORY_OK;
}

void tc_split_tables(const lory_dims& D, const Layout& Lo, char* ws, bf16** hi, bf16** lo, bf16** comb, int* Epad) {
  const WsPtrs q = ws_ptrs(D, Lo, ws);
  *hi = q.w_hi;
  *lo = q.w_lo;
  *comb = D.E <= 32 ? q.w_comb : nullptr;
  *Epad = e_pad(D);
}

int tc_ffn_forward(const lory_dims& D, const Layout& Lo, char* ws, const bf16* x, const bf16* w1, const bf16* w2,
                   const bf16* w3, bf16* y, cudaStream_t st, bool w_is_split, const bf16* residual) {
  const int S = D.B * (D.L / D.T), T = D.T, d = D.d, f = D.f, E = D.E, Ep = e_pad(D);
  const WsPtrs q = ws_ptrs(D, Lo, ws);

  if (!(D.flags & LORY_FLAG_REUSE_MERGED)) {
    if (!w_is_split) {
      prof_begin("split_w", st);
      split_w_kernel<<<(unsigned)ceil_div((long)S * (E <= 32 ? 192 : Ep), 256), 256, 0, st>>>(q.w, q.w_hi, q.w_lo, q.w_comb, S, E, Ep);
      prof_end(st);
      LORY_AFTER_LAUNCH();
    }

    const bf16* src[3] = {w1, w3, w2};
    bf16* dst[3] = {q.wbar1, q.wbar3, q.wbar2};
    LORY_TRY(launch_merge(D, q, src, dst, st));
  }

  // G = X Wbar1^T, U = X Wbar3^T, H = silu(G) * U, one group per segment
  {
    CUtensorMap m_x, m_b1, m_b3, m_g, m_u, m_h;
    LORY_TRY(make_map(&m_x, x, d, T, S, d, (uint64_t)T * d, 128));
    LORY_TRY(make_blocked_map(&m_b1, q.wbar1, f, d, S, 64, 1, 1, 2));  // 128 rows (n) x 64 cols (k)
    LORY_TRY(make_blocked_map(&m_b3, q.wbar3, f, d, S, 64, 1, 1, 2));
    LORY_TRY(make_map(&m_g, q.G, f, T, S, f, (uint64_t)T * f, 32));  // stores: one warp's 32 rows
    LORY_TRY(make_map(&m_u, q.U, f, T, S, f, (uint64_t)T * f, 32));
    LORY_TRY(make_map(&m_h, q.H, f, T, S, f, (uint64_t)T * f, 32));
    TcGemmParams p = {};
    p.M = T; p.N = f; p.K = d; p.groups = S; p.status = q.status;
    if (T <= 32) {  // a decode step: 32-row A tiles, the freed shared memory holds more weight stages
      CUtensorMap m_xs;
      LORY_TRY(make_map(&m_xs, x, d, T, S, d, (uint64_t)T * d, 32));
      LORY_TRY((launch_tc<false, false, 256, MODE_DUALB, EPI_SWIGLU, true, false, 1, 32>("gemm1_swiglu", m_xs, m_xs, m_b1,
                                                                                         m_b3, m_g, m_u, m_h, p, st)));
    } else if (use_pairs(T))  // leader loads the Wbar1 rows (G half of the accumulator), its peer the Wbar3 rows (U half)
      LORY_TRY((launch_tc<false, false, 256, MODE_DUALB, EPI_SWIGLU, true, false, 2>("gemm1_swiglu", m_x, m_x, m_b1, m_b3,
                                                                                      m_g, m_u, m_h, p, st)));
    else
      LORY_TRY((launch_tc<false, false, 256, MODE_DUALB, EPI_SWIGLU, true>("gemm1_swiglu", m_x, m_x, m_b1, m_b3, m_g,
                                                                            m_u, m_h, p, st)));
  }
  // Y = H Wbar2^T
  {
    CUtensorMap m_h, m_b2, m_y;
    const bool pair = use_pairs(T);
    LORY_TRY(make_map(&m_h, q.H, f, T, S, f, (uint64_t)T * f, 128));
    // Few, short groups (a decode step: a handful of new tokens per sequence): 256-column tiles would leave most
    // SMs without one while each tile streams a long strip of Wbar2; 64-column tiles spread that read over 4 x the SMs.
    const bool narrow = !pair && ceil_div(T, 128) * ceil_div(d, 256) * S < sm_count();
    // B tile: 256 rows (n = d index) x 64 cols (k = f index); a CTA pair loads 128 rows each
    LORY_TRY(make_blocked_map(&m_b2, q.wbar2, d, f, S, 64, 1, 1, narrow ? 1 : (pair ? 2 : 4)));
    LORY_TRY(make_map(&m_y, y, d, T, S, d, (uint64_t)T * d, 32));
    TcGemmParams p = {};
    p.M = T; p.N = d; p.K = f; p.groups = S; p.status = q.status;
    p.residual = residual;
    if (narrow && T <= 32 && !residual) {
      CUtensorMap m_hs;
      LORY_TRY(make_map(&m_hs, q.H, f, T, S, f, (uint64_t)T * f, 32));
      LORY_TRY((launch_tc<false, false, 64, MODE_PLAIN, EPI_BF16, true, false, 1, 32>("gemm2", m_hs, m_hs, m_b2, m_b2, m_y,
                                                                                      m_y, m_y, p, st)));
    } else if (narrow) {
      if (residual)
        LORY_TRY((launch_tc<false, false, 64, MODE_PLAIN, EPI_BF16_RESADD, true>("gemm2", m_h, m_h, m_b2, m_b2, m_y, m_y,
                                                                                  m_y, p, st)));
      else
        LORY_TRY((launch_tc<false, false, 64, MODE_PLAIN, EPI_BF16, true>("gemm2", m_h, m_h, m_b2, m_b2, m_y, m_y, m_y,
                                                                          p, st)));
    } else if (residual) {  // y = residual + H Wbar2^T: the block's skip connection rides in the epilogue
      if (pair)
        LORY_TRY((launch_tc<false, false, 256, MODE_PLAIN, EPI_BF16_RESADD, true, false, 2>("gemm2", m_h, m_h, m_b2, m_b2,
                                                                                             m_y, m_y, m_y, p, st)));
      else
        LORY_TRY((launch_tc<false, false, 256, MODE_PLAIN, EPI_BF16_RESADD, true>("gemm2", m_h, m_h, m_b2, m_b2, m_y, m_y,
                                                                                   m_y, p, st)));
    } else if (pair)
      LORY_TRY((launch_tc<false, false, 256, MODE_PLAIN, EPI_BF16, true, false, 2>("gemm2", m_h, m_h, m_b2, m_b2, m_y,
                                                                                    m_y, m_y, p, st)));
    else
      LORY_TRY((launch_tc<false, false, 256, MODE_PLAIN, EPI_BF16, true>("gemm2", m_h, m_h, m_b2, m_b2, m_y, m_y, m_y,
                                                                          p, st)));
  }
  return LORY_OK;
}

// Weight gradients and merge adjoint, one parameter rectangle at a time through the ring (see adjoint_chunks).
// Per rectangle: dWbar_k[rect] = A^T B over every segment (K = T) into the ring, then dW_k[rect] = w^T dWbar_k[rect]
// and the rectangle's share of dw, added to the slabs.  The stream orders the launches: a rectangle is consumed
// before the next one overwrites the ring.
static int tc_adjoint_chunked(const lory_dims& D, const WsPtrs& q, const bf16* x, const bf16* w1, const bf16* w2,
                              const bf16* w3, const bf16* dy, bf16* dw1, bf16* dw2, bf16* dw3, cudaStream_t st) {
  const int S = D.B * (D.L / D.T), T = D.T, d = D.d, f = D.f;
  const AdjChunks ch = adjoint_chunks(D);
  bf16* ring = q.dwbar1;
  // matrix k: rows come from the columns of a_src (inner extent R[k]), columns from those of b_src (inner extent C[k])
  const int R[3] = {f, f, d}, C[3] = {d, d, f};
  const bf16* a_src[3] = {q.dG, q.dU, dy};
  const bf16* b_src[3] = {x, x, q.H};
  const bf16* wk[3] = {w1, w3, w2};
  bf16* dwk[3] = {dw1, dw3, dw2};
  LORY_CUDA_OK(cudaMemsetAsync(q.dw_partial, 0, (size_t)tc_dw_slabs(D) * S * D.E * sizeof(float), st));
  for (int k = 0; k < 3; ++k) {
    for (int r0 = 0; r0 < R[k]; r0 += ch.rows) {
      for (int c0 = 0; c0 < C[k]; c0 += ch.cols[k]) {
        const int Rc = R[k] - r0 < ch.rows ? R[k] - r0 : ch.rows;
        const int Cc = C[k] - c0 < ch.cols[k] ? C[k] - c0 : ch.cols[k];
        CUtensorMap m_a, m_b, m_o;
        LORY_TRY(make_map(&m_a, a_src[k] + r0, Rc, T, S, R[k], (uint64_t)T * R[k], 64));
        LORY_TRY(make_map(&m_b, b_src[k] + c0, Cc, T, S, C[k], (uint64_t)T * C[k], 64));
        LORY_TRY(make_blocked_map(&m_o, ring, Rc, Cc, S, 64, 1, 1, 2));
        LORY_TRY(launch_wgrad(m_a, m_b, m_o, Rc, Cc, T, S, R[k] >= 256, q.status, st));
        AdjPiece pc[3] = {};
        const uint64_t off = (uint64_t)r0 * C[k] + c0;
        pc[k] = AdjPiece{ring, wk[k] + off, dwk[k] + off, Rc, Cc, (uint64_t)f * d, (uint64_t)C[k]};
        LORY_TRY(launch_stage2(D, q, pc, true, st));
      }
    }
  }
  return LORY_OK;
}

int tc_ffn_backward(const lory_dims& D, const Layout& Lo, char* ws, const bf16* x, const bf16* w1, const bf16* w2,
                    const bf16* w3, const bf16* dy, bf16* dw1, bf16* dw2, bf16* dw3, cudaStream_t st) {
  const int S = D.B * (D.L / D.T), T = D.T, d = D.d, f = D.f;
  const WsPtrs q = ws_ptrs(D, Lo, ws);

  // dH = dY Wbar2; dG, dU in the epilogue
  {
    CUtensorMap m_dy, m_b2, m_dgo, m_duo, m_gi, m_ui;
    const bool pair = use_pairs(T);
    LORY_TRY(make_map(&m_dy, dy, d, T, S, d, (uint64_t)T * d, 128));
    // B[k = d index (rows), n = f index]: 4 col blocks per tile, 2 per CTA of a pair
    LORY_TRY(make_blocked_map(&m_b2, q.wbar2, d, f, S, 64, 1, pair ? 2 : 4, 1));
    LORY_TRY(make_map(&m_dgo, q.dG, f, T, S, f, (uint64_t)T * f, 128));
    LORY_TRY(make_map(&m_duo, q.dU, f, T, S, f, (uint64_t)T * f, 128));
    LORY_TRY(make_map(&m_gi, q.G, f, T, S, f, (uint64_t)T * f, 128));
    LORY_TRY(make_map(&m_ui, q.U, f, T, S, f, (uint64_t)T * f, 128));
    TcGemmParams p = {};
    p.M = T; p.N = f; p.K = d; p.groups = S; p.status = q.status;
    if (pair)
      LORY_TRY((launch_tc<false, true, 256, MODE_PLAIN, EPI_DSWIGLU, true, false, 2>("dh_dswiglu", m_dy, m_dy, m_b2, m_b2,
                                                                                      m_dgo, m_duo, m_duo, p, st, &m_gi,
                                                                                      &m_ui)));
    else
      LORY_TRY((launch_tc<false, true, 256, MODE_PLAIN, EPI_DSWIGLU, true>("dh_dswiglu", m_dy, m_dy, m_b2, m_b2, m_dgo,
                                                                            m_duo, m_duo, p, st, &m_gi, &m_ui)));
  }
  if (D.flags & LORY_FLAG_CHUNKED_ADJOINT) return tc_adjoint_chunked(D, q, x, w1, w2, w3, dy, dw1, dw2, dw3, st);
  // dWbar2[d, f] = dY^T H;  dWbar1[f, d] = dG^T X;  dWbar3[f, d] = dU^T X     (K = T), stored blocked
  {
    CUtensorMap m_dyT, m_h, m_dg, m_du, m_x, m_o2, m_o1, m_o3;
    LORY_TRY(make_map(&m_dyT, dy, d, T, S, d, (uint64_t)T * d, 64));
    LORY_TRY(make_map(&m_h, q.H, f, T, S, f, (uint64_t)T * f, 64));
    LORY_TRY(make_map(&m_dg, q.dG, f, T, S, f, (uint64_t)T * f, 64));
    LORY_TRY(make_map(&m_du, q.dU, f, T, S, f, (uint64_t)T * f, 64));
    LORY_TRY(make_map(&m_x, x, d, T, S, d, (uint64_t)T * d, 64));
    LORY_TRY(make_blocked_map(&m_o2, q.dwbar2, d, f, S, 64, 1, 1, 2));  // 128 rows x 64 cols per store
    LORY_TRY(make_blocked_map(&m_o1, q.dwbar1, f, d, S, 64, 1, 1, 2));
    LORY_TRY(make_blocked_map(&m_o3, q.dwbar3, f, d, S, 64, 1, 1, 2));
    // 256-row CTA-pair tiles whenever the output has at least 256 rows
    LORY_TRY(launch_wgrad(m_dyT, m_h, m_o2, d, f, T, S, d >= 256, q.status, st));
    LORY_TRY(launch_wgrad(m_dg, m_x, m_o1, f, d, T, S, f >= 256, q.status, st));
    LORY_TRY(launch_wgrad(m_du, m_x, m_o3, f, d, T, S, f >= 256, q.status, st));
  }
  // adjoint of the merge
  {
    const AdjPiece pc[3] = {{q.dwbar1, w1, dw1, f, d, (uint64_t)f * d, (uint64_t)d},
                            {q.dwbar3, w3, dw3, f, d, (uint64_t)f * d, (uint64_t)d},
                            {q.dwbar2, w2, dw2, d, f, (uint64_t)f * d, (uint64_t)f}};
    LORY_TRY(launch_stage2(D, q, pc, false, st));
  }
  return LORY_OK;
}

// dX = dG Wbar1 + dU Wbar3 + dh_bar / T  (the mean-pool gradient of the router path rides in the epilogue)
int tc_ffn_backward_dx(const lory_dims& D, const Layout& Lo, char* ws, const float* dh_bar, bf16* dx,
                       cudaStream_t st) {
  const int S = D.B * (D.L / D.T), T = D.T, d = D.d, f = D.f;
  const WsPtrs q = ws_ptrs(D, Lo, ws);
  CUtensorMap m_dg, m_du, m_b1, m_b3, m_dx;
  const bool pair = use_pairs(T);
  LORY_TRY(make_map(&m_dg, q.dG, f, T, S, f, (uint64_t)T * f, 128));
  LORY_TRY(make_map(&m_du, q.dU, f, T, S, f, (uint64_t)T * f, 128));
  // B[k = f index (rows), n = d index]: 4 col blocks per tile, 2 per CTA of a pair
  LORY_TRY(make_blocked_map(&m_b1, q.wbar1, f, d, S, 64, 1, pair ? 2 : 4, 1));
  LORY_TRY(make_blocked_map(&m_b3, q.wbar3, f, d, S, 64, 1, pair ? 2 : 4, 1));
  LORY_TRY(make_map(&m_dx, dx, d, T, S, d, (uint64_t)T * d, 32));
  TcGemmParams p = {};
  p.M = T; p.N = d; p.K = f; p.groups = S; p.status = q.status;
  p.rowvec = dh_bar; p.row_scale = 1.0f / (float)T;
  if (pair)
    LORY_TRY((launch_tc<false, true, 256, MODE_DUALK, EPI_BF16_ROWADD, true, false, 2>("dx", m_dg, m_du, m_b1, m_b3, m_dx,
                                                                                        m_dx, m_dx, p, st)));
  else
    LORY_TRY((launch_tc<false, true, 256, MODE_DUALK, EPI_BF16_ROWADD, true>("dx", m_dg, m_du, m_b1, m_b3, m_dx, m_dx,
                                                                              m_dx, p, st)));
  return LORY_OK;
}

// ---------------------------------------------------------------------------------------
// Self-test of the bounded wait every pipeline role uses: one thread waits on an mbarrier that nothing
// ever completes, with a small poll limit; the wait must give up, and the status word must say so.
// ---------------------------------------------------------------------------------------
__global__ void bounded_wait_selftest_kernel(uint32_t* status, uint32_t limit) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ volatile uint32_t abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
    if (!ptx::mbar_wait(&bar, 0, &abort_flag, limit)) atomicOr(status, STATUS_TIMEOUT_EPI);
  }
}

// The three predicates of the debug build on values that must fail each of them; nothing is accessed.
__global__ void debug_bounds_selftest_kernel(uint32_t* status) {
  extern __shared__ uint8_t dyn[];
  // (a) a tile coordinate: negative, beyond the extent, or off the 16-byte grid
  dbg::check(dbg::coord_ok(-1, 8) || dbg::coord_ok(8, 8) || dbg::inner_ok(4, 64), status);
  // (b) a shared-memory stage that ends one byte after the 1024 bytes this launch was given
  dbg::check(dbg::smem_ok(dyn + 1, 1024), status);
  // (c) a TMEM column range: 64 columns starting at column 480 of a 512-column allocation
  dbg::check(dbg::tmem_ok(480u, 0u, 512u, 64u), status);
}

int tc_debug_bounds_selftest(uint32_t* status_word, cudaStream_t st) {
  debug_bounds_selftest_kernel<<<1, 1, 1024, st>>>(status_word);
  LORY_AFTER_LAUNCH();
  return LORY_OK;
}

int tc_bounded_wait_selftest(uint32_t* status_word, cudaStream_t st) {
  bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(status_word, 10000u);
  LORY_AFTER_LAUNCH();
  return LORY_OK;
}

}  // namespace lory
