// Grouped bf16 GEMM on the 5th-generation tensor cores: TMA-fed shared-memory pipeline,
// tcgen05.mma with fp32 accumulators in TMEM (double buffered), warp-specialised persistent CTAs.
//
//   C_g[m, n] = sum_k A_g[m, k] * B_g[k, n]          g = 0 .. groups-1
//
// Operands are described by 3-D tensor maps (innermost dim contiguous, rows, group) and may be
// K-major (innermost = K) or MN-major (innermost = M resp. N); all tiles use the 128-byte swizzle.
// B (and the bf16 output) may instead live in the blocked per-segment weight layout
// [row block][col block][segment][64][64] (B_BLK / C_BLK), addressed through 5-D tensor maps: every
// 64 x 64 block of one segment is one contiguous 8 KB piece of memory.
// CTA tile: 128 x BN x 64 (256 x BN over a CTA pair).  192 threads: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM
// owner, warps 2..5 = epilogue (one TMEM lane quarter each).
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "umma.cuh"

namespace lory {

enum TcMode {
  MODE_PLAIN = 0,  // one A map, one B map
  MODE_DUALB = 1,  // B tile = rows of B0 (first BN/2 columns of the accumulator) and of B1 (second half)
  MODE_DUALK = 2   // K loop runs over (A0, B0) and then over (A1, B1) into the same accumulator
};
enum TcEpi {
  EPI_BF16 = 0,    // tmC0 (bf16) = acc
  EPI_SWIGLU = 2,  // acc = [G | U]: tmC0 = G, tmC1 = U, tmC2 = silu(G) * U
  EPI_DSWIGLU = 3, // acc = dH; G (tmE0) and U (tmE1) tiles come in by TMA; tmC0 = dG, tmC1 = dU
  EPI_BF16_ROWADD = 4,  // tmC0 (bf16) = acc + rowvec[g, n] * row_scale   (rowvec float [groups, N])
  EPI_BF16_RESADD = 5   // tmC0 (bf16) = acc + residual[g*M + m, n]       (residual bf16 [groups*M, N])
};

struct TcGemmParams {
  int M, N, K;  // per-group extents; N counts output columns of C (per half for MODE_DUALB)
  int groups;
  int m_tiles, n_tiles;
  const float* rowvec;  // EPI_BF16_ROWADD
  const __nv_bfloat16* residual;  // EPI_BF16_RESADD
  float row_scale;
  uint32_t* status;
};

// CTAS = 2: two CTAs of a cluster share one 256 x BN tile (tcgen05 cta_group::2); each loads its own
// 128 rows of A and one half of B's BN columns, which cuts the L2 -> shared-memory traffic per flop by a third.
// AROWS < 128 (groups of at most AROWS rows: a decode step): only AROWS rows of A are loaded per stage, and the
// shared memory that frees goes into more stages, i.e. more weight bytes in flight per SM.  The MMA still reads 128
// rows; rows AROWS.. of its A operand are whatever follows in shared memory (inside the CTA's allocation: the output
// staging follows the last stage), they only reach accumulator rows that are never stored.
template <int BN, int EPI, int CTAS = 1, int AROWS = 128>
struct TcTile {
  static constexpr int BM = 128, BK = 64;
  static constexpr int A_BYTES = AROWS * BK * 2;
  static constexpr int B_BYTES = (BN / CTAS) * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int OUT_BYTES = 128 * 128;  // one 128-row x 64-column bf16 staging tile
  static constexpr int NARROW_STAGES = (227 * 1024 - 512 - 2 * OUT_BYTES - 1024) / STAGE_BYTES;
  // the SwiGLU-backward epilogue trades pipeline stages for two input staging tiles (G, U)
  static constexpr int STAGES = (AROWS < 128) ? (NARROW_STAGES > 16 ? 16 : NARROW_STAGES)
                                : (CTAS == 2) ? ((EPI == EPI_DSWIGLU) ? 5 : 6)
                                              : ((EPI == EPI_DSWIGLU) ? 3 : ((BN == 256) ? 4 : 6));
  static constexpr int IN_BYTES = (EPI == EPI_DSWIGLU) ? 2 * OUT_BYTES : 0;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 2 * OUT_BYTES + IN_BYTES + 1024;  // + alignment slack
};

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float2 unpack_bf16(uint32_t v) {
  return __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&v));
}

// Output staging: the four epilogue warps write a 128-row x 64-column bf16 tile into shared memory
// in the 128-byte-swizzled layout and one thread hands it to the TMA engine, which clips rows and
// columns that fall outside the tensor.  Two buffers alternate; `n` counts the stores issued.
struct OutStager {
  uint8_t* buf;
  uint32_t n;
};
// w holds this thread's row: 64 bf16 packed in 32 words.  Returns the staged buffer; the elected
// thread then issues its TMA store and commit, and every thread bumps os.n (stage_done).
__device__ __forceinline__ uint8_t* stage_tile(OutStager& os, int row_in_tile, bool issuer, const uint32_t (&w)[32]) {
  uint8_t* b = os.buf + (os.n & 1u) * (128 * 128);
  if (os.n >= 2) {
    if (issuer) ptx::tma_store_wait_read<1>();  // the store that last used this buffer has read it
    ptx::named_barrier(1, 128);
  }
  uint8_t* rowp = b + row_in_tile * 128;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    uint4 v = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
    *reinterpret_cast<uint4*>(rowp + ((j ^ (row_in_tile & 7)) << 4)) = v;
  }
  ptx::fence_async_smem();
  ptx::named_barrier(1, 128);
  return b;
}
// c0/c1/c2 = column, row, group of the tile.
template <bool BLK = false>
__device__ __forceinline__ void stage_and_store(OutStager& os, const CUtensorMap* tm, int c0, int c1, int c2,
                                                int row_in_tile, bool issuer, const uint32_t (&w)[32]) {
  uint8_t* b = stage_tile(os, row_in_tile, issuer, w);
  if (issuer) {
    if (BLK) ptx::tma_store_5d(tm, b, 0, 0, c2, c0 >> 6, c1 >> 6);  // two 64 x 64 blocks of segment c2
    else ptx::tma_store_3d(tm, b, c0, c1, c2);
    ptx::tma_store_commit();
  }
  os.n++;
}
// Per-warp output staging: an epilogue warp writes its own 32 rows x 64 columns (4 KB, 128-byte swizzle) into
// its private pair of buffers and its lane 0 hands them to the TMA engine.  No barrier between warps: the four
// epilogue warps drift apart and hide each other's latencies.  `n` counts this warp's stores.
struct WarpStager {
  uint8_t* buf;  // this warp's 2 x 4 KB, 1024-byte aligned
  uint32_t n;
};
__device__ __forceinline__ uint8_t* warp_stage(WarpStager& ws, int lane, const uint32_t (&w)[32]) {
  uint8_t* b = ws.buf + (ws.n & 1u) * 4096;
  if (ws.n >= 2) {
    if (lane == 0) ptx::tma_store_wait_read<1>();  // the store that last used this buffer has read it
    __syncwarp();
  }
  uint8_t* rowp = b + lane * 128;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    uint4 v = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
    *reinterpret_cast<uint4*>(rowp + ((j ^ (lane & 7)) << 4)) = v;
  }
  ptx::fence_async_smem();
  __syncwarp();
  return b;
}
// c0 = first column, row0 = first of this warp's 32 rows, c2 = group.  Box of the map: 32 rows x 64 columns.
template <bool BLK = false>
__device__ __forceinline__ void warp_stage_and_store(WarpStager& ws, const CUtensorMap* tm, int c0, int row0, int c2,
                                                     int lane, const uint32_t (&w)[32]) {
  uint8_t* b = warp_stage(ws, lane, w);
  if (lane == 0) {
    if (BLK) ptx::tma_store_5d(tm, b, 0, row0 & 63, c2, c0 >> 6, row0 >> 6);  // half of one 64 x 64 block
    else ptx::tma_store_3d(tm, b, c0, row0, c2);
    ptx::tma_store_commit();
  }
  ws.n++;
}
template <bool A_MN, bool B_MN, int BN, int MODE, int EPI, bool B_BLK = false, bool C_BLK = false, int CTAS = 1,
          int AROWS = 128>
__global__ void __launch_bounds__(192, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
               const __grid_constant__ CUtensorMap tmB0, const __grid_constant__ CUtensorMap tmB1,
               const __grid_constant__ CUtensorMap tmC0, const __grid_constant__ CUtensorMap tmC1,
               const __grid_constant__ CUtensorMap tmC2, const __grid_constant__ CUtensorMap tmE0,
               const __grid_constant__ CUtensorMap tmE1, const TcGemmParams p) {
  using Tile = TcTile<BN, EPI, CTAS, AROWS>;
  static_assert(AROWS == 128 || (!A_MN && CTAS == 1 && EPI != EPI_DSWIGLU), "short A tiles: K-major A, single CTA");
  constexpr bool PAIR = (CTAS == 2);
  const int rank = PAIR ? (int)ptx::cluster_ctarank() : 0;  // 0 = leader: arms the full barriers, issues the MMAs
  const int wid = blockIdx.x / CTAS, wstride = gridDim.x / CTAS;
  constexpr int STAGES = Tile::STAGES;
  constexpr int TILE_N = (MODE == MODE_DUALB) ? BN / 2 : BN;  // output columns per tile
  static_assert(!(MODE == MODE_DUALB && B_MN), "MODE_DUALB expects K-major B");
  static_assert(EPI != EPI_SWIGLU || (MODE == MODE_DUALB && BN == 256), "SwiGLU epilogue needs [G|U] tiles");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t full_bar[STAGES];
  __shared__ __align__(8) uint64_t empty_bar[STAGES];
  __shared__ __align__(8) uint64_t tmem_full_bar[2];
  __shared__ __align__(8) uint64_t tmem_empty_bar[2];
  __shared__ __align__(8) uint64_t epi_bar;  // completion of the epilogue's own TMA loads (EPI_DSWIGLU)
  __shared__ uint32_t tmem_base_smem;
  __shared__ volatile uint32_t abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = p.m_tiles * p.n_tiles * p.groups;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&empty_bar[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&tmem_full_bar[a], 1);
      ptx::mbar_init(&tmem_empty_bar[a], 128 * CTAS);
    }
    ptx::mbar_init(&epi_bar, 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tmA0);
    ptx::prefetch_tmap(&tmB0);
    if (MODE == MODE_DUALK) ptx::prefetch_tmap(&tmA1);
    if (MODE != MODE_PLAIN) ptx::prefetch_tmap(&tmB1);
    ptx::prefetch_tmap(&tmC0);
  }
  if (warp == 1) {
    if (PAIR) {
      ptx::tmem_alloc_pair(&tmem_base_smem, 2 * BN);
      ptx::tmem_relinquish_pair();
    } else {
      ptx::tmem_alloc(&tmem_base_smem, 2 * BN);
      ptx::tmem_relinquish();
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (PAIR) ptx::cluster_sync();  // both CTAs' barriers exist before either signals the other
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_smem;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      int s = 0;        // position in the stage ring and its phase, advanced by hand (no division per stage)
      uint32_t ph = 0;
      uint32_t issued = 0, last_parity = 0;
      bool ok = true;
      for (int tile = wid; tile < num_tiles; tile += wstride) {
        const int m_tile = tile % p.m_tiles;
        const int rest = tile / p.m_tiles;
        const int n_tile = rest % p.n_tiles;
        const int g = rest / p.n_tiles;
        int m0 = m_tile * (128 * CTAS) + 128 * rank, n0 = n_tile * TILE_N;
        int gc = g;
        const int nkb = (p.K + 63) / 64;
        const int total = (MODE == MODE_DUALK) ? 2 * nkb : nkb;
        // debug build: the tile's coordinates against the padded problem extents (a violated bound is recorded
        // and the tile is loaded from coordinate zero instead, so that every barrier still completes)
        if (!dbg::check(dbg::inner_ok(m0, p.m_tiles * 128 * CTAS) && dbg::inner_ok(n0, p.n_tiles * TILE_N) &&
                            dbg::coord_ok(gc, p.groups),
                        p.status)) {
          m0 = 128 * rank;
          n0 = 0;
          gc = 0;
        }
        for (int i = 0; i < total; ++i, s = (s + 1 == STAGES ? 0 : s + 1), ph ^= (s == 0)) {
          if (!ptx::mbar_wait(&empty_bar[s], ph ^ 1, &abort_flag)) {
            atomicOr(p.status, STATUS_TIMEOUT_TMA);
            abort_flag = 1;
            ok = false;
          }
          const bool second = (MODE == MODE_DUALK) && (i >= nkb);
          const int kb = second ? i - nkb : i;
          const int kc = dbg::check(dbg::inner_ok(kb * 64, nkb * 64), p.status) ? kb * 64 : 0;
          const CUtensorMap* ta = second ? &tmA1 : &tmA0;
          const CUtensorMap* tb = second ? &tmB1 : &tmB0;
          uint8_t* sA = smem + (size_t)s * Tile::STAGE_BYTES;
          uint8_t* sB = sA + Tile::A_BYTES;
          // a stage outside the shared-memory allocation is never written: the consumer's bounded wait reports it
          if (!dbg::check(dbg::smem_ok(sA, Tile::STAGE_BYTES), p.status)) continue;
          if (!PAIR) ptx::mbar_expect_tx(&full_bar[s], Tile::STAGE_BYTES);
          else if (rank == 0) ptx::mbar_expect_tx(&full_bar[s], 2 * Tile::STAGE_BYTES);  // both CTAs' bytes land here
          issued |= 1u << s;
          last_parity = (last_parity & ~(1u << s)) | (ph << s);
          uint64_t* fb = &full_bar[s];
          auto ld3 = [&](void* dst, const CUtensorMap* tm, int c0, int c1, int c2) {
            if (PAIR) ptx::tma_load_3d_pair(dst, tm, fb, c0, c1, c2);
            else ptx::tma_load_3d(dst, tm, fb, c0, c1, c2);
          };
          auto ld5 = [&](void* dst, const CUtensorMap* tm, int c2, int c3, int c4) {
            if (PAIR) ptx::tma_load_5d_pair(dst, tm, fb, 0, 0, c2, c3, c4);
            else ptx::tma_load_5d(dst, tm, fb, 0, 0, c2, c3, c4);
          };
          if (A_MN) {
            ld3(sA, ta, m0, kc, gc);
            ld3(sA + 8192, ta, m0 + 64, kc, gc);
          } else {
            ld3(sA, ta, kc, m0, gc);
          }
          // this CTA's share of B: all BN columns (CTAS = 1) or half of them (pair)
          constexpr int NB = BN / 64 / CTAS;  // 64-wide blocks of B per CTA
          const int nblk0 = (n0 >> 6) + rank * NB;
          if (B_BLK) {
            // coordinates: (col in block, row in block, segment, col block, row block)
            if (B_MN) {
              ld5(sB, tb, gc, nblk0, kc >> 6);  // box: NB col blocks
            } else if (MODE == MODE_DUALB) {
              if (PAIR) {
                ld5(sB, rank ? &tmB1 : &tmB0, gc, kc >> 6, n0 >> 6);  // leader: G half, peer: U half
              } else {
                ld5(sB, &tmB0, gc, kc >> 6, n0 >> 6);  // box: BN/128 row blocks
                ld5(sB + (BN / 2) * 128, &tmB1, gc, kc >> 6, n0 >> 6);
              }
            } else {
              ld5(sB, tb, gc, kc >> 6, nblk0);  // box: NB row blocks
            }
          } else if (B_MN) {
#pragma unroll
            for (int j = 0; j < NB; ++j) ld3(sB + j * 8192, tb, (nblk0 + j) * 64, kc, gc);
          } else if (MODE == MODE_DUALB) {
            if (PAIR) {
              ld3(sB, rank ? &tmB1 : &tmB0, kc, n0, gc);
            } else {
              ld3(sB, &tmB0, kc, n0, gc);
              ld3(sB + (BN / 2) * 128, &tmB1, kc, n0, gc);
            }
          } else {
            ld3(sB, tb, kc, nblk0 * 64, gc);
          }
        }
      }
      if (!ok || abort_flag) {
        // let this thread's copies in flight land before the CTA's shared memory goes away
        for (int s = 0; s < STAGES; ++s)
          if (issued & (1u << s)) ptx::mbar_wait(&full_bar[s], (last_parity >> s) & 1, &abort_flag, 1u << 20);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(128 * CTAS, BN, A_MN, B_MN);
      // Shared-memory descriptors differ only in their 14-bit address field (16-byte units): the constant part is
      // built once, the stage ring advances by hand, and per MMA only an addition is left (measured neutral for
      // these GEMMs, whose MMAs are long; the merge adjoint, with its short ones, gained 10-16 % from the same).
      const uint64_t adesc0 = A_MN ? ptx::make_smem_desc(0, 8192, 1024) : ptx::make_smem_desc(0, 16, 1024);
      const uint64_t bdesc0 = B_MN ? ptx::make_smem_desc(0, 8192, 1024) : ptx::make_smem_desc(0, 16, 1024);
      constexpr uint32_t a_step16 = (A_MN ? 2048u : 32u) >> 4, b_step16 = (B_MN ? 2048u : 32u) >> 4;
      const uint32_t smem16 = ptx::smem_u32(smem) >> 4;
      int s = 0;
      uint32_t ph = 0, tile_iter = 0;
      const int nkb = (p.K + 63) / 64;
      const int total = (MODE == MODE_DUALK) ? 2 * nkb : nkb;
      for (int tile = wid; tile < num_tiles; tile += wstride, ++tile_iter) {
        const uint32_t acc = tile_iter & 1;
        if (!ptx::mbar_wait(&tmem_empty_bar[acc], ((tile_iter >> 1) & 1) ^ 1, &abort_flag)) {
          atomicOr(p.status, STATUS_TIMEOUT_MMA);
          abort_flag = 1;
        }
        ptx::tc_fence_after_sync();
        const uint32_t tmem_d = tmem_base + acc * BN;
        const bool acc_ok = dbg::check(dbg::tmem_ok(tmem_d, tmem_base, 2 * BN, BN), p.status);
        for (int i = 0; i < total; ++i, s = (s + 1 == STAGES ? 0 : s + 1), ph ^= (s == 0)) {
          if (!ptx::mbar_wait(&full_bar[s], ph, &abort_flag)) {
            atomicOr(p.status, STATUS_TIMEOUT_MMA);
            abort_flag = 1;
          }
          ptx::tc_fence_after_sync();
          const uint32_t a16 = smem16 + (uint32_t)s * (Tile::STAGE_BYTES >> 4);   // this stage, 16-byte units
          const uint32_t b16 = a16 + (Tile::A_BYTES >> 4);
#pragma unroll
          for (int k16 = 0; k16 < 4; ++k16) {
            const uint64_t adesc = adesc0 | (uint64_t)((a16 + k16 * a_step16) & 0x3FFFu);
            const uint64_t bdesc = bdesc0 | (uint64_t)((b16 + k16 * b_step16) & 0x3FFFu);
            if (!acc_ok) continue;  // debug build: an accumulator outside the TMEM allocation is never written
            if (PAIR) ptx::umma_bf16_pair(tmem_d, adesc, bdesc, idesc, (i > 0 || k16 > 0) ? 1u : 0u);
            else ptx::umma_bf16(tmem_d, adesc, bdesc, idesc, (i > 0 || k16 > 0) ? 1u : 0u);
          }
          // frees the stage (in both CTAs of a pair) once these MMAs have read it
          if (PAIR) ptx::umma_commit_pair(&empty_bar[s]);
          else ptx::umma_commit(&empty_bar[s]);
        }
        if (PAIR) ptx::umma_commit_pair(&tmem_full_bar[acc]);
        else ptx::umma_commit(&tmem_full_bar[acc]);
      }
    }
  } else {
    // ------------------------------ epilogue ------------------------------
    auto arrive_tmem_empty = [&](uint64_t* bar) {
      if (PAIR) ptx::mbar_arrive_leader(bar);  // the leader's MMA warp waits for both CTAs' epilogues
      else ptx::mbar_arrive(bar);
    };
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    const int row_in_tile = q * 32 + lane;
    const bool issuer = (threadIdx.x == 64);
    OutStager os;  // whole-tile staging (SwiGLU-backward epilogue)
    os.buf = smem + (size_t)STAGES * Tile::STAGE_BYTES;
    os.n = 0;
    WarpStager wsg;  // per-warp staging (all other epilogues)
    wsg.buf = os.buf + q * 8192;
    wsg.n = 0;
    const bool staging_ok = dbg::check(dbg::smem_ok(os.buf, 2 * Tile::OUT_BYTES + Tile::IN_BYTES), p.status);
    uint32_t tile_iter = 0;
    for (int tile = wid; tile < num_tiles; tile += wstride, ++tile_iter) {
      const int m_tile = tile % p.m_tiles;
      const int rest = tile / p.m_tiles;
      const int n_tile = rest % p.n_tiles;
      const int g = rest / p.n_tiles;
      const int m0 = m_tile * (128 * CTAS) + 128 * rank;
      const int n0 = n_tile * TILE_N;
      const uint32_t acc = tile_iter & 1;
      if (!ptx::mbar_wait(&tmem_full_bar[acc], (tile_iter >> 1) & 1, &abort_flag)) {
        atomicOr(p.status, STATUS_TIMEOUT_EPI);
        abort_flag = 1;
      }
      __syncwarp();  // every lane polls by itself; the warp-wide tcgen05 instructions below need it whole again
      ptx::tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
      // debug build: this tile's output coordinates and accumulator columns; a tile that fails is drained
      // (its accumulator handed back) without reading TMEM or storing anything
      if (!dbg::check(staging_ok && dbg::inner_ok(n0, p.n_tiles * TILE_N) &&
                          dbg::coord_ok(m0, p.m_tiles * 128 * CTAS) && dbg::coord_ok(g, p.groups) &&
                          dbg::tmem_ok(taddr, tmem_base, 2 * BN, BN),
                      p.status)) {
        ptx::tc_fence_before_sync();
        arrive_tmem_empty(&tmem_empty_bar[acc]);
        continue;
      }

      if (EPI == EPI_BF16 || EPI == EPI_BF16_ROWADD || EPI == EPI_BF16_RESADD) {
        // software pipeline: the TMEM load of the next 64-column group is in flight while the
        // current group is converted, staged and handed to TMA
        const int ngroups = min(BN / 64, (p.N - n0 + 63) / 64);
        uint32_t r[64];
        ptx::tmem_ld_32x64(taddr, r);
#pragma unroll 1
        for (int c = 0; c < ngroups; ++c) {
          ptx::tmem_ld_wait();
          uint32_t w[32];
          if (EPI == EPI_BF16_ROWADD) {
            // every row of the tile receives the same vector: rowvec[g, n0 + c*64 .. +63] * row_scale
            const float* rv = p.rowvec + (size_t)g * p.N + n0 + c * 64;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
              if (n0 + c * 64 + 4 * j < p.N) v = *reinterpret_cast<const float4*>(rv + 4 * j);
              w[2 * j] = pack_bf16(__uint_as_float(r[4 * j]) + v.x * p.row_scale,
                                   __uint_as_float(r[4 * j + 1]) + v.y * p.row_scale);
              w[2 * j + 1] = pack_bf16(__uint_as_float(r[4 * j + 2]) + v.z * p.row_scale,
                                       __uint_as_float(r[4 * j + 3]) + v.w * p.row_scale);
            }
          } else if (EPI == EPI_BF16_RESADD) {
            // this thread's row of the residual: 64 bf16 = eight 16-byte pieces, zero outside the tensor
            const int rowg = m0 + q * 32 + lane, col0 = n0 + c * 64;
            const __nv_bfloat16* rs = p.residual + ((size_t)g * p.M + rowg) * p.N + col0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              uint4 v = make_uint4(0u, 0u, 0u, 0u);
              if (rowg < p.M && col0 + 8 * j < p.N) v = *reinterpret_cast<const uint4*>(rs + 8 * j);
              const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
              for (int t = 0; t < 4; ++t) {
                const float2 o = unpack_bf16(vw[t]);
                w[4 * j + t] = pack_bf16(__uint_as_float(r[8 * j + 2 * t]) + o.x, __uint_as_float(r[8 * j + 2 * t + 1]) + o.y);
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) w[j] = pack_bf16(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
          }
          if (c + 1 < ngroups) {
            ptx::tmem_ld_32x64(taddr + (c + 1) * 64, r);
          } else {
            ptx::tc_fence_before_sync();
            arrive_tmem_empty(&tmem_empty_bar[acc]);  // accumulator fully read: the MMA warp may reuse it
          }
          // blocked outputs go out as whole 128-row tiles (two contiguous 8 KB blocks per store); the others per warp
          if (C_BLK) stage_and_store<true>(os, &tmC0, n0 + c * 64, m0, g, row_in_tile, issuer, w);
          else warp_stage_and_store<false>(wsg, &tmC0, n0 + c * 64, m0 + q * 32, g, lane, w);
        }
      } else if (EPI == EPI_SWIGLU) {
#pragma unroll 1
        for (int c = 0; c < TILE_N / 64; ++c) {
          if (n0 + c * 64 >= p.N) break;
          uint32_t wg[32], wu[32], wh[32];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            uint32_t rg[32], ru[32];
            ptx::tmem_ld_32x32(taddr + c * 64 + h * 32, rg);
            ptx::tmem_ld_32x32(taddr + TILE_N + c * 64 + h * 32, ru);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              float g0 = __uint_as_float(rg[2 * j]), g1 = __uint_as_float(rg[2 * j + 1]);
              float u0 = __uint_as_float(ru[2 * j]), u1 = __uint_as_float(ru[2 * j + 1]);
              wg[h * 16 + j] = pack_bf16(g0, g1);
              wu[h * 16 + j] = pack_bf16(u0, u1);
              wh[h * 16 + j] = pack_bf16(g0 * sigmoid_fast(g0) * u0, g1 * sigmoid_fast(g1) * u1);
            }
          }
          warp_stage_and_store(wsg, &tmC0, n0 + c * 64, m0 + q * 32, g, lane, wg);
          warp_stage_and_store(wsg, &tmC1, n0 + c * 64, m0 + q * 32, g, lane, wu);
          warp_stage_and_store(wsg, &tmC2, n0 + c * 64, m0 + q * 32, g, lane, wh);
        }
      } else {  // EPI_DSWIGLU
        // G and U tiles of the next 64-column group are fetched by TMA (issued by this role's
        // elected thread) while the current group is computed and stored.
        const int ngroups = min(BN / 64, (p.N - n0 + 63) / 64);
        uint8_t* bufG = os.buf + 2 * Tile::OUT_BYTES;
        uint8_t* bufU = bufG + Tile::OUT_BYTES;
        uint8_t* outG = os.buf;
        uint8_t* outU = os.buf + Tile::OUT_BYTES;
        if (issuer && tile_iter == 0) {  // later tiles were prefetched by the previous tile's last group
          ptx::mbar_expect_tx(&epi_bar, 2 * Tile::OUT_BYTES);
          ptx::tma_load_3d(bufG, &tmE0, &epi_bar, n0, m0, g);
          ptx::tma_load_3d(bufU, &tmE1, &epi_bar, n0, m0, g);
        }
        uint32_t r[64];
        ptx::tmem_ld_32x64(taddr, r);
#pragma unroll 1
        for (int c = 0; c < ngroups; ++c) {
          if (!ptx::mbar_wait(&epi_bar, (os.n >> 1) & 1, &abort_flag)) {
            atomicOr(p.status, STATUS_TIMEOUT_EPI);
            abort_flag = 1;
          }
          __syncwarp();  // every lane polls by itself; the warp-wide tcgen05 instructions below need it whole again
          uint32_t wg[32], wu[32];
          {
            const uint4* rowG = reinterpret_cast<const uint4*>(bufG + row_in_tile * 128);
            const uint4* rowU = reinterpret_cast<const uint4*>(bufU + row_in_tile * 128);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int sw = j ^ (row_in_tile & 7);
              uint4 gq = rowG[sw], uq = rowU[sw];
              wg[4 * j] = gq.x; wg[4 * j + 1] = gq.y; wg[4 * j + 2] = gq.z; wg[4 * j + 3] = gq.w;
              wu[4 * j] = uq.x; wu[4 * j + 1] = uq.y; wu[4 * j + 2] = uq.z; wu[4 * j + 3] = uq.w;
            }
          }
          ptx::named_barrier(1, 128);  // every thread holds its G, U row: the input buffers are free
          if (issuer) {
            int nt = tile, nc = c + 1;
            if (nc >= ngroups) { nt = tile + wstride; nc = 0; }
            if (nt < num_tiles) {
              const int nm = nt % p.m_tiles, nrest = nt / p.m_tiles;
              ptx::mbar_expect_tx(&epi_bar, 2 * Tile::OUT_BYTES);
              ptx::tma_load_3d(bufG, &tmE0, &epi_bar, (nrest % p.n_tiles) * TILE_N + nc * 64, nm * (128 * CTAS) + 128 * rank, nrest / p.n_tiles);
              ptx::tma_load_3d(bufU, &tmE1, &epi_bar, (nrest % p.n_tiles) * TILE_N + nc * 64, nm * (128 * CTAS) + 128 * rank, nrest / p.n_tiles);
            }
          }
          ptx::tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            float2 gg = unpack_bf16(wg[j]), uu = unpack_bf16(wu[j]);
            float dh0 = __uint_as_float(r[2 * j]), dh1 = __uint_as_float(r[2 * j + 1]);
            float s0 = sigmoid_fast(gg.x), s1 = sigmoid_fast(gg.y);
            wg[j] = pack_bf16(dh0 * uu.x * s0 * (1.0f + gg.x * (1.0f - s0)), dh1 * uu.y * s1 * (1.0f + gg.y * (1.0f - s1)));
            wu[j] = pack_bf16(dh0 * gg.x * s0, dh1 * gg.y * s1);
          }
          if (c + 1 < ngroups) {
            ptx::tmem_ld_32x64(taddr + (c + 1) * 64, r);
          } else {
            ptx::tc_fence_before_sync();
            arrive_tmem_empty(&tmem_empty_bar[acc]);
          }
          if (os.n > 0) {
            if (issuer) ptx::tma_store_wait_read<0>();  // the previous group's stores have read the output buffers
            ptx::named_barrier(1, 128);
          }
          {
            uint4* rowG = reinterpret_cast<uint4*>(outG + row_in_tile * 128);
            uint4* rowU = reinterpret_cast<uint4*>(outU + row_in_tile * 128);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int sw = j ^ (row_in_tile & 7);
              rowG[sw] = make_uint4(wg[4 * j], wg[4 * j + 1], wg[4 * j + 2], wg[4 * j + 3]);
              rowU[sw] = make_uint4(wu[4 * j], wu[4 * j + 1], wu[4 * j + 2], wu[4 * j + 3]);
            }
          }
          ptx::fence_async_smem();
          ptx::named_barrier(1, 128);
          if (issuer) {
            ptx::tma_store_3d(&tmC0, outG, n0 + c * 64, m0, g);
            ptx::tma_store_3d(&tmC1, outU, n0 + c * 64, m0, g);
            ptx::tma_store_commit();
          }
          os.n += 2;
        }
      }
      if (EPI == EPI_SWIGLU) {
        ptx::tc_fence_before_sync();
        arrive_tmem_empty(&tmem_empty_bar[acc]);
      }
    }
    if (lane == 0) ptx::tma_store_wait_all<0>();  // every store of this warp has landed before the CTA retires
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (PAIR) ptx::cluster_sync();  // the peer's shared memory and barriers stay valid until both CTAs are done
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    if (PAIR) ptx::tmem_dealloc_pair(tmem_base, 2 * BN);
    else ptx::tmem_dealloc(tmem_base, 2 * BN);
  }
}

}  // namespace lory
