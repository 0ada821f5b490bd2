// Per-segment weight gradients on the tensor cores with one operand resident in shared memory:
//
//   C_g[m, n] = sum_t A_g[t, m] * B_g[t, n]        g = segment, t < T <= 256 (the contraction is over the tokens)
//
// dWbar1 = dG^T X, dWbar3 = dU^T X, dWbar2 = dY^T H: both operands are MN-major (their rows are tokens), the
// output goes to the blocked per-segment layout.  The shorter the segment, the more operand bytes a 256 x 256 tile
// of a CTA pair needs per flop (32 KB per CTA for 512 cycles of MMA at T = 64); but all the tiles of one output row
// strip share their A operand (and all tiles of one column strip their B operand), and one CTA's part of such an
// operand is at most 64 KB.  So a CTA pair takes whole strips: the strip's operand (RES_A: A, rows m0..m0+255 of
// the output; else B, columns n0..n0+255) is loaded once into a resident buffer, whose 64-token blocks are handed
// back one by one during the strip's last tile, the other operand streams through a ring, and the loads per tile
// are halved.  Used for T <= 128, where it measures 4-9 % faster than the grouped GEMM; at T = 256 the two tie.
// Roles as in the grouped GEMM: warp 0 TMA producer, warp 1 MMA issuer (leader CTA) and TMEM owner, warps 2..5
// epilogue; tcgen05.mma.cta_group::2, fp32 accumulators double-buffered in TMEM.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "umma.cuh"

namespace lory {

struct WgradParams {
  int M, N, K;          // per-segment output rows, columns; K = T <= 256
  int groups;           // segments
  int m_tiles, n_tiles; // 256-row / 256-column tiles
  uint32_t* status;
};

struct WgradTile {
  static constexpr int PIECE = 16384;   // one CTA's part of one operand for one 64-token block: 128 x 64 bf16
  static constexpr int KB_MAX = 4;      // 64-token blocks of the contraction (T <= 256)
  static constexpr int STAGES = 6;      // ring of the streamed operand: 96 KB in flight per CTA
  static constexpr int RES_BUFS = 1;    // buffers of the resident operand (its 64-token blocks are released one by one)
  static constexpr int OUT_BYTES = 128 * 128;   // one 128-row x 64-column staging piece
  static constexpr int OUT_BUFS = 4;            // a whole tile's four pieces: a store has a tile's time to drain
  static constexpr int SMEM_BYTES = RES_BUFS * KB_MAX * PIECE + STAGES * PIECE + OUT_BUFS * OUT_BYTES + 1024;
};

template <bool RES_A>
__global__ void __launch_bounds__(192, 1)
wgrad_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
             const __grid_constant__ CUtensorMap tmC, const WgradParams p) {
  using W = WgradTile;
  constexpr int STAGES = W::STAGES, NRES = W::RES_BUFS * W::KB_MAX;
  const int rank = (int)ptx::cluster_ctarank();  // 0 = leader: arms the full barriers, issues the MMAs
  const int wid = blockIdx.x / 2, wstride = gridDim.x / 2;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* s_res = smem;                              // [RES_BUFS][KB_MAX] pieces of the resident operand
  uint8_t* s_ring = smem + NRES * W::PIECE;           // [STAGES] pieces of the streamed operand
  uint8_t* s_out = s_ring + STAGES * W::PIECE;        // OUT_BUFS x 16 KB output staging
  __shared__ __align__(8) uint64_t full_s[STAGES];
  __shared__ __align__(8) uint64_t empty_s[STAGES];
  __shared__ __align__(8) uint64_t full_r[NRES];
  __shared__ __align__(8) uint64_t empty_r[NRES];
  __shared__ __align__(8) uint64_t tmem_full_bar[2];
  __shared__ __align__(8) uint64_t tmem_empty_bar[2];
  __shared__ uint32_t tmem_base_smem;
  __shared__ volatile uint32_t abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nkb = (p.K + 63) / 64;                                  // <= KB_MAX (checked by the host)
  const int inner = RES_A ? p.n_tiles : p.m_tiles;                  // tiles of a strip
  const int num_strips = (RES_A ? p.m_tiles : p.n_tiles) * p.groups;
  // strip -> (its fixed tile index, segment); tile j of the strip -> (m_tile, n_tile)
  const int outer = RES_A ? p.m_tiles : p.n_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(&full_s[s], 1);
      ptx::mbar_init(&empty_s[s], 1);
    }
    for (int s = 0; s < NRES; ++s) {
      ptx::mbar_init(&full_r[s], 1);
      ptx::mbar_init(&empty_r[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&tmem_full_bar[a], 1);
      ptx::mbar_init(&tmem_empty_bar[a], 256);
    }
    abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tmA);
    ptx::prefetch_tmap(&tmB);
    ptx::prefetch_tmap(&tmC);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(&tmem_base_smem, 512);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync();  // both CTAs' barriers exist before either signals the other
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_smem;

  if (warp == 0) {
    // ------------------------------ TMA producer (one thread in each CTA) ------------------------------
    if (lane == 0) {
      uint32_t it = 0, ri = 0;   // streamed pieces issued; strips started
      bool ok = true;
      // one piece: this CTA's 128 rows (A) or 128 columns (B) of a 64-token block = two boxes of 64
      auto load_piece = [&](uint8_t* dst, const CUtensorMap* tm, uint64_t* bar, int x0, int kc, int g) {
        ptx::tma_load_3d_pair(dst, tm, bar, x0, kc, g);
        ptx::tma_load_3d_pair(dst + 8192, tm, bar, x0 + 64, kc, g);
      };
      for (int strip = wid; strip < num_strips; strip += wstride, ++ri) {
        int fix = strip % outer, g = strip / outer;
        if (!dbg::check(dbg::coord_ok(fix, outer) && dbg::coord_ok(g, p.groups), p.status)) {
          fix = 0;
          g = 0;
        }
        const int rbuf = (int)(ri % W::RES_BUFS) * W::KB_MAX;
        const uint32_t rph = (ri / W::RES_BUFS) & 1u;
        const int xr = fix * 256 + 128 * rank;       // first row (RES_A) / column (else) of the resident piece
        for (int j = 0; j < inner; ++j) {
          const int xs = j * 256 + 128 * rank;       // first column / row of the streamed piece
          for (int kb = 0; kb < nkb; ++kb, ++it) {
            if (j == 0) {
              // the strip's own operand, block kb: its buffer was last read by the strip before the previous one
              if (!ptx::mbar_wait(&empty_r[rbuf + kb], rph ^ 1, &abort_flag)) {
                atomicOr(p.status, STATUS_TIMEOUT_TMA);
                abort_flag = 1;
                ok = false;
              }
              uint8_t* dst = s_res + (size_t)(rbuf + kb) * W::PIECE;
              if (dbg::check(dbg::smem_ok(dst, W::PIECE), p.status)) {
                if (rank == 0) ptx::mbar_expect_tx(&full_r[rbuf + kb], 2 * W::PIECE);  // both CTAs' bytes land here
                load_piece(dst, RES_A ? &tmA : &tmB, &full_r[rbuf + kb], xr, kb * 64, g);
              }
            }
            const int s = (int)(it % STAGES);
            const uint32_t ph = (it / STAGES) & 1u;
            if (!ptx::mbar_wait(&empty_s[s], ph ^ 1, &abort_flag)) {
              atomicOr(p.status, STATUS_TIMEOUT_TMA);
              abort_flag = 1;
              ok = false;
            }
            uint8_t* dst = s_ring + (size_t)s * W::PIECE;
            if (!dbg::check(dbg::smem_ok(dst, W::PIECE), p.status)) continue;
            if (rank == 0) ptx::mbar_expect_tx(&full_s[s], 2 * W::PIECE);
            load_piece(dst, RES_A ? &tmB : &tmA, &full_s[s], xs, kb * 64, g);
          }
        }
      }
      if (!ok || abort_flag) {
        // let the copies in flight land before this CTA's shared memory goes away (the leader owns the barriers
        // that count them; a short bounded wait is all the peer can do)
        for (int s = 0; s < STAGES; ++s) ptx::mbar_wait(&full_s[s], 0, &abort_flag, 1u << 16);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader CTA) ------------------------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(256, 256, true, true);
      const uint32_t res0 = ptx::smem_u32(s_res), ring0 = ptx::smem_u32(s_ring);
      uint32_t it = 0, ri = 0, tile_iter = 0;
      for (int strip = wid; strip < num_strips; strip += wstride, ++ri) {
        const int rbuf = (int)(ri % W::RES_BUFS) * W::KB_MAX;
        const uint32_t rph = (ri / W::RES_BUFS) & 1u;
        for (int j = 0; j < inner; ++j, ++tile_iter) {
          const uint32_t acc = tile_iter & 1u;
          if (!ptx::mbar_wait(&tmem_empty_bar[acc], ((tile_iter >> 1) & 1u) ^ 1u, &abort_flag)) {
            atomicOr(p.status, STATUS_TIMEOUT_MMA);
            abort_flag = 1;
          }
          ptx::tc_fence_after_sync();
          const uint32_t tmem_d = tmem_base + acc * 256;
          const bool acc_ok = dbg::check(dbg::tmem_ok(tmem_d, tmem_base, 512, 256), p.status);
          for (int kb = 0; kb < nkb; ++kb, ++it) {
            if (j == 0 && !ptx::mbar_wait(&full_r[rbuf + kb], rph, &abort_flag)) {
              atomicOr(p.status, STATUS_TIMEOUT_MMA);
              abort_flag = 1;
            }
            const int s = (int)(it % STAGES);
            const uint32_t ph = (it / STAGES) & 1u;
            if (!ptx::mbar_wait(&full_s[s], ph, &abort_flag)) {
              atomicOr(p.status, STATUS_TIMEOUT_MMA);
              abort_flag = 1;
            }
            ptx::tc_fence_after_sync();
            const uint32_t r_addr = res0 + (uint32_t)(rbuf + kb) * W::PIECE;
            const uint32_t s_addr = ring0 + (uint32_t)s * W::PIECE;
            const uint32_t a_addr = RES_A ? r_addr : s_addr, b_addr = RES_A ? s_addr : r_addr;
#pragma unroll
            for (int k16 = 0; k16 < 4; ++k16) {
              // MN-major pieces: 16 token rows = 2048 bytes per K step, the next 64 rows / columns 8192 bytes further
              const uint64_t adesc = ptx::make_smem_desc(a_addr + k16 * 2048, 8192, 1024);
              const uint64_t bdesc = ptx::make_smem_desc(b_addr + k16 * 2048, 8192, 1024);
              if (!acc_ok) continue;
              ptx::umma_bf16_pair(tmem_d, adesc, bdesc, idesc, (kb > 0 || k16 > 0) ? 1u : 0u);
            }
            ptx::umma_commit_pair(&empty_s[s]);                               // the ring stage, in both CTAs
            if (j == inner - 1) ptx::umma_commit_pair(&empty_r[rbuf + kb]);   // last use of the strip's operand
          }
          ptx::umma_commit_pair(&tmem_full_bar[acc]);
        }
      }
    }
  } else {
    // ------------------------------ epilogue: fp32 accumulator -> bf16 -> blocked output ------------------------------
    const int q = warp & 3;
    const int row_in_tile = q * 32 + lane;
    const bool issuer = (threadIdx.x == 64);
    uint32_t n_stores = 0;  // pieces handed to the TMA engine so far; piece n uses staging buffer n % OUT_BUFS
    const bool staging_ok = dbg::check(dbg::smem_ok(s_out, W::OUT_BUFS * W::OUT_BYTES), p.status);
    uint32_t tile_iter = 0;
    for (int strip = wid; strip < num_strips; strip += wstride) {
      const int fix = strip % outer, g = strip / outer;
      for (int j = 0; j < inner; ++j, ++tile_iter) {
        const int m0 = (RES_A ? fix : j) * 256 + 128 * rank;
        const int n0 = (RES_A ? j : fix) * 256;
        const uint32_t acc = tile_iter & 1u;
        if (!ptx::mbar_wait(&tmem_full_bar[acc], (tile_iter >> 1) & 1u, &abort_flag)) {
          atomicOr(p.status, STATUS_TIMEOUT_EPI);
          abort_flag = 1;
        }
        __syncwarp();  // every lane polls by itself; the warp-wide tcgen05 instructions below need it whole again
        ptx::tc_fence_after_sync();
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256;
        if (!dbg::check(staging_ok && dbg::inner_ok(n0, p.n_tiles * 256) && dbg::coord_ok(m0, p.m_tiles * 256) &&
                            dbg::coord_ok(g, p.groups) && dbg::tmem_ok(taddr, tmem_base, 512, 256),
                        p.status)) {
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive_leader(&tmem_empty_bar[acc]);
          continue;
        }
        const int ngroups = min(4, (p.N - n0 + 63) / 64);
        uint32_t r[64];
        ptx::tmem_ld_32x64(taddr, r);
#pragma unroll 1
        for (int c = 0; c < ngroups; ++c) {
          ptx::tmem_ld_wait();
          uint32_t w[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) w[i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
          if (c + 1 < ngroups) {
            ptx::tmem_ld_32x64(taddr + (c + 1) * 64, r);
          } else {
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive_leader(&tmem_empty_bar[acc]);  // accumulator fully read: the MMA warp may reuse it
          }
          // a whole 128-row x 64-column piece (two contiguous 8 KB blocks of segment g) through staging buffer
          // n % OUT_BUFS: wait until the store that used it OUT_BUFS pieces ago has read it, fill it (128-byte
          // swizzle), hand it to the TMA engine
          uint8_t* b = s_out + (size_t)(n_stores % W::OUT_BUFS) * W::OUT_BYTES;
          if (n_stores >= W::OUT_BUFS) {
            if (issuer) ptx::tma_store_wait_read<W::OUT_BUFS - 1>();
            ptx::named_barrier(1, 128);
          }
          uint8_t* rowp = b + row_in_tile * 128;
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *reinterpret_cast<uint4*>(rowp + ((i ^ (row_in_tile & 7)) << 4)) =
                make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
          ptx::fence_async_smem();
          ptx::named_barrier(1, 128);
          if (issuer) {
            ptx::tma_store_5d(&tmC, b, 0, 0, g, (n0 + c * 64) >> 6, m0 >> 6);
            ptx::tma_store_commit();
          }
          ++n_stores;
        }
      }
    }
    if (lane == 0) ptx::tma_store_wait_all<0>();
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::cluster_sync();  // the peer's shared memory and barriers stay valid until both CTAs are done
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc_pair(tmem_base, 512);
  }
}

}  // namespace lory
