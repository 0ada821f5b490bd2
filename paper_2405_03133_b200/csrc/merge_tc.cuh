// Expert merging on the tensor cores (Eq. 2):  Wbar_k[s, r, c] = sum_e w[s, e] * W_k[e, r, c],  k = 1, 3, 2.
//
// One tile = 256 parameters (1, 2 or 4 neighbouring rows of 256, 128 or 64 consecutive columns), for 128 segments at once:
//   D[s, 256] = (w_hi + w_lo)[s, E] . W_k[E, 256 parameters]          (two MMAs per 16 experts)
// The routing weights (bf16 hi + lo, K-major) stay resident in shared memory; each expert tile is
// loaded once by TMA (4 boxes of 64 columns x E rows, one per row and column block of the tile) and used for
// every 128-segment tile.
// With S <= 64 the segments are placed twice in the 128 rows of the weight tile, and the two copies of the
// result are split by columns between the epilogue warps.
// Output goes to the blocked per-segment layout [row block][col block][segment][64][64]: the 128
// segments' 128-byte row pieces of one block are 8 KB apart inside one contiguous region.
// Roles: warp 0 TMA, warp 1 MMA, warps 2..5 epilogue.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "umma.cuh"

namespace lory {

struct MergeMaps {
  CUtensorMap w_hi, w_lo;  // (Epad, S, 1)      box (64, 128, 1)
  CUtensorMap theta[3];    // (C, E, R)         box (64, Epad16, 1)
  CUtensorMap out[3];      // blocked 5-D       box (64, 1, 32, 1, 1): one warp's 32 segments
};

struct MergeParams {
  int S, E, Epad16, s_tiles;  // S: segments of this launch (at most 256); s_tiles = ceil(S / 128)
  int seg_base;               // first segment of this launch (launches cover the segments 256 at a time)
  int dup;           // 1 (S <= 64): the w maps have 64-row boxes and the segments are placed twice (rows 0..63, 64..127);
                     // 2 (S <= 32): 32-row boxes, placed four times
  int rpt_shift;     // log2 of the rows per tile (1, 2 or 4 rows of 256, 128 or 64 columns)
  int ctiles[3];     // column tiles per row
  int tile_end[3];   // exclusive prefix sums of rows_padded * ctiles
  int stages, stage_bytes;
  uint32_t* status;
};

__global__ void __launch_bounds__(192, 1) merge_kernel(const __grid_constant__ MergeMaps maps, const MergeParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* s_w = smem;                                   // [s_tiles][hi 16 KB | lo 16 KB]
  uint8_t* s_out = smem + (size_t)p.s_tiles * 32768;     // 2 x 16 KB
  uint8_t* s_stage = s_out + 32768;
  __shared__ __align__(8) uint64_t full_bar[8];
  __shared__ __align__(8) uint64_t empty_bar[8];
  __shared__ __align__(8) uint64_t tmem_full_bar[2];
  __shared__ __align__(8) uint64_t tmem_empty_bar[2];
  __shared__ __align__(8) uint64_t w_bar;
  __shared__ uint32_t tmem_base_smem;
  __shared__ volatile uint32_t abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = p.tile_end[2];
  const int STAGES = p.stages;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 8; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&empty_bar[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&tmem_full_bar[a], 1);
      ptx::mbar_init(&tmem_empty_bar[a], 128);
    }
    ptx::mbar_init(&w_bar, 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&maps.w_hi);
    ptx::prefetch_tmap(&maps.theta[0]);
    ptx::prefetch_tmap(&maps.out[0]);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&tmem_base_smem, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_smem;

  // tile -> (matrix k, row r, first column c0).  Consecutive tiles walk the 64 rows of one row block for a fixed
  // column tile, so that the CTAs running at the same time fill neighbouring 128-byte pieces of the same output
  // blocks (whole DRAM pages instead of isolated pieces).
  const int rsh = p.rpt_shift;            // a tile has 1 << rsh rows ...
  const int cb_per_row = 4 >> rsh;        // ... of this many 64-column blocks each
  auto decode = [&](int tile, int& k, int& r, int& c0) {
    k = tile < p.tile_end[0] ? 0 : (tile < p.tile_end[1] ? 1 : 2);
    const int local = tile - (k == 0 ? 0 : p.tile_end[k - 1]);
    const int per_rb = (64 >> rsh) * p.ctiles[k];
    const int rb = local / per_rb, rem = local - rb * per_rb;
    r = rb * 64 + ((rem & ((64 >> rsh) - 1)) << rsh);
    c0 = (rem >> (6 - rsh)) * (256 >> rsh);
  };
  // chunk j of a tile (64 of its 256 accumulator columns): row offset and column-block offset inside the tile
  auto chunk_row = [&](int j) { return j / cb_per_row; };
  auto chunk_cb = [&](int j) { return j % cb_per_row; };

  // debug build: a decoded tile against the padded tile grid of its matrix
  auto tile_ok = [&](int k, int r, int c0) {
    if (!dbg::kOn) return true;
    if (k < 0 || k > 2) return false;
    const int tiles_k = p.tile_end[k] - (k ? p.tile_end[k - 1] : 0);
    return dbg::coord_ok(r, (tiles_k / p.ctiles[k]) << rsh) && dbg::inner_ok(c0, p.ctiles[k] * (256 >> rsh));
  };

  if (warp == 0) {
    if (lane == 0) {
      ptx::mbar_expect_tx(&w_bar, (uint32_t)p.s_tiles * 32768u);
      if (p.dup) {
        const int copies = 2 * p.dup, bytes = 16384 / copies;   // 2 x 64 rows or 4 x 32 rows of 128 bytes
        for (int h = 0; h < copies; ++h) {
          ptx::tma_load_3d(s_w + h * bytes, &maps.w_hi, &w_bar, 0, 0, 0);
          ptx::tma_load_3d(s_w + 16384 + h * bytes, &maps.w_lo, &w_bar, 0, 0, 0);
        }
      } else {
        for (int st = 0; st < p.s_tiles; ++st) {
          ptx::tma_load_3d(s_w + st * 32768, &maps.w_hi, &w_bar, 0, p.seg_base + st * 128, 0);
          ptx::tma_load_3d(s_w + st * 32768 + 16384, &maps.w_lo, &w_bar, 0, p.seg_base + st * 128, 0);
        }
      }
      uint32_t it = 0, issued = 0, last_parity = 0;
      const int box_bytes = p.Epad16 * 128;
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
        int k, r, c0;
        decode(tile, k, r, c0);
        // debug build: matrix index, row and first column of the tile against the padded tile grid
        if (!dbg::check(tile_ok(k, r, c0), p.status)) {
          k = 0; r = 0; c0 = 0;
        }
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1;
        if (!ptx::mbar_wait(&empty_bar[s], ph ^ 1, &abort_flag)) {
          atomicOr(p.status, STATUS_TIMEOUT_TMA);
          abort_flag = 1;
        }
        uint8_t* sB = s_stage + (size_t)s * p.stage_bytes;
        if (!dbg::check(dbg::smem_ok(sB, (uint32_t)p.stage_bytes), p.status)) continue;
        ptx::mbar_expect_tx(&full_bar[s], (uint32_t)p.stage_bytes);
        issued |= 1u << s;
        last_parity = (last_parity & ~(1u << s)) | (ph << s);
#pragma unroll
        for (int j = 0; j < 4; ++j)
          ptx::tma_load_3d(sB + j * box_bytes, &maps.theta[k], &full_bar[s], c0 + 64 * chunk_cb(j), 0, r + chunk_row(j));
      }
      if (abort_flag) {
        for (int s = 0; s < STAGES; ++s)
          if (issued & (1u << s)) ptx::mbar_wait(&full_bar[s], (last_parity >> s) & 1, &abort_flag, 1u << 20);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = ptx::make_idesc_bf16(128, 256, false, true);
      const int ksteps = p.Epad16 / 16;
      const uint32_t lbo = (uint32_t)p.Epad16 * 128;  // next 64 columns = next box
      if (!ptx::mbar_wait(&w_bar, 0, &abort_flag)) {
        atomicOr(p.status, STATUS_TIMEOUT_MMA);
        abort_flag = 1;
      }
      const uint32_t wbase = ptx::smem_u32(s_w);
      uint32_t it = 0, ai = 0;
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1;
        if (!ptx::mbar_wait(&full_bar[s], ph, &abort_flag)) {
          atomicOr(p.status, STATUS_TIMEOUT_MMA);
          abort_flag = 1;
        }
        const uint32_t bbase = ptx::smem_u32(s_stage + (size_t)s * p.stage_bytes);
        for (int st = 0; st < p.s_tiles; ++st, ++ai) {
          const uint32_t acc = ai & 1;
          if (!ptx::mbar_wait(&tmem_empty_bar[acc], ((ai >> 1) & 1) ^ 1, &abort_flag)) {
            atomicOr(p.status, STATUS_TIMEOUT_MMA);
            abort_flag = 1;
          }
          ptx::tc_fence_after_sync();
          const uint32_t tmem_d = tmem_base + acc * 256;
          const uint32_t a_hi = wbase + st * 32768, a_lo = a_hi + 16384;
          const bool acc_ok = dbg::check(dbg::tmem_ok(tmem_d, tmem_base, 512, 256) && st < 2, p.status);
          for (int kk = 0; kk < ksteps && acc_ok; ++kk) {
            const uint64_t bdesc = ptx::make_smem_desc(bbase + kk * 2048, lbo, 1024);
            ptx::umma_bf16(tmem_d, ptx::make_smem_desc(a_hi + kk * 32, 16, 1024), bdesc, idesc, kk > 0 ? 1u : 0u);
            ptx::umma_bf16(tmem_d, ptx::make_smem_desc(a_lo + kk * 32, 16, 1024), bdesc, idesc, 1u);
          }
          ptx::umma_commit(&tmem_full_bar[acc]);
        }
        ptx::umma_commit(&empty_bar[s]);
      }
    }
  } else {
    const int q = warp & 3;
    WarpStager wsg;
    wsg.buf = s_out + q * 8192;
    wsg.n = 0;
    // S > 64: this warp's accumulator rows are segments q*32 .. q*32+31 and it walks all four 64-column chunks.
    // S <= 64 (p.dup == 1): rows 64..127 repeat rows 0..63, so warps 0, 1 take chunks 0, 1 and warps 2, 3 chunks 2, 3.
    // S <= 32 (p.dup == 2): every 32-row quarter holds all segments, and warp q takes chunk q alone: four stores per
    // tile, none of them empty (with two copies half of the eight stores lie past the last segment).
    const int seg0 = p.dup == 2 ? 0 : (p.dup ? (q & 1) * 32 : q * 32);
    const int c_begin = p.dup == 2 ? q : (p.dup ? (q >> 1) * 2 : 0);
    const int c_end = p.dup == 2 ? q + 1 : (p.dup ? c_begin + 2 : 4);
    uint32_t ai = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      int k, r, c0;
      decode(tile, k, r, c0);
      for (int st = 0; st < p.s_tiles; ++st, ++ai) {
        const uint32_t acc = ai & 1;
        if (!ptx::mbar_wait(&tmem_full_bar[acc], (ai >> 1) & 1, &abort_flag)) {
          atomicOr(p.status, STATUS_TIMEOUT_EPI);
          abort_flag = 1;
        }
        __syncwarp();  // every lane polls by itself; the warp-wide tcgen05 instructions below need it whole again
        ptx::tc_fence_after_sync();
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256;
        // debug build: accumulator columns, staging buffer and output coordinates of this warp's stores; a tile
        // that fails is drained without reading TMEM or storing
        if (!dbg::check(dbg::tmem_ok(taddr + c_begin * 64, tmem_base, 512, (c_end - c_begin) * 64) &&
                            dbg::smem_ok(wsg.buf, 8192) && tile_ok(k, r, c0) &&
                            dbg::coord_ok(st * 128 + seg0, p.s_tiles * 128),
                        p.status)) {
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive(&tmem_empty_bar[acc]);
          continue;
        }
        uint32_t rr[64];
        ptx::tmem_ld_32x64(taddr + c_begin * 64, rr);
#pragma unroll 1
        for (int c = c_begin; c < c_end; ++c) {
          ptx::tmem_ld_wait();
          uint32_t w[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) w[j] = pack_bf16(__uint_as_float(rr[2 * j]), __uint_as_float(rr[2 * j + 1]));
          if (c + 1 < c_end) {
            ptx::tmem_ld_32x64(taddr + (c + 1) * 64, rr);
          } else {
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&tmem_empty_bar[acc]);
          }
          uint8_t* b = warp_stage(wsg, lane, w);
          if (lane == 0) {
            // (col in block, row in block, segment, col block, row block); blocks past the matrix are clipped
            ptx::tma_store_5d(&maps.out[k], b, 0, (r & 63) + chunk_row(c), p.seg_base + st * 128 + seg0,
                              (c0 >> 6) + chunk_cb(c), r >> 6);
            ptx::tma_store_commit();
          }
          wsg.n++;
        }
      }
    }
    if (lane == 0) ptx::tma_store_wait_all<0>();
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace lory
