// Adjoint of the merge in one pass over the per-segment weight gradients (bf16, S <= 256, E <= 64):
//
//   dW_k[e, p]  = sum_s w[s, e] * dWbar_k[s, p]          k = 1, 3, 2   (written as bf16)
//   dw[s, e]   += sum_p dWbar_k[s, p] * W_k[e, p]                      (per-CTA fp32 partial slab)
//
// dWbar_k lives in the blocked layout [row block][col block][segment][64][64].  One tile = one matrix
// row r and 128 consecutive columns; for each group of 128 segments its [128 x 128] piece of dWbar_k
// (128-byte row pieces 8 KB apart) is brought into shared memory ONCE by TMA and feeds two
// tcgen05.mma chains: as the N-contiguous B operand of the first product (K = segments) and as
// the K-major A operand of the second (K = parameters).  The routing weights (bf16 hi + lo) stay
// resident in shared memory, the lo tile right behind the hi tile, so that one M = 128 MMA yields
// hi-weighted sums in accumulator rows 0..63 and lo-weighted sums in rows 64..127; the epilogue adds
// the two halves.  With E <= 32 one 64-wide table holds hi in columns 0..31 and lo in 32..63 and is placed
// in shared memory twice, so that all four epilogue warps have work: two per 64-column half of the tile.  The dw accumulator stays in TMEM for the whole kernel.
// With E <= 32 and at most 64 segments (p.fast) the first product runs as two MMAs per 16 segments, [hi|hi] and
// [lo|lo] tables into ONE accumulator: every 32-lane quarter then holds the finished sums of all experts, and the
// epilogue warps take whole tiles in turn (two per accumulator, one 64-column half each) without exchanging
// anything (d = 2048, f = 5504: E = 32, S = 16: 1.52 -> 1.17 ms; S = 64: 1.95 -> 1.64 ms; E = 16, S = 64: 1.65 -> 1.54 ms;
// at S = 128 the doubled MMA count costs more than it saves, so the arrangement above stays there).
// With 17..64 segments a tile of this arrangement is 192 columns wide (three blocks; block b of a CTA's i-th tile
// goes to epilogue warp (3 i + b) mod 4): a third fewer MMAs of the first product per byte.
// Roles: warp 0 TMA, warp 1 issues the first product and owns TMEM, warps 2..5 epilogue, warp 6 issues the second
// product.  Two issuing threads because with few segments a tile is small (24 KB at S = 64) and the instruction
// stream of ONE thread issuing both products (12 MMAs with their descriptors, 2 commits, 2 waits) was what a tile
// waited for (E = 8, S = 128: 0.52 -> 0.45 ms; E = 16, S = 64, d = 2048: 1.83 -> 1.65 ms); each stage is handed back
// once both threads' MMAs have read it (its barrier counts two arrivals).  A third issuer (the second product split
// by column block into accumulators of their own) measured no faster.  Where the kernel waits for memory anyway
// (more than 64 segments and more than 16 experts: E = 32, S = 128) the second issuer measured 5 % SLOWER on the
// same GPU (0.57 -> 0.60 ms, 12 % more DRAM reads: tiles that share fetched lines drift apart), so there warp 1
// issues both products (p.split = 0) and warp 6 idles.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "umma.cuh"

namespace lory {

struct Stage2Maps {
  CUtensorMap w_hi, w_lo;  // (Epad, S, 1)   box (64, 128, 1); with E <= 32 both map the combined hi|lo table
  CUtensorMap dwbar[3];    // blocked 5-D    box (64, 1, min(128, S rounded up to 8), 2, 1)
  CUtensorMap theta[3];    // (C, E, R)      box (64, Epad16, 1)
  CUtensorMap out[3];      // (C, E, R)      box (64, 32, 1): one warp's 32 experts, rows clipped to E
};

struct Stage2Params {
  int S, E, Epad16, s_tiles;  // S: segments of this launch (at most 256); s_tiles = ceil(S / 128)
  int seg_base, S_total;      // first segment of this launch; all segments (row count of a dw slab)
  int rpt_shift;    // 0: a tile is ncb * 64 columns of one row; 1: 64 columns of two neighbouring rows
  int ncb;          // 64-column blocks of a tile: 2, or 3 on the fast path with 33..64 segments (fewer MMAs per byte)
  int ctiles[3];    // column tiles per row
  uint32_t cmagic[3];  // ceil(2^32 / ctiles), 0 for ctiles == 1: n / ctiles == __umulhi(n, cmagic) for every tile index n
  int tile_end[3];  // exclusive prefix sums of (rows rounded up to 64) * ctiles
  int cb_stride;    // bytes between the two 64-column blocks of a dWbar tile in shared memory (= segments per box * 128)
  int dup;          // E <= 32: w_hi and w_lo are both the combined table [hi | lo | hi | hi | lo | lo] (32 columns each)
  int split;        // the second product is issued by a warp of its own
  int fast;         // E <= 32 and S <= 64: hi and lo sums meet in the accumulator (see the kernel)
  int w_bytes;      // shared memory of the resident weight tiles
  int xch_bytes;    // one exchange buffer: 32 lanes x 256 B, or x 128 B with E <= 32
  int stages;       // pipeline depth (<= 8)
  int stage_bytes, tx_bytes;
  const __nv_bfloat16* acc_base[3];  // the three output tensors (or sub-rectangles of them), read by the accumulating variant
  int rows[3], cols[3];              // extent of each
  long e_stride[3], row_stride[3];   // elements between experts and between rows of each
  int slab_add;       // add to the dw slab instead of overwriting it (a launch that covers part of the parameters)
  float* dw_partial;  // [slabs, S, E]; CTA b owns slab b
  uint32_t* status;
};

// ACC: add the values already in the output tensors (gradient accumulation).
template <bool ACC>
__global__ void __launch_bounds__(224, 1)
stage2_kernel(const __grid_constant__ Stage2Maps maps, const Stage2Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* s_w = smem;                                // [s_tiles][hi 16 KB | lo 16 KB]; fast: [hi|hi, hi|hi, lo|lo, lo|lo] 16 KB each
  uint8_t* s_out = smem + (size_t)p.w_bytes;          // 2 storing warps x 2 x 4 KB output staging
  uint8_t* s_xch = s_out + 16384;                     // 2 warp couples x 2 buffers: lo halves on their way to the hi warps
                                                      // (fast: staging of the other two storing warps)
  uint8_t* s_stage = s_xch + 4 * p.xch_bytes;
  __shared__ __align__(8) uint64_t full_bar[8];
  __shared__ __align__(8) uint64_t empty_bar[8];
  constexpr int NACC = 2;  // per-tile accumulators in flight (three were measured: no faster), the dw accumulator behind them
  __shared__ __align__(8) uint64_t tmem_full_bar[NACC];
  __shared__ __align__(8) uint64_t tmem_empty_bar[NACC];
  __shared__ __align__(8) uint64_t w_bar, d2_bar;
  __shared__ uint32_t tmem_base_smem;
  __shared__ volatile uint32_t abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = p.tile_end[2];
  const int STAGES = p.stages;
  const int NCB = p.ncb;   // 64-column blocks per tile (2; 3 on the fast path with 33..64 segments)
  // tile -> (matrix k, row r, first column c0)
  auto decode = [&](int tile, int& k, int& r, int& c0) {
    k = tile < p.tile_end[0] ? 0 : (tile < p.tile_end[1] ? 1 : 2);
    const int local = tile - (k == 0 ? 0 : p.tile_end[k - 1]);
    // local / ctiles[k] without the division (a single tile per row has no 32-bit reciprocal: magic 0)
    r = p.cmagic[k] ? (int)__umulhi((uint32_t)local, p.cmagic[k]) : local;
    c0 = (local - r * p.ctiles[k]) * (p.rpt_shift ? 64 : NCB * 64);
    r <<= p.rpt_shift;
  };
  // the two 64-column halves of a tile: columns c0 and c0 + 64 of row r, or (two-row tiles) column c0 of rows r, r + 1
  const int half_col = p.rpt_shift ? 0 : 64, half_row = p.rpt_shift ? 1 : 0;
  const uint32_t ACC_COLS = (uint32_t)NCB * 64u;   // TMEM columns of one per-tile accumulator

  // debug build: a decoded tile against the padded tile grid of its matrix
  auto tile_ok = [&](int k, int r, int c0) {
    if (!dbg::kOn) return true;
    if (k < 0 || k > 2) return false;
    const int tiles_k = p.tile_end[k] - (k ? p.tile_end[k - 1] : 0);
    return dbg::coord_ok(r, (tiles_k / p.ctiles[k]) << p.rpt_shift) && dbg::inner_ok(c0, p.ctiles[k] * (p.rpt_shift ? 64 : NCB * 64));
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < 8; ++s) {
      ptx::mbar_init(&full_bar[s], 1);
      ptx::mbar_init(&empty_bar[s], p.split ? 2 : 1);   // one arrival per MMA-issuing thread
    }
    for (int a = 0; a < NACC; ++a) {
      ptx::mbar_init(&tmem_full_bar[a], 1);
      ptx::mbar_init(&tmem_empty_bar[a], p.fast ? 32 * p.ncb : 128);   // fast: one warp per 64-column block reads it
    }
    ptx::mbar_init(&w_bar, 1);
    ptx::mbar_init(&d2_bar, 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&maps.w_hi);
    ptx::prefetch_tmap(&maps.dwbar[0]);
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
  const uint32_t tmem_d2 = tmem_base + NACC * ACC_COLS;

  // second product of one stage: dw [s, e] += dWbar [s, p] . W^T [p, e]   (one accumulator per group of 128 segments,
  // resident in TMEM for the whole kernel; with fewer than 128 segments in the box the rows past them hold whatever
  // follows in shared memory, and their accumulator rows are never read).  d16: the stage's address in 16-byte units.
  const uint32_t idesc2 = ptx::make_idesc_bf16(128, p.Epad16, false, false);
  auto issue_second = [&](uint32_t d16, int st, bool first) {
    const uint64_t d2ab = ptx::make_smem_desc(0, 16, 1024);   // K-major tiles; only the 14-bit address varies
    const uint32_t cb16 = (uint32_t)p.cb_stride >> 4, t16 = (uint32_t)(p.Epad16 * 128) >> 4;
    const uint32_t tb16 = d16 + (uint32_t)NCB * cb16;         // the stage's expert tile
    const uint32_t tmem_d2s = tmem_d2 + st * p.Epad16;
#pragma unroll
    for (int j = 0; j < NCB; ++j) {
#pragma unroll
      for (int k16 = 0; k16 < 4; ++k16) {
        const uint64_t adesc = d2ab | (uint64_t)(d16 + j * cb16 + k16 * 2);
        const uint64_t bdesc = d2ab | (uint64_t)(tb16 + j * t16 + k16 * 2);
        ptx::umma_bf16(tmem_d2s, adesc, bdesc, idesc2, (!first || j > 0 || k16 > 0) ? 1u : 0u);
      }
    }
  };

  if (warp == 0) {
    if (lane == 0) {
      // routing weights, once
      ptx::mbar_expect_tx(&w_bar, p.fast ? 65536u : (uint32_t)p.s_tiles * 32768u);
      if (p.fast) {
        // columns 64..127 of the combined table are [hi | hi], 128..191 [lo | lo]; each tile sits in shared memory
        // twice, so that the MMA's second 64-row group repeats the first
        for (int h = 0; h < 2; ++h) {
          ptx::tma_load_3d(s_w + h * 16384, &maps.w_hi, &w_bar, 64, p.seg_base, 0);
          ptx::tma_load_3d(s_w + 32768 + h * 16384, &maps.w_hi, &w_bar, 128, p.seg_base, 0);
        }
      } else {
        for (int st = 0; st < p.s_tiles; ++st) {
          ptx::tma_load_3d(s_w + st * 32768, &maps.w_hi, &w_bar, 0, p.seg_base + st * 128, 0);
          ptx::tma_load_3d(s_w + st * 32768 + 16384, &maps.w_lo, &w_bar, 0, p.seg_base + st * 128, 0);
        }
      }
      uint32_t issued = 0, last_parity = 0;
      int s = 0;          // position in the stage ring and its phase, advanced by hand: a division per tile on
      uint32_t ph = 0;    // this one thread is time the whole pipeline waits for
      const uint32_t tx = (uint32_t)p.tx_bytes;
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
        int k, r, c0;
        decode(tile, k, r, c0);
        if (!dbg::check(tile_ok(k, r, c0), p.status)) {
          k = 0; r = 0; c0 = 0;
        }
        for (int st = 0; st < p.s_tiles; ++st, s = (s + 1 == STAGES ? 0 : s + 1), ph ^= (s == 0)) {
          if (!ptx::mbar_wait(&empty_bar[s], ph ^ 1, &abort_flag)) {
            atomicOr(p.status, STATUS_TIMEOUT_TMA);
            abort_flag = 1;
          }
          uint8_t* sD = s_stage + (size_t)s * p.stage_bytes;
          uint8_t* sT = sD + NCB * p.cb_stride;
          if (!dbg::check(dbg::smem_ok(sD, (uint32_t)p.stage_bytes) && dbg::coord_ok(st, 2), p.status)) continue;
          ptx::mbar_expect_tx(&full_bar[s], tx);
          issued |= 1u << s;
          last_parity = (last_parity & ~(1u << s)) | (ph << s);
          // (col in block, row in block, segment, col block, row block): two col blocks, 128 segments
          if (p.rpt_shift) {  // two boxes of one column block each (rows r, r + 1)
            ptx::tma_load_5d(sD, &maps.dwbar[k], &full_bar[s], 0, r & 63, p.seg_base + st * 128, c0 >> 6, r >> 6);
            ptx::tma_load_5d(sD + p.cb_stride, &maps.dwbar[k], &full_bar[s], 0, (r & 63) + 1, p.seg_base + st * 128,
                             c0 >> 6, r >> 6);
          } else {            // one box of two column blocks
            ptx::tma_load_5d(sD, &maps.dwbar[k], &full_bar[s], 0, r & 63, p.seg_base + st * 128, c0 >> 6, r >> 6);
          }
          for (int j = 0; j < NCB; ++j)
            ptx::tma_load_3d(sT + j * p.Epad16 * 128, &maps.theta[k], &full_bar[s], c0 + j * half_col, 0, r + j * half_row);
        }
      }
      if (abort_flag) {
        for (int s = 0; s < STAGES; ++s)
          if (issued & (1u << s)) ptx::mbar_wait(&full_bar[s], (last_parity >> s) & 1, &abort_flag, 1u << 20);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc1 = ptx::make_idesc_bf16(128, NCB * 64, true, true);
      if (!ptx::mbar_wait(&w_bar, 0, &abort_flag)) {
        atomicOr(p.status, STATUS_TIMEOUT_MMA);
        abort_flag = 1;
      }
      const uint32_t wbase = ptx::smem_u32(s_w);
      // Shared-memory descriptors differ only in their 14-bit address field (16-byte units): the constant part is
      // built once and the address added per instruction, which keeps this one thread's work per tile small.
      const uint64_t d1a = ptx::make_smem_desc(0, 16384, 1024);                    // w tile, lo 16 KB behind hi
      const uint64_t d1b = ptx::make_smem_desc(0, (uint32_t)p.cb_stride, 1024);    // dWbar tile as [segment, column]
      const uint32_t stage16 = (uint32_t)p.stage_bytes >> 4;
      const uint32_t stage0_16 = ptx::smem_u32(s_stage) >> 4, w16 = wbase >> 4;
      int s = 0;
      uint32_t ph = 0, tcount = 0;
      const bool d2_ok = dbg::check(dbg::tmem_ok(tmem_d2, tmem_base, 512, (uint32_t)(p.s_tiles * p.Epad16)), p.status);
      uint32_t acc = 0, acc_ph = 0;   // accumulator ring position and phase
      for (int tile = blockIdx.x; tile < num_tiles;
           tile += gridDim.x, ++tcount, acc = (acc + 1 == NACC ? 0 : acc + 1), acc_ph ^= (acc == 0)) {
        if (!ptx::mbar_wait(&tmem_empty_bar[acc], acc_ph ^ 1, &abort_flag)) {
          atomicOr(p.status, STATUS_TIMEOUT_MMA);
          abort_flag = 1;
        }
        const uint32_t tmem_d1 = tmem_base + acc * ACC_COLS;
        // debug build: the per-tile accumulator inside the 512 columns
        const bool acc_ok = dbg::check(dbg::tmem_ok(tmem_d1, tmem_base, 512, ACC_COLS), p.status);
        for (int st = 0; st < p.s_tiles; ++st, s = (s + 1 == STAGES ? 0 : s + 1), ph ^= (s == 0)) {
          if (!ptx::mbar_wait(&full_bar[s], ph, &abort_flag)) {
            atomicOr(p.status, STATUS_TIMEOUT_MMA);
            abort_flag = 1;
          }
          ptx::tc_fence_after_sync();
          const uint32_t d16 = stage0_16 + (uint32_t)s * stage16;   // this stage's dWbar tile, 16-byte units
          const uint32_t whi16 = w16 + (uint32_t)st * (32768u >> 4);
          const int rows = min(128, p.S - st * 128);
          const int ksteps = (rows + 15) / 16;
          // rows 0..63: w_hi^T [e, s] . dWbar [s, p]; rows 64..127: w_lo^T . dWbar (the A operand's second
          // 64-row group lies 16 KB after the first: that is the lo tile)
          if (p.fast) {
            // every 32-row quarter: (w_hi + w_lo)^T [e, s] . dWbar [s, p], the two halves as two MMAs into one accumulator
            for (int kk = 0; kk < ksteps && acc_ok; ++kk) {
              const uint64_t bdesc = d1b | (uint64_t)(d16 + kk * 128);
              ptx::umma_bf16(tmem_d1, d1a | (uint64_t)(w16 + kk * 128), bdesc, idesc1, kk > 0 ? 1u : 0u);
              ptx::umma_bf16(tmem_d1, d1a | (uint64_t)(w16 + (32768u >> 4) + kk * 128), bdesc, idesc1, 1u);
            }
          } else {
            for (int kk = 0; kk < ksteps && acc_ok; ++kk) {
              ptx::umma_bf16(tmem_d1, d1a | (uint64_t)(whi16 + kk * 128), d1b | (uint64_t)(d16 + kk * 128), idesc1,
                             (st > 0 || kk > 0) ? 1u : 0u);
            }
          }
          if (!p.split && d2_ok) issue_second(d16, st, tcount == 0);   // no second issuer: both products from here
          ptx::umma_commit(&empty_bar[s]);
        }
        ptx::umma_commit(&tmem_full_bar[acc]);
      }
      if (!p.split) ptx::umma_commit(&d2_bar);
    }
  } else if (warp == 6) {
    // the second product from a thread of its own (p.split)
    if (lane == 0 && p.split) {
      const uint32_t stage16 = (uint32_t)p.stage_bytes >> 4;
      const uint32_t stage0_16 = ptx::smem_u32(s_stage) >> 4;
      const bool acc_ok = dbg::check(dbg::tmem_ok(tmem_d2, tmem_base, 512, (uint32_t)(p.s_tiles * p.Epad16)), p.status);
      int s = 0;
      uint32_t ph = 0, tcount = 0;
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++tcount) {
        for (int st = 0; st < p.s_tiles; ++st, s = (s + 1 == STAGES ? 0 : s + 1), ph ^= (s == 0)) {
          if (!ptx::mbar_wait(&full_bar[s], ph, &abort_flag)) {
            atomicOr(p.status, STATUS_TIMEOUT_MMA);
            abort_flag = 1;
          }
          ptx::tc_fence_after_sync();
          if (acc_ok) issue_second(stage0_16 + (uint32_t)s * stage16, st, tcount == 0);
          ptx::umma_commit(&empty_bar[s]);
        }
      }
      ptx::umma_commit(&d2_bar);
    }
  } else {
    const int q = warp & 3;
    const int row_in_tile = q * 32 + lane;
    WarpStager wsg;
    wsg.n = 0;
    // E > 32: warps 0, 1 of this role own the hi rows (experts 0..31, 32..63), warps 2, 3 the matching lo rows,
    // and every warp walks both 64-column halves of the tile.
    // E <= 32 (p.dup): accumulator rows 0..31 are hi, 32..63 lo, and rows 64..127 repeat them (the weight tile
    // is in shared memory twice), so warps 0, 1 take columns 0..63 and warps 2, 3 columns 64..127.
    const bool dup = p.dup != 0;
    const int pair = dup ? (q >> 1) : (q & 1);          // which hi/lo couple this warp belongs to
    const bool is_hi = dup ? ((q & 1) == 0) : (q < 2);
    const bool has_rows = dup ? true : (pair * 32 < p.E);
    const int c_begin = dup ? pair : 0, c_end = dup ? pair + 1 : 2;
    const int e0 = dup ? 0 : pair * 32;                 // first expert row of the stored box
    wsg.buf = s_out + pair * 8192;                      // only the hi warp of a couple stores
    // this lane's bf16 row (128 values, or 64 with E <= 32), its 16-byte chunks swizzled by lane
    const int xlane = p.xch_bytes >> 5, xmask = (xlane >> 4) - 1;
    uint8_t* xch = s_xch + pair * 2 * p.xch_bytes + lane * xlane;
    if (p.fast) {
      // Every 32-lane quarter of an accumulator holds the finished sums of all (<= 32) experts, so any warp can take
      // any 64-column block of any tile from its own lanes.  Block b of this CTA's i-th tile goes to warp
      // (i * NCB + b) mod 4: with two blocks per tile warps 0, 1 serve the even tiles and 2, 3 the odd ones; with
      // three, every warp serves three tiles out of four.  No exchange between warps, and a warp has more than a
      // tile period for its load - convert - store chain.
      wsg.buf = s_out + q * 8192;   // four storing warps: the exchange buffers serve as staging too
      uint32_t i = 0;
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++i) {
        const int half = (int)((q - i * (uint32_t)NCB) & 3u);   // the block of this tile that is this warp's, if < NCB
        if (half >= NCB) continue;
        const uint32_t my_acc = i & 1u;
        int k, row, c0;
        decode(tile, k, row, c0);
        if (!ptx::mbar_wait(&tmem_full_bar[my_acc], (i >> 1) & 1u, &abort_flag)) {
          atomicOr(p.status, STATUS_TIMEOUT_EPI);
          abort_flag = 1;
        }
        __syncwarp();  // every lane polls by itself; the warp-wide tcgen05 instructions below need it whole again
        ptx::tc_fence_after_sync();
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + my_acc * ACC_COLS + half * 64;
        if (!dbg::check(tile_ok(k, row, c0) && dbg::tmem_ok(taddr, tmem_base, 512, 64) && dbg::smem_ok(wsg.buf, 8192),
                        p.status)) {
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive(&tmem_empty_bar[my_acc]);
          continue;
        }
        uint32_t r[64];
        ptx::tmem_ld_32x64(taddr, r);
        const int col0 = c0 + half * half_col, rowc = row + half * half_row;
        uint4 old[8];
        if (ACC) {  // gradient accumulation: this lane's 64 old values (expert `lane`), zero where the tile leaves the tensor
          const bool row_ok = lane < p.E && rowc < p.rows[k];
          const __nv_bfloat16* src = p.acc_base[k] + (size_t)lane * p.e_stride[k] + (size_t)rowc * p.row_stride[k] + col0;
#pragma unroll
          for (int j = 0; j < 8; ++j)
            old[j] = (row_ok && col0 + 8 * j < p.cols[k]) ? *reinterpret_cast<const uint4*>(src + 8 * j)
                                                          : make_uint4(0u, 0u, 0u, 0u);
        }
        ptx::tmem_ld_wait();
        ptx::tc_fence_before_sync();
        ptx::mbar_arrive(&tmem_empty_bar[my_acc]);   // the values are in registers: the accumulator may be reused
        uint32_t w[32];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t ol[4] = {ACC ? old[j].x : 0u, ACC ? old[j].y : 0u, ACC ? old[j].z : 0u, ACC ? old[j].w : 0u};
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            float a = __uint_as_float(r[8 * j + 2 * t]), b = __uint_as_float(r[8 * j + 2 * t + 1]);
            if (ACC) {
              const float2 o2 = unpack_bf16(ol[t]);
              a += o2.x;
              b += o2.y;
            }
            w[4 * j + t] = pack_bf16(a, b);
          }
        }
        warp_stage_and_store(wsg, &maps.out[k], col0, 0, rowc, lane, w);
      }
    }
    uint32_t it = 0;
    uint32_t acc = 0, acc_ph = 0;   // accumulator ring position and phase
    for (int tile = p.fast ? num_tiles : (int)blockIdx.x; tile < num_tiles;
         tile += gridDim.x, ++it, acc = (acc + 1 == NACC ? 0 : acc + 1), acc_ph ^= (acc == 0)) {
      int k, row, c0;
      decode(tile, k, row, c0);
      if (!ptx::mbar_wait(&tmem_full_bar[acc], acc_ph, &abort_flag)) {
        atomicOr(p.status, STATUS_TIMEOUT_EPI);
        abort_flag = 1;
      }
      __syncwarp();  // every lane polls by itself; the warp-wide tcgen05 instructions below need it whole again
      ptx::tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * ACC_COLS;
      // debug build: a tile whose coordinates, accumulator columns or staging buffers are out of range is drained
      // (every term is the same for the two warps of a couple, which meet at a named barrier below)
      const bool tile_fine = dbg::check(tile_ok(k, row, c0) && dbg::tmem_ok(taddr, tmem_base, 512, 128) &&
                                            dbg::smem_ok(wsg.buf, 8192) &&
                                            dbg::smem_ok(s_xch + pair * 2 * p.xch_bytes, 2u * (uint32_t)p.xch_bytes),
                                        p.status);
      if (!has_rows || !tile_fine) {
        ptx::tc_fence_before_sync();
        ptx::mbar_arrive(&tmem_empty_bar[acc]);
        continue;
      }
      uint8_t* xb = xch + (it & 1u) * p.xch_bytes;
      uint32_t r[64];
      ptx::tmem_ld_32x64(taddr + c_begin * 64, r);
      if (!is_hi) {
        // lo half: round to bf16 (these sums are 2^-9 of the result) and pass them to the partner warp
#pragma unroll 1
        for (int c = c_begin; c < c_end; ++c) {
          ptx::tmem_ld_wait();
          uint32_t w[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) w[j] = pack_bf16(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
          if (c + 1 < c_end) {
            ptx::tmem_ld_32x64(taddr + (c + 1) * 64, r);
          } else {
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&tmem_empty_bar[acc]);
          }
          const int cx = (c - c_begin) * 8;
#pragma unroll
          for (int j = 0; j < 8; ++j)
            *reinterpret_cast<uint4*>(xb + (((cx + j) ^ (lane & xmask)) << 4)) =
                make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
        }
        ptx::named_barrier(2 + pair, 64);  // hand-over; the buffers alternate, so one barrier per tile is enough
      } else {
        ptx::named_barrier(2 + pair, 64);
#pragma unroll 1
        for (int c = c_begin; c < c_end; ++c) {
          // gradient accumulation: this lane's 64 old values (expert e0 + lane, row, 64 columns), zero where
          // the tile leaves the tensor
          uint4 old[8];
          if (ACC) {
            const int e = e0 + lane, col0 = c0 + c * half_col, rowc = row + c * half_row;
            const bool row_ok = e < p.E && rowc < p.rows[k];
            const __nv_bfloat16* src = p.acc_base[k] + (size_t)e * p.e_stride[k] + (size_t)rowc * p.row_stride[k] + col0;
#pragma unroll
            for (int j = 0; j < 8; ++j)
              old[j] = (row_ok && col0 + 8 * j < p.cols[k]) ? *reinterpret_cast<const uint4*>(src + 8 * j)
                                                            : make_uint4(0u, 0u, 0u, 0u);
          }
          ptx::tmem_ld_wait();
          uint32_t w[32];
          const int cx = (c - c_begin) * 8;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 lo4 = *reinterpret_cast<const uint4*>(xb + (((cx + j) ^ (lane & xmask)) << 4));
            const uint32_t lo[4] = {lo4.x, lo4.y, lo4.z, lo4.w};
            const uint32_t ol[4] = {old[j].x, old[j].y, old[j].z, old[j].w};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              float2 l2 = unpack_bf16(lo[t]);
              if (ACC) {
                const float2 o2 = unpack_bf16(ol[t]);
                l2.x += o2.x;
                l2.y += o2.y;
              }
              w[4 * j + t] = pack_bf16(__uint_as_float(r[8 * j + 2 * t]) + l2.x, __uint_as_float(r[8 * j + 2 * t + 1]) + l2.y);
            }
          }
          if (c + 1 < c_end) {
            ptx::tmem_ld_32x64(taddr + (c + 1) * 64, r);
          } else {
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&tmem_empty_bar[acc]);
          }
          warp_stage_and_store(wsg, &maps.out[k], c0 + c * half_col, e0, row + c * half_row, lane, w);
        }
      }
    }
    // the partial dw slab of this CTA
    if (!ptx::mbar_wait(&d2_bar, 0, &abort_flag)) {
      atomicOr(p.status, STATUS_TIMEOUT_EPI);
      abort_flag = 1;
    }
    __syncwarp();  // every lane polls by itself; the warp-wide tcgen05 instructions below need it whole again
    ptx::tc_fence_after_sync();
    float* slab = p.dw_partial + ((size_t)blockIdx.x * p.S_total + p.seg_base) * p.E;
    for (int st = 0; st < p.s_tiles; ++st) {
      const int srow = st * 128 + row_in_tile;
#pragma unroll 1
      for (int c = 0; c * 32 < p.Epad16; ++c) {
        uint32_t r[32];
        ptx::tmem_ld_32x32(tmem_d2 + ((uint32_t)(q * 32) << 16) + st * p.Epad16 + c * 32, r);
        ptx::tmem_ld_wait();
        if (srow < p.S) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c * 32 + j < p.E) {
              float* dst = slab + (size_t)srow * p.E + c * 32 + j;
              *dst = p.slab_add ? *dst + __uint_as_float(r[j]) : __uint_as_float(r[j]);
            }
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
