// Tensor-core (tcgen05 / TMEM / TMA) pipeline of the bf16 mode.
#pragma once
#include "common.cuh"
#include "layout.cuh"

namespace lory {

// Bytes of the bf16 hi/lo split of the routing weights kept in the workspace.
size_t tc_w_split_bytes(const lory_dims& D);
// Whether the tensor-core pipeline covers this problem (else the plain-FMA pipeline runs).
bool tc_supported(const lory_dims& D);
// Elements of the blocked layout of a per-segment [R, C] matrix over all segments.
size_t tc_blocked_elems(const lory_dims& D, int R, int C);
// Elements of the buffer the chunked adjoint (LORY_FLAG_CHUNKED_ADJOINT) keeps one rectangle of per-segment weight
// gradients in: sized from the device's L2 (environment variable LORY_ADJOINT_CHUNK_MB overrides the budget).
size_t tc_adjoint_ring_elems(const lory_dims& D);
// Number of [S,E] partial slabs the tensor-core dw contraction writes.
int tc_dw_slabs(const lory_dims& D);

// Where the bf16 hi / lo tables of the routing weights live in the workspace ([S, *Epad] each), and the
// combined [S, 64] table (NULL unless E <= 32).  The routing step may fill them directly.
void tc_split_tables(const lory_dims& D, const Layout& Lo, char* ws, bf16** hi, bf16** lo, bf16** comb, int* Epad);

// Merge + merged SwiGLU FFN forward (Eq. 2; Section 3.1).  ws holds the regions of Lo.
// w_is_split: the hi / lo tables are already filled (else they are derived here from the fp32 weights).
// residual (optional, [tokens, d]): added to y in the epilogue of the last GEMM.
int tc_ffn_forward(const lory_dims& D, const Layout& Lo, char* ws, const bf16* x, const bf16* w1, const bf16* w2,
                   const bf16* w3, bf16* y, cudaStream_t st, bool w_is_split = false,
                   const bf16* residual = nullptr);

// Backward of the merged FFNs (all but dX) and of the merge; leaves Lo.n_slabs partial dw slabs in the workspace.
int tc_ffn_backward(const lory_dims& D, const Layout& Lo, char* ws, const bf16* x, const bf16* w1, const bf16* w2,
                    const bf16* w3, const bf16* dy, bf16* dw1, bf16* dw2, bf16* dw3, cudaStream_t st);
// dX = dG Wbar1 + dU Wbar3 + dh_bar/T; runs after the router backward has produced dh_bar [S, d].
int tc_ffn_backward_dx(const lory_dims& D, const Layout& Lo, char* ws, const float* dh_bar, bf16* dx,
                       cudaStream_t st);

// Evaluates the debug build's three kinds of bounds check on made-up out-of-range values (no access is made):
// raises STATUS_DEBUG_BOUNDS in a debug build, nothing in a release build.
int tc_debug_bounds_selftest(uint32_t* status_word, cudaStream_t st);

// Launches a one-thread kernel whose bounded mbarrier wait must expire and raise the status word.
int tc_bounded_wait_selftest(uint32_t* status_word, cudaStream_t st);

}  // namespace lory
