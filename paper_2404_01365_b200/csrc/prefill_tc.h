// Tensor-core (tcgen05 / TMEM / TMA) path of the prompt-phase FF for bf16 storage.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "griffin_ff.h"

namespace griffin {

// Tiling of the down projection Y = Z W_2^T for S tokens: tile width (128 or 256 outputs) and the
// number of K splits (1..4; more than one when that fills the SMs better than whole tiles and the
// fp32 partial sums cost less than it saves).  Pure arithmetic on the shape, so that workspace sizing
// and launch agree.
void gemm2_plan(int S, int d, int d_ff, int *bn, int *splits);

// Column tiles of the first GEMM: 128 neurons each with a gate (gate | up side by side in the
// accumulator), 256 without.
int gemm1_col_tiles(const griffin_ff_desc *desc);

// The first GEMM has m_tiles x n_col_tiles tiles for one CTA per SM.  When the last round of
// tiles would leave more than half of the SMs idle, those tiles are cut along K into *ks parts
// (2..4) whose fp32 partial accumulators meet in a small finishing kernel: *tail_first is the
// first tile that is cut (= the number of tiles when none is).  Pure arithmetic on the shape.
void gemm1_tail_plan(int S, int d, int n_col_tiles, int *tail_first, int *ks);
// Bytes of fp32 scratch that the parts of the cut tiles need (0 when none is cut).
size_t gemm1_tail_bytes(int S, int d, int n_col_tiles);

// The same cut for the last round of the down projection's tiles (whole tiles 256 outputs wide only).
void gemm2_tail_plan(int S, int d, int d_ff, int *tail_first, int *ks);
size_t gemm2_tail_bytes(int S, int d, int d_ff);

// Whether the tensor-core kernels take this shape (bf16, d and d_ff multiples of 64, ...).
bool prefill_tc_supported(const griffin_ff_desc *desc, int S);

// Steps 1 and 2 of the prompt phase: writes Z (bf16), the bf16 residual zlo = z - bf16(z) and the per-tile partial
// row sums of squares rowsq [S, *n_col_tiles]; writes Y unless y is NULL.  after_ff1 (may be
// NULL) is recorded on the stream between the two GEMMs: what only needs Z may start there.
griffin_status launch_prefill_tc(const griffin_ff_desc *desc, const griffin_ff_weights *w, const void *x, int S,
                                 void *y, __nv_bfloat16 *z, __nv_bfloat16 *zlo, float *rowsq, float *ypart, int *n_col_tiles, void *ws,
                                 cudaStream_t stream, cudaEvent_t after_ff1);

}  // namespace griffin
