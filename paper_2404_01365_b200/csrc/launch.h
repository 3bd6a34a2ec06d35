// Host-side launchers behind the C ABI (one per kernel family).  Arguments are already
// validated by the caller in api.cu.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "griffin_ff.h"

namespace griffin {

// Number of SMs of the current device (cached per device); <= 0 on error.
int device_sm_count();

// Adds n to the count of kernels this library has launched in this process (griffin_kernel_launches).
void count_launches(int n);

// Launches `func` (counted), optionally as a programmatic dependent launch: it may then be scheduled before the
// previous kernel on the stream has completed, and must itself wait (griddepcontrol.wait) before it touches
// anything that kernel writes.
cudaError_t launch_maybe_overlapped(const void *func, dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool overlap,
                                    void **args);

// Raises the opt-in dynamic shared memory limit of `fn` on the current device when needed.
cudaError_t ensure_dynamic_smem(const void *fn, size_t bytes);

// Whether a grid of `grid` CTAs of this kernel, with this many threads and this much dynamic shared memory, can be
// resident on the current device all at once (what the kernels whose CTAs meet through a counter need; call it
// after ensure_dynamic_smem).  A host-side occupancy query, remembered per kernel and shared-memory size.
bool grid_can_meet(const void *fn, int threads, size_t smem, int grid);

griffin_status launch_decode(const griffin_ff_desc *desc, int B, const griffin_ff_compact *sets, const void *b_down,
                             const void *x, void *y, float *z, void *ws, uint32_t flags, cudaStream_t stream);

// Decode with the z scratch in the library's own static device array (no workspace).
griffin_status launch_decode_static(const griffin_ff_desc *desc, int B, const griffin_ff_compact *sets,
                                    const void *b_down, const void *x, void *y, uint32_t flags, cudaStream_t stream);

// Status word in front of the current device's static array; clears the header when it was raised.
griffin_status static_scratch_status(cudaStream_t stream);

// Index-direct decode (decode_indexed.cu): expert rows read in place from neuron-major weights.
constexpr int IDX_MAX_GRID = 148;  // CTAs (= partial-sum rows per sequence in the workspace) at most
size_t decode_indexed_scratch_bytes(int d, int n_seq);
griffin_status launch_decode_indexed(const griffin_ff_desc *desc, int B, const griffin_ff_weights_nm *w,
                                     const int32_t *idx, int k, const void *x, void *y, float *ypart, void *ws,
                                     uint32_t flags, cudaStream_t stream);

griffin_status launch_select_topk(const float *score, int n_seq, int d_ff, int k, int32_t *idx, cudaStream_t stream);

griffin_status launch_combine_scores(const float *score, const int32_t *prompt_len_host, int n_seq, int d_ff,
                                     float *out, cudaStream_t stream);

griffin_status launch_compact(const griffin_ff_desc *desc, const griffin_ff_weights *w, const int32_t *idx,
                              const griffin_ff_compact *out, void *ws, cudaStream_t stream);

griffin_status launch_compact_nm(const griffin_ff_desc *desc, const griffin_ff_weights_nm *w, const int32_t *idx,
                                 const griffin_ff_compact *out, void *ws, cudaStream_t stream);

// Carve-up of the workspace behind its header for the prompt-phase path.
struct PrefillScratch {
    size_t z_off, zf_off, rowsq_off, inv_off, colpart_off, ypart_off, total;  // byte offsets from the scratch base
    int n_col_tiles;                                        // partial row sums kept per token
    int n_row_chunks;                                       // partial column sums kept per neuron
};
PrefillScratch prefill_scratch(const griffin_ff_desc *desc, int S);

// sumsq (may be NULL): running sum of squares of the statistic over the pieces of a prompt; `first`
// starts it afresh.  score may be NULL when sumsq is given.
griffin_status launch_prefill_score(const griffin_ff_desc *desc, const griffin_ff_weights *w, const void *x, int S,
                                    void *y, float *score, float *sumsq, int first, uint8_t *scratch, void *ws,
                                    cudaStream_t stream);

}  // namespace griffin
