// Pieces shared by the decode kernels (fp32-FMA, warp-MMA and tcgen05).
#pragma once

#include "common.cuh"
#include "launch.h"

namespace griffin {

constexpr int DEC_CONSUMER_WARPS = 8;
constexpr int DEC_CONSUMERS = DEC_CONSUMER_WARPS * 32;
constexpr int DEC_THREADS = DEC_CONSUMERS + 32;  // + producer warp
constexpr int DEC_MAX_ROWS = 64;                 // rows per work item (neurons / output rows)
constexpr int DEC_DOWN_ITER = 2;                 // 16-byte vectors per consumer thread per row segment
constexpr int DEC_PART_FLOATS = DEC_MAX_ROWS * DEC_CONSUMER_WARPS * 2;  // one parity buffer

struct DecodeSeq {
    const void *w_gate, *w_up, *w_down, *b_gate, *b_up;
};
struct DecodeParams {
    DecodeSeq seq[GRIFFIN_MAX_BATCH];
    const void *b_down;
    const void *x;  // [B, d]
    void *y;        // [B, d]
    float *z;       // [B, ldk] fp32 scratch
    void *ws;       // workspace header (status word), may be null
    int d, k, ldk, B;
    int n_slices;  // work items per sequence
    int n_slices_dn;  // fused bf16 kernel: work items per sequence of the down half
    int n_stages;
    int kt_len;    // down kernel: elements per k-tile (multiple of 8)
    int n_ktiles;
};

struct DecSmem {
    uint8_t *stages;
    uint64_t *full, *empty;
    float *part;
    volatile int *abort;
};

__device__ __forceinline__ DecSmem carve(uint8_t *smem, int n_stages, int stage_bytes) {
    DecSmem s;
    s.stages = smem;
    s.full = reinterpret_cast<uint64_t *>(smem + (size_t)n_stages * stage_bytes);
    s.empty = s.full + n_stages;
    s.part = reinterpret_cast<float *>(s.empty + n_stages);
    s.abort = reinterpret_cast<volatile int *>(s.part + 2 * DEC_PART_FLOATS);
    return s;
}
static inline size_t dec_smem_bytes(int n_stages, int stage_bytes) {
    return (size_t)n_stages * stage_bytes + 2 * n_stages * sizeof(uint64_t) + 2 * DEC_PART_FLOATS * sizeof(float) + 16;
}

__device__ __forceinline__ void consumer_barrier() {
    asm volatile("bar.sync 1, %0;" ::"n"(DEC_CONSUMERS) : "memory");
}

// After its last issue the producer stays until every copy it started has landed, so the
// CTA's shared memory is never released under a copy in flight.  (Only matters after a
// give-up: normally the consumers have already waited for every stage.)
__device__ __forceinline__ void producer_drain(const DecSmem &s, int n_stages, uint32_t issued) {
    const uint32_t first = issued > (uint32_t)n_stages ? issued - n_stages : 0;
    for (uint32_t it = first; it < issued; ++it) {
        const int stage = it % n_stages;
        const uint32_t parity = (it / n_stages) & 1;
        if (mbar_try_wait(&s.full[stage], parity)) continue;
        const long long t0 = clock64();
        while (!mbar_try_wait(&s.full[stage], parity))
            if (clock64() - t0 > WAIT_LIMIT_CYCLES) break;
    }
}


__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int *p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Grid-wide meeting point between the two halves, called by one thread per arriving party
// after the party's z entries have been written and are visible to this thread (a CTA-level
// barrier is enough for that: the fence below is cumulative).  Every call of a kernel adds
// n arrivals to a counter that runs round modulo 2 n and is never reset: a call whose
// arrivals find it below n is complete when it reaches n, the next one when it wraps to 0.
// (A party of the call after next cannot arrive before every party of this call has left:
// all CTAs of a grid must be resident to meet, one per SM.)  Bounded: gives up after
// WAIT_LIMIT_CYCLES.
__device__ __forceinline__ bool grid_meet(unsigned int *counter, unsigned int n, volatile int *abort, void *ws) {
    __threadfence();
    const bool upper = atomicInc(counter, 2 * n - 1) >= n;
    const long long t0 = clock64();
    for (;;) {
        const unsigned int v = ld_acquire_u32(counter);
        if (upper ? v < n : v >= n) return true;
        if (*abort) return false;
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
            *abort = 1;
            raise_status(ws, DEV_STATUS_TIMEOUT, 9);
            return false;
        }
    }
}

// The same in two steps, for a party that has other work to start between reporting in and waiting:
// grid_arrive returns which half of the counter's round this call's arrivals fall into.
__device__ __forceinline__ bool grid_arrive(unsigned int *counter, unsigned int n) {
    __threadfence();
    return atomicInc(counter, 2 * n - 1) >= n;
}
__device__ __forceinline__ bool grid_wait(const unsigned int *counter, unsigned int n, bool upper, volatile int *abort, void *ws) {
    const long long t0 = clock64();
    for (;;) {
        const unsigned int v = ld_acquire_u32(counter);
        if (upper ? v < n : v >= n) return true;
        if (*abort) return false;
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
            *abort = 1;
            raise_status(ws, DEV_STATUS_TIMEOUT, 9);
            return false;
        }
    }
}

// The arrival alone, for a party that has given up on its work: the other parties of this launch are not
// held up by it and the counter stays in phase for the next launch.
__device__ __forceinline__ void grid_arrive_only(unsigned int *counter, unsigned int n) {
    __threadfence();
    atomicInc(counter, 2 * n - 1);
}

// Launches `func`, optionally allowing it to start before the previous kernel on the stream
// has completed (programmatic dependent launch).
cudaError_t launch_maybe_overlapped(const void *func, dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    bool overlap, void **args);

// Number of work items per sequence: a multiple of the grid, fine enough that one item has at
// most DEC_MAX_ROWS rows.
int slices_for(int rows, int grid);

// bf16 decode through warp-level MMA (decode_mma.cu).
// act: the code of sigma (0..3); gated: whether the block has a gate (Eq. 3) or not (Eq. 2).
griffin_status decode_bf16_mma(DecodeParams &p, int act, bool gated, uint32_t flags, cudaStream_t stream);

// bf16 decode streamed through registers, without a shared-memory ring (decode_stream.cu).
griffin_status decode_bf16_stream(DecodeParams &p, int act, bool gated, uint32_t flags, cudaStream_t stream);

// bf16 decode of a batch that shares one expert set (decode_shared.cu): the weights are streamed once per
// pass of up to 8 vectors, which are the columns of the warp-level MMA.
bool decode_shared_set(const DecodeParams &p);  // 2 or more sequences that all name the same buffers
griffin_status decode_bf16_shared(DecodeParams &p, int act, bool gated, uint32_t flags, cudaStream_t stream);

// bf16 decode through tcgen05 (decode_tc.cu): d and ldk multiples of 128, a workspace for the
// meeting point.
bool decode_tc_supported(const DecodeParams &p);
bool decode_tc_shared(const DecodeParams &p);  // 2..8 sequences that all use one expert set: streamed once for all
griffin_status decode_bf16_tc(DecodeParams &p, int act, uint32_t flags, cudaStream_t stream);

}  // namespace griffin
