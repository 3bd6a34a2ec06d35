// Warp-level tensor-core (mma.sync) machinery shared by the decode kernels that stream weight
// rows through a ring of shared-memory stages: stage geometry, the "virtual row" product of a
// pair of staged rows with a vector, and the ring bookkeeping of the two consumer groups.
#pragma once

#include "decode_common.cuh"

namespace griffin {

constexpr int DEC_GROUP_WARPS = 4;           // consumer warps per group (two groups)
constexpr int MMA_CHUNK_UNITS_MAX = 1024;  // 16 KB of one row per stage at most
#ifndef GRIFFIN_DEC_STAGE_KB
#define GRIFFIN_DEC_STAGE_KB 32
#endif
constexpr int MMA_STAGE_TARGET = GRIFFIN_DEC_STAGE_KB * 1024;
#ifndef GRIFFIN_DEC_SMEM_KB
#define GRIFFIN_DEC_SMEM_KB 227
#endif
constexpr int MMA_SMEM_TARGET = GRIFFIN_DEC_SMEM_KB * 1024;  // shared memory the ring, the vector and the rest may take

struct MmaPlan {
    int row_units;    // 16-byte units per real row
    int n_chunks;     // pieces a row is cut into
    int chunk_units;  // units per piece (the last may be shorter)
    int R;            // pairs per stage: 1, 2 or 4
    int stage_bytes;
    int n_stages;
    int vec_bytes;
};

struct MmaSmem {
    uint8_t *stages;
    uint8_t *vec;  // gate_up: x as bf16 [d]; down: z_hi [ldk] then z_lo [ldk]
    uint64_t *full, *empty;
    float2 *part;  // [2 parities][DEC_MAX_ROWS pairs][8 warps]
    volatile int *abort;
};
__device__ __forceinline__ MmaSmem carve_mma(uint8_t *smem, const MmaPlan &pl) {
    MmaSmem s;
    s.stages = smem;
    s.vec = smem + (size_t)pl.n_stages * pl.stage_bytes;
    s.full = reinterpret_cast<uint64_t *>(s.vec + pl.vec_bytes);
    s.empty = s.full + pl.n_stages;
    s.part = reinterpret_cast<float2 *>(s.empty + pl.n_stages);
    s.abort = reinterpret_cast<volatile int *>(s.part + 2 * DEC_MAX_ROWS * DEC_CONSUMER_WARPS);
    return s;
}
static inline size_t mma_fixed_smem(int n_stages) {
    return 2 * n_stages * sizeof(uint64_t) + 2 * DEC_MAX_ROWS * DEC_CONSUMER_WARPS * sizeof(float2) + 16;
}

static inline MmaPlan make_plan(int row_elems, int vec_bytes, int stage_target, int blocks_per_warp) {
    MmaPlan pl;
    pl.row_units = row_elems / 8;
    pl.n_chunks = (pl.row_units + MMA_CHUNK_UNITS_MAX - 1) / MMA_CHUNK_UNITS_MAX;
    pl.chunk_units = (pl.row_units + pl.n_chunks - 1) / pl.n_chunks;
    const int pair_bytes = 2 * pl.chunk_units * 16;
    pl.R = pair_bytes * 4 <= stage_target ? 4 : (pair_bytes * 2 <= stage_target ? 2 : 1);
    // the DEC_GROUP_WARPS / R warps that share a pair must not get more blocks than they have registers for
    const int row_blocks = (pl.chunk_units + 31) / 32;
    while (pl.R > 1 && (row_blocks + DEC_GROUP_WARPS / pl.R - 1) / (DEC_GROUP_WARPS / pl.R) > blocks_per_warp) pl.R >>= 1;
    pl.stage_bytes = pl.R * pair_bytes;
    pl.vec_bytes = vec_bytes;
    int n = ((int)MMA_SMEM_TARGET - vec_bytes - (int)mma_fixed_smem(8)) / pl.stage_bytes;
    pl.n_stages = n < 2 ? 2 : (n > 8 ? 8 : n);
    return pl;
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Adds the diagonal of the 16 x 8 accumulator tile: the sum over g of C[g][g] ends up in lane
// 0 and the sum over g of C[g + 8][g] in lane 4 (the value returned by other lanes means
// nothing).  Lane (g, t) holds columns 2t, 2t+1 of rows g, g+8, so the 8 lanes that hold a
// diagonal entry are 0, 4, 9, 13, 18, 22, 27, 31.  In the first exchange (xor 4) the lower
// lane of each couple hands over its second-row entry and takes the partner's first-row
// entry, so that from then on each lane carries one sum and three shuffles do for both rows.
__device__ __forceinline__ float diagonal_sum(const float (&c)[4], int lane) {
    const int g = lane >> 2, t = lane & 3;
    float v0 = 0.f, v1 = 0.f;
    if (t == (g >> 1)) {
        v0 = (g & 1) ? c[1] : c[0];
        v1 = (g & 1) ? c[3] : c[2];
    }
    const bool lower = (lane & 4) == 0;
    const float got = __shfl_xor_sync(0xffffffffu, lower ? v1 : v0, 4);
    float v = (lower ? v0 : v1) + got;
    v += __shfl_xor_sync(0xffffffffu, v, 9);
    v += __shfl_xor_sync(0xffffffffu, v, 18);
    return v;
}

// This warp's share of one pair's chunk: blocks q, q + WPG, ... of 32 units each, never more
// than MMA_BLOCKS_PER_WARP of them (a stage holds at most 32 / R blocks per row and the
// WPG = 4 / R warps of a consumer group share the pair).  The kernel is bound by the number of
// instructions its few warps can issue, so the common case is kept to the loads and the MMAs
// themselves: blocks are taken in batches of four whole blocks with no predicates and
// compile-time offsets from per-lane base pointers; only what is left after the last whole
// batch (at most four blocks, the last of which may be cut short by the end of the row) takes
// the guarded path, where lanes past the end supply zeros (stale bytes could be NaN).  All
// shared-memory reads of a batch are issued before its first MMA, and the MMAs go to four
// independent accumulators, so latencies overlap instead of adding up.
//   p0, p1 : this lane's unit of the first block of the two staged rows; pv, pw : the same for
//   the vector held in shared memory (down: z_hi and z_lo); xr : the vector's units held in
//   registers (gate_up, where x is the same for every neuron of the item); my_full : whole
//   blocks of this warp; tail_lanes : lanes with data in the block after them (0: no such block)
constexpr int MMA_BLOCKS_PER_WARP = 8;
// The second half takes larger stages (two pairs of rows of W_2_hat where one pair is more than
// half a first-half stage): every stage costs its consumers a fixed round of waiting, reducing
// and handing back, and this half runs at their pace.  A warp then has up to 12 blocks.
#ifndef GRIFFIN_DEC_DOWN_STAGE_KB
#define GRIFFIN_DEC_DOWN_STAGE_KB 48
#endif
constexpr int MMA_BLOCKS_PER_WARP_DOWN = 12;
template <bool DOWN> struct BlocksPerWarp { static constexpr int N = DOWN ? MMA_BLOCKS_PER_WARP_DOWN : MMA_BLOCKS_PER_WARP; };
#ifndef GRIFFIN_DEC_BATCH
#define GRIFFIN_DEC_BATCH 4
#endif
#ifndef GRIFFIN_DEC_ACCS
#define GRIFFIN_DEC_ACCS 8
#endif
constexpr int MMA_BATCH = GRIFFIN_DEC_BATCH;
constexpr int MMA_ACCS = GRIFFIN_DEC_ACCS;
// Whether z crosses the halves as two bf16 numbers z_hi + z_lo per entry (every block of
// W_2_hat then meets both, at twice the MMAs) or as one, rounded to bf16 like the Z that the
// prompt-phase kernels hand to their second GEMM.  The second half is bound by its own
// instructions, not by HBM, and the extra bits are below the rounding of the bf16 output.
#ifndef GRIFFIN_DEC_Z_LO
#define GRIFFIN_DEC_Z_LO 0
#endif
constexpr bool Z_LO = GRIFFIN_DEC_Z_LO != 0;  // independent accumulators: an MMA never waits for the one issued just before it
// The MMAs of one batch: first every block against v, then (down) every block against w, so
// that two MMAs into the same accumulator are MMA_ACCS instructions apart.
template <bool DOWN, int N>
__device__ __forceinline__ void batch_mma(float (&acc)[MMA_ACCS][4], const uint4 (&r0)[MMA_BATCH],
                                          const uint4 (&r1)[MMA_BATCH], const uint4 (&v)[MMA_BATCH],
                                          const uint4 (&w)[MMA_BATCH]) {
#pragma unroll
    for (int i = 0; i < N; ++i) {
        mma_bf16(acc[(2 * i) & (MMA_ACCS - 1)], r0[i].x, r1[i].x, r0[i].y, r1[i].y, v[i].x, v[i].y);
        mma_bf16(acc[(2 * i + 1) & (MMA_ACCS - 1)], r0[i].z, r1[i].z, r0[i].w, r1[i].w, v[i].z, v[i].w);
    }
    if (DOWN && Z_LO) {
#pragma unroll
        for (int i = 0; i < N; ++i) {
            mma_bf16(acc[(2 * i) & (MMA_ACCS - 1)], r0[i].x, r1[i].x, r0[i].y, r1[i].y, w[i].x, w[i].y);
            mma_bf16(acc[(2 * i + 1) & (MMA_ACCS - 1)], r0[i].z, r1[i].z, r0[i].w, r1[i].w, w[i].z, w[i].w);
        }
    }
}
// VREG: the vector's units come from the registers xr (and wr for down's z_lo) instead of
// shared memory.
template <bool DOWN, bool VREG, int WPG>
__device__ __forceinline__ void pair_mma(float (&acc)[MMA_ACCS][4], const uint4 *p0, const uint4 *p1, const uint4 *pv,
                                         const uint4 *pw, const uint4 (&xr)[BlocksPerWarp<DOWN>::N],
                                         const uint4 (&wr)[BlocksPerWarp<DOWN>::N], int my_full, int tail_lanes,
                                         int lane) {
    constexpr int BS = WPG * 32;  // units between consecutive blocks of this warp
#pragma unroll
    for (int b0 = 0; b0 < BlocksPerWarp<DOWN>::N; b0 += MMA_BATCH) {
        uint4 r0[MMA_BATCH], r1[MMA_BATCH], v[MMA_BATCH], w[MMA_BATCH];
        if (b0 + MMA_BATCH <= my_full) {  // warp-uniform: four whole blocks
#pragma unroll
            for (int i = 0; i < MMA_BATCH; ++i) {
                r0[i] = p0[(b0 + i) * BS];
                r1[i] = p1[(b0 + i) * BS];
                if (VREG) {
                    v[i] = xr[b0 + i];
                    if (DOWN && Z_LO) w[i] = wr[b0 + i];
                } else {
                    v[i] = pv[(b0 + i) * BS];
                    if (DOWN && Z_LO) w[i] = pw[(b0 + i) * BS];
                }
            }
            batch_mma<DOWN, MMA_BATCH>(acc, r0, r1, v, w);
        } else if (b0 == 0 || b0 <= my_full) {  // a shorter batch ends the warp's blocks
            const int n = my_full - b0 + (tail_lanes > 0 ? 1 : 0);  // blocks left, the cut one included
            if (n > 0) {
                const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int i = 0; i < MMA_BATCH; ++i) {
                    if (b0 + i >= my_full) {  // warp-uniform: only the cut block needs zeros
                        r0[i] = zero; r1[i] = zero; v[i] = zero; w[i] = zero;
                    }
                    if (b0 + i < my_full || (i < n && lane < tail_lanes)) {
                        r0[i] = p0[(b0 + i) * BS];
                        r1[i] = p1[(b0 + i) * BS];
                        if (!VREG) {
                            v[i] = pv[(b0 + i) * BS];
                            if (DOWN && Z_LO) w[i] = pw[(b0 + i) * BS];
                        }
                    }
                    if (VREG) {  // (zero past the end of the row)
                        v[i] = xr[b0 + i];
                        if (DOWN && Z_LO) w[i] = wr[b0 + i];
                    }
                }
                // warp-uniform
                if (n == 1) batch_mma<DOWN, 1>(acc, r0, r1, v, w);
                else if (n == 2) batch_mma<DOWN, (2 < MMA_BATCH ? 2 : MMA_BATCH)>(acc, r0, r1, v, w);
                else if (n == 3) batch_mma<DOWN, (3 < MMA_BATCH ? 3 : MMA_BATCH)>(acc, r0, r1, v, w);
                else batch_mma<DOWN, MMA_BATCH>(acc, r0, r1, v, w);
            }
        }
    }
}

// Whole blocks of warp q (of WPG) among the blocks of a chunk of `units` units, and the lanes
// with data in its cut block, if the chunk's cut block is this warp's.
template <int WPG>
__device__ __forceinline__ void my_blocks(int units, int q, int &my_full, int &tail_lanes) {
    const int whole = units >> 5, rem = units & 31;
    my_full = whole > q ? (whole - q + WPG - 1) / WPG : 0;
    tail_lanes = (rem != 0 && (whole % WPG) == q) ? rem : 0;
}

__device__ __forceinline__ void producer_drain_mma(const MmaSmem &s, int n_stages, const uint32_t (&issued)[2]) {
    const int ns2 = n_stages >> 1;
    for (int grp = 0; grp < 2; ++grp) {
        const uint32_t first = issued[grp] > (uint32_t)ns2 ? issued[grp] - ns2 : 0;
        for (uint32_t it = first; it < issued[grp]; ++it) {
            const int stage = grp * ns2 + (int)(it % ns2);
            const uint32_t parity = (it / ns2) & 1;
            if (mbar_try_wait(&s.full[stage], parity)) continue;
            const long long t0 = clock64();
            while (!mbar_try_wait(&s.full[stage], parity))
                if (clock64() - t0 > WAIT_LIMIT_CYCLES) break;
        }
    }
}

// Position of one consumer group in its half of the ring: the slot used next, how often the
// half has been gone round (its low bit is the barrier parity) and the uses so far.
struct RingPos {
    int slot;
    uint32_t round;
    uint32_t uses;
    __device__ __forceinline__ void advance(int ns2) {
        ++uses;
        if (++slot == ns2) {
            slot = 0;
            ++round;
        }
    }
};

// barrier among the 128 threads of one consumer group (ids 2 and 3; 0 is __syncthreads, 1 all consumers)
__device__ __forceinline__ void group_barrier(int group) {
    asm volatile("bar.sync %0, %1;" ::"r"(2 + group), "n"(DEC_GROUP_WARPS * 32) : "memory");
}

}  // namespace griffin
