// Generation-phase pruned FF (Eqs. 4 and 5 of the GRIFFIN paper) for bf16 storage, as ONE kernel
// per call:
//   first half   z_hat = sigma(W_g_hat x + b_g_hat) * (W_1_hat x + b_1_hat)
//   meeting      every CTA has written its z entries; all CTAs wait for each other (bounded)
//   second half  y_hat = W_2_hat z_hat + b_2
//
// One persistent CTA per SM.  A producer warp streams weight rows into a ring of
// shared-memory stages with 1-D bulk copies (TMA, no multicast) tracked by mbarriers; it
// touches weights only, so it runs ahead of the previous kernel on the stream (programmatic
// dependent launch) and of the meeting point.  Eight consumer warps, in two groups that take
// alternate stages, hand the staged rows to the warp-level tensor-core instruction
// mma.sync.m16n8k16 instead of unpacking and multiplying element by element.  The products are
// matrix-vector products, so this is not about FLOPs: it cuts the instructions issued per
// staged byte several times over, which is what kept an FMA version from reaching HBM speed.
//
// Stages are made of few, large, contiguous copies (measured on B200: every bulk copy costs
// about 30 ns of issue time and every stage hand-over about 240 ns, whatever their size, so
// a stage should carry 24-32 KB in two to four copies).  A stage therefore holds R "pairs"
// of whole rows (or 16 KB chunks of long rows): for gate_up a pair is (gate row j, up row
// j), for down it is (row c, row c+1) of W_2_hat.  Both rows of a pair meet the same vector
// (x, or z).
//
// How one pair meets the vector in the MMA (M = 16, N = 8, K = 16):
//   * A row is a sequence of 16-byte units (8 elements).  In a block of 32 units, lane l of
//     a warp reads unit l of both rows and of the vector: every 8 consecutive lanes read 128
//     contiguous bytes, so there are no bank conflicts and nothing needs padding.
//   * With g = lane / 4 and t = lane % 4, the MMA takes the lane's row data as rows g
//     (first real row) and g + 8 (second real row) of A, and its vector data as column g
//     of B, both at K positions 2t, 2t+1, 2t+8, 2t+9: "virtual row" g of a real row is the
//     set of units read by lanes 4g..4g+3, "virtual vector" g the matching units of x (or
//     z).  The unit's first four elements feed one MMA and the last four a second one (the
//     MMA sums over K, so any assignment of elements to K positions works as long as the
//     row and the vector agree, and here the same lane supplies both).
//   * C[m][n] pairs virtual row m with virtual vector n; only the diagonal m = n belongs to
//     the dot product.  Lane (g, t = g / 2) holds it; three shuffles add the 8 diagonal
//     entries.  The tensor core does 8x the needed multiplies, which is free here.
//   * second half: z crosses in bf16 (with GRIFFIN_DEC_Z_LO as two bf16 numbers z_hi + z_lo
//     per entry; each block then runs the MMAs once against each, into the same accumulators).
//   * The 4 / R warps of a group share a pair; their partial sums meet in shared memory at
//     the end of a work item, in a fixed order, so results are bitwise reproducible.
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
static size_t mma_fixed_smem(int n_stages) {
    return 2 * n_stages * sizeof(uint64_t) + 2 * DEC_MAX_ROWS * DEC_CONSUMER_WARPS * sizeof(float2) + 16;
}

static MmaPlan make_plan(int row_elems, int vec_bytes, int stage_target, int blocks_per_warp) {
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

// The two halves of a decode call share one kernel, one ring and one stage counter:
//   DOWN = false: gate_up, z[b, j] = sigma(gate_j . x + b_gate_j) * (up_j . x + b_up_j);
//                 item = (sequence, slice of neurons), pair = neuron.
//   DOWN = true : down, y[b, c] = w_down_c[c, :] . z[b] + b_down[c];
//                 item = (sequence, chunk of output rows), pair = two consecutive rows.
struct FusedPlan {
    MmaPlan gu, dn;   // per-half geometry (their n_stages / stage_bytes are overridden below)
    int slot_bytes;   // ring slot = the larger of the two halves' stages
    int n_stages;
    int vec_bytes;    // z_hi | z_lo (ldk * 4) when it is staged in shared memory
};

__device__ __forceinline__ MmaSmem carve_fused(uint8_t *smem, const FusedPlan &fp) {
    MmaSmem s;
    s.stages = smem;
    s.vec = smem + (size_t)fp.n_stages * fp.slot_bytes;
    s.full = reinterpret_cast<uint64_t *>(s.vec + fp.vec_bytes);
    s.empty = s.full + fp.n_stages;
    s.part = reinterpret_cast<float2 *>(s.empty + fp.n_stages);
    s.abort = reinterpret_cast<volatile int *>(s.part + 2 * DEC_MAX_ROWS * DEC_CONSUMER_WARPS);
    return s;
}

// Producer side of one half.  Lane l < 2R copies row (l & 1) of pair (l >> 1).  Weights only.
template <bool DOWN>
__device__ __forceinline__ bool produce_half(const DecodeParams &p, const MmaPlan &plan, const MmaSmem &s, int n_stages,
                                             int slot_bytes, int n_slices, RingPos (&pos)[2], uint32_t &pgc, int lane) {
    const MmaPlan pl = plan;  // in registers: the asm statements in the loops clobber memory, and a reload costs a round trip
    void *const ws = p.ws;
    const int n_items = p.B * n_slices;
    const int total_rows = DOWN ? p.d : p.k;
    const int ns2 = n_stages >> 1;
    const size_t row_bytes = (size_t)pl.row_units * 16;
    const int chunk_bytes_max = pl.chunk_units * 16;
    const int my_pair = lane >> 1, my_row = lane & 1;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int b = item / n_slices, sl = item - b * n_slices;
        const int r0 = (int)((long long)sl * total_rows / n_slices);
        const int r1 = (int)((long long)(sl + 1) * total_rows / n_slices);
        const int n_pairs = DOWN ? (r1 - r0 + 1) / 2 : r1 - r0;
        const uint8_t *mat =
            static_cast<const uint8_t *>(DOWN ? p.seq[b].w_down : (my_row ? p.seq[b].w_up : p.seq[b].w_gate));
        for (int pg = 0; pg < n_pairs; pg += pl.R, ++pgc) {
            // consumer group (pgc & 1) owns this pair group; each group has its own half of the
            // ring and its own count of stage uses, so that every barrier sees one strictly
            // sequential user (a group skipping over the other's stages would otherwise wait on
            // a parity that an older phase already satisfies)
            const int grp = pgc & 1;
            const int pair = pg + my_pair;
            const int grow = DOWN ? r0 + 2 * pair + my_row : r0 + pair;  // row in the matrix
            const bool mine = lane < 2 * pl.R && pair < n_pairs && grow < r1;
            // rows copied in this stage (the same for every chunk of the group)
            const int rows_in_stage = DOWN ? min(2 * pl.R, r1 - r0 - 2 * pg) : 2 * min(pl.R, n_pairs - pg);
            RingPos cur = grp ? pos[1] : pos[0];  // (constant indices keep both in registers)
            for (int c = 0; c < pl.n_chunks; ++c, cur.advance(ns2)) {
                const int units = min(pl.chunk_units, pl.row_units - c * pl.chunk_units);
                const int stage = grp * ns2 + cur.slot;
                const uint32_t use = cur.round;
                int go = 1;
                if (lane == 0) {
                    if (use > 0 && !wait_or_abort(&s.empty[stage], (use - 1) & 1, s.abort, ws, DOWN ? 7 : 5)) go = 0;
                    if (go) mbar_arrive_expect_tx(&s.full[stage], (uint32_t)(rows_in_stage * units * 16));
                }
                go = __shfl_sync(0xffffffffu, go, 0);
                if (!go) {
                    if (grp) pos[1] = cur; else pos[0] = cur;
                    return false;
                }
                if (mine)
                    bulk_g2s(s.stages + (size_t)stage * slot_bytes + (size_t)lane * chunk_bytes_max,
                             mat + (size_t)grow * row_bytes + (size_t)c * chunk_bytes_max, (uint32_t)units * 16,
                             &s.full[stage]);
            }
            if (grp) pos[1] = cur; else pos[0] = cur;
        }
    }
    return true;
}

// barrier among the 128 threads of one consumer group (ids 2 and 3; 0 is __syncthreads, 1 all consumers)
__device__ __forceinline__ void group_barrier(int group) {
    asm volatile("bar.sync %0, %1;" ::"r"(2 + group), "n"(DEC_GROUP_WARPS * 32) : "memory");
}

// Consumer side of one half (all 8 consumer warps).  Returns false after a give-up.
// VREG: a row is one chunk, so every stage of an item meets the same units of the vector and
// each lane keeps its units of it in registers (read straight from global memory, once per
// item); otherwise (rows longer than MMA_CHUNK_UNITS_MAX units, down only) the vector is
// staged in shared memory and read from there block by block.
template <bool DOWN, bool VREG, int WPG>
__device__ __forceinline__ bool consume_half(const DecodeParams &p, const MmaPlan &plan, const MmaSmem &s, int n_stages,
                                             int slot_bytes, int n_slices, RingPos &pos, uint32_t &pgc,
                                             int &item_parity, int act, int tid, int warp, int lane) {
    const MmaPlan pl = plan;  // in registers: the asm statements in the loops clobber memory, and a reload costs a round trip
    void *const ws = p.ws;
    const int n_items = p.B * n_slices;
    const int total_rows = DOWN ? p.d : p.k;
    const int chunk_bytes_max = pl.chunk_units * 16;
    // The 8 consumer warps form two groups of 4 that take alternate stages (pair groups), so
    // that one group's waiting, shuffling and hand-back overlaps the other group's reads.
    const int group = warp / DEC_GROUP_WARPS, wig = warp - group * DEC_GROUP_WARPS;
    constexpr int wpg = WPG;  // warps of a group per pair (4 / R)
    const int ns2 = n_stages >> 1;
    const int my_pair = wig / wpg, q = wig - my_pair * wpg;
    // this lane's unit of this warp's first block, within a staged row and within the vector
    const int lane_unit = q * 32 + lane;
    int my_full, tail_lanes;  // this warp's blocks of a chunk (all chunks but a row's last are alike)
    my_blocks<WPG>(pl.chunk_units, q, my_full, tail_lanes);
    // the scratch holds, per sequence, z_hi [ldk] then z_lo [ldk] in bf16 (same bytes as fp32 [ldk])
    __nv_bfloat16 *zbits = reinterpret_cast<__nv_bfloat16 *>(p.z);
    int cur_b = -1;
    uint4 xr[BlocksPerWarp<DOWN>::N], wr[BlocksPerWarp<DOWN>::N];  // x, or z_hi and z_lo
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, item_parity ^= 1) {
        const int b = item / n_slices, sl = item - b * n_slices;
        const int r0 = (int)((long long)sl * total_rows / n_slices);
        const int r1 = (int)((long long)(sl + 1) * total_rows / n_slices);
        const int n_pairs = DOWN ? (r1 - r0 + 1) / 2 : r1 - r0;
        float2 *part = s.part + item_parity * (DEC_MAX_ROWS * DEC_CONSUMER_WARPS);
        const uint32_t pgc0 = pgc;  // pair-group count at the start of the item: who owns which pair
        // the groups finish an item independently; before a further item (partial-sum buffers
        // and the staged vector are about to be reused) they meet
        if (item != (int)blockIdx.x) consumer_barrier();
        if (b != cur_b) {  // this sequence's vector: x, or z_hi [ldk] then z_lo [ldk]
            // (x was written by earlier work on the stream, z by other CTAs of this grid: both
            // are read through L2)
            const uint4 *src = DOWN ? reinterpret_cast<const uint4 *>(zbits + (size_t)b * 2 * p.ldk)
                                    : reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(p.x) +
                                                                      (size_t)b * p.d);
            if (VREG) {
                const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int i = 0; i < BlocksPerWarp<DOWN>::N; ++i) {
                    const int u = i * (WPG * 32) + lane_unit;
                    xr[i] = u < pl.row_units ? __ldcg(src + u) : zero;
                    if (DOWN && Z_LO) wr[i] = u < pl.row_units ? __ldcg(src + pl.row_units + u) : zero;
                }
            } else {
                for (int v = tid; v < (DOWN && Z_LO ? 2 : 1) * pl.row_units; v += DEC_CONSUMERS)
                    reinterpret_cast<uint4 *>(s.vec)[v] = __ldcg(src + v);
                consumer_barrier();
            }
            cur_b = b;
        }
        const uint4 *vec0 = reinterpret_cast<const uint4 *>(s.vec);
        // After a give-up anywhere in the CTA the remaining work is skipped, but every barrier is
        // still visited in the same order by both groups, so that nobody is left waiting.
        bool ok = !*s.abort;
        for (int pg = 0; pg < n_pairs; pg += pl.R, ++pgc) {
            if (!ok) continue;
            if ((int)(pgc & 1) != group) continue;  // the other group's stage(s)
            const bool have = pg + my_pair < n_pairs;
            float acc[MMA_ACCS][4] = {};
            if (pl.n_chunks > 1) my_blocks<WPG>(pl.chunk_units, q, my_full, tail_lanes);
            for (int c = 0; c < pl.n_chunks; ++c, pos.advance(ns2)) {
                const int stage = group * ns2 + pos.slot;  // this group's half of the ring
                if (!wait_or_abort(&s.full[stage], pos.round & 1, s.abort, ws, DOWN ? 8 : 6)) {
                    ok = false;
                    break;
                }
                if (have) {
                    if (c == pl.n_chunks - 1 && c > 0)  // a long row's last chunk may be shorter
                        my_blocks<WPG>(pl.row_units - c * pl.chunk_units, q, my_full, tail_lanes);
                    const uint4 *p0 = reinterpret_cast<const uint4 *>(s.stages + (size_t)stage * slot_bytes +
                                                                      (size_t)(2 * my_pair) * chunk_bytes_max) +
                                      lane_unit;
                    const uint4 *pv = vec0 + c * pl.chunk_units + lane_unit;
                    pair_mma<DOWN, VREG, WPG>(acc, p0, p0 + pl.chunk_units, pv, pv + pl.row_units, xr, wr, my_full,
                                              tail_lanes, lane);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&s.empty[stage]);
            }
            if (ok && have) {
                float sum[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {  // a fixed order: results are reproducible
                    float lo = (acc[0][e] + acc[1][e]) + (acc[2][e] + acc[3][e]);
                    if (MMA_ACCS == 8) lo += (acc[4 % MMA_ACCS][e] + acc[5 % MMA_ACCS][e]) + (acc[6 % MMA_ACCS][e] + acc[7 % MMA_ACCS][e]);
                    sum[e] = lo;
                }
                const float dsum = diagonal_sum(sum, lane);
                float *slot = reinterpret_cast<float *>(&part[(pg + my_pair) * DEC_CONSUMER_WARPS + q]);
                if (lane == 0) slot[0] = dsum;  // first row of the pair
                if (lane == 4) slot[1] = dsum;  // second row
            }
        }
        group_barrier(group);  // this group's partial sums are in place
        if (*s.abort) ok = false;
        // every thread of the group looks after the rows of the pairs its group owned
        const int tig = tid - group * (DEC_GROUP_WARPS * 32);
        const int my_row = tig;  // rows of the item: r0 + my_row (at most DEC_MAX_ROWS of them)
        const int my_rows_pair = DOWN ? my_row >> 1 : my_row;
        if (ok && my_row < r1 - r0 && (int)((pgc0 + my_rows_pair / pl.R) & 1) == group) {
            const int pair = my_rows_pair;
            float a0 = 0.f, a1 = 0.f;
            for (int w = 0; w < wpg; ++w) {
                const float2 v = part[pair * DEC_CONSUMER_WARPS + w];
                a0 += v.x;
                a1 += v.y;
            }
            if (!DOWN) {
                const int j = r0 + my_row;
                if (p.seq[b].b_gate) a0 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[b].b_gate)[j]);
                if (p.seq[b].b_up) a1 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[b].b_up)[j]);
                // z leaves in bf16 (Z_LO: as two bf16 numbers, z_hi + z_lo), ready to be the down half's vector
                const float zv = sigma_rt(act, a0) * a1;
                const __nv_bfloat16 h = __float2bfloat16_rn(zv);
                zbits[(size_t)b * 2 * p.ldk + j] = h;
                if (Z_LO) zbits[(size_t)b * 2 * p.ldk + p.ldk + j] = __float2bfloat16_rn(zv - __bfloat162float(h));
            } else {
                const int c = r0 + my_row;
                float acc = (my_row & 1) ? a1 : a0;
                if (p.b_down) acc += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.b_down)[c]);
                static_cast<__nv_bfloat16 *>(p.y)[(size_t)b * p.d + c] = __float2bfloat16_rn(acc);
            }
        }
        if (!DOWN && sl == n_slices - 1)  // the last slice also clears the padding of z
            for (int j = p.k + tid; j < p.ldk; j += DEC_CONSUMERS) {
                zbits[(size_t)b * 2 * p.ldk + j] = __float2bfloat16_rn(0.f);
                if (Z_LO) zbits[(size_t)b * 2 * p.ldk + p.ldk + j] = __float2bfloat16_rn(0.f);
            }
    }
    return !*s.abort;
}

#ifndef GRIFFIN_DEC_MIN_CTAS
#define GRIFFIN_DEC_MIN_CTAS 1
#endif
__global__ void __launch_bounds__(DEC_THREADS, GRIFFIN_DEC_MIN_CTAS) decode_fused_kernel(const __grid_constant__ DecodeParams p,
                                                                   const __grid_constant__ FusedPlan fp, int act) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const MmaSmem s = carve_fused(smem_raw, fp);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < fp.n_stages; ++i) {
            mbar_init(&s.full[i], 1);
            mbar_init(&s.empty[i], DEC_GROUP_WARPS);  // the group that owns the stage hands it back
        }
        *s.abort = 0;
        mbar_fence_init();
    }
    __syncthreads();
    pdl_launch_dependents();

    if (warp == DEC_CONSUMER_WARPS) {
        // ---- producer warp: weights only, so it never waits for the previous grid, nor for
        //      the meeting point: the first stages of W_2_hat are on their way while the
        //      consumers are still waiting for the other CTAs' z
        RingPos pos[2] = {{0, 0, 0}, {0, 0, 0}};
        uint32_t pgc = 0;
        if (produce_half<false>(p, fp.gu, s, fp.n_stages, fp.slot_bytes, p.n_slices, pos, pgc, lane))
            produce_half<true>(p, fp.dn, s, fp.n_stages, fp.slot_bytes, p.n_slices_dn, pos, pgc, lane);
        const uint32_t issued[2] = {pos[0].uses, pos[1].uses};
        if (lane == 0) producer_drain_mma(s, fp.n_stages, issued);
        return;
    }

    // ---- consumers
    pdl_wait_prior_grids();  // x, the z scratch and the outputs belong to earlier work on the stream
    RingPos pos = {0, 0, 0};  // of this warp's group
    uint32_t pgc = 0;         // pair groups seen by everybody
    int item_parity = 0;
#define GRIFFIN_CONSUME(DOWN_, VREG_, WPG_, PLAN_, SLICES_) \
    consume_half<DOWN_, VREG_, WPG_>(p, PLAN_, s, fp.n_stages, fp.slot_bytes, SLICES_, pos, pgc, item_parity, act, tid, warp, lane)
    // warps per pair as a compile-time constant: block offsets become immediates.  A row of
    // W_g_hat or W_1_hat (d <= GRIFFIN_MAX_D elements) is always one chunk.
    switch (fp.gu.R) {
        case 4: GRIFFIN_CONSUME(false, true, 1, fp.gu, p.n_slices); break;
        case 2: GRIFFIN_CONSUME(false, true, 2, fp.gu, p.n_slices); break;
        default: GRIFFIN_CONSUME(false, true, 4, fp.gu, p.n_slices); break;
    }
    // each group reports on its own: 2 arrivals per CTA
    const int group = warp / DEC_GROUP_WARPS;
    group_barrier(group);  // this group's z entries are written (the thread that reports in makes them visible device-wide)
    if ((tid & (DEC_GROUP_WARPS * 32 - 1)) == 0)
        grid_meet(&static_cast<WsHeader *>(p.ws)->meet_warp, 2 * gridDim.x, s.abort, p.ws);
    group_barrier(group);  // the group has seen everybody: z is complete
    if (fp.dn.n_chunks == 1) {
        switch (fp.dn.R) {
            case 4: GRIFFIN_CONSUME(true, true, 1, fp.dn, p.n_slices_dn); break;
            case 2: GRIFFIN_CONSUME(true, true, 2, fp.dn, p.n_slices_dn); break;
            default: GRIFFIN_CONSUME(true, true, 4, fp.dn, p.n_slices_dn); break;
        }
    } else {  // chunks of 8 KB or more: at most two pairs per stage
        if (fp.dn.R == 2) GRIFFIN_CONSUME(true, false, 2, fp.dn, p.n_slices_dn);
        else GRIFFIN_CONSUME(true, false, 4, fp.dn, p.n_slices_dn);
    }
#undef GRIFFIN_CONSUME
}

griffin_status decode_bf16_mma(DecodeParams &p, int act, uint32_t flags, cudaStream_t stream) {
    const int sms = device_sm_count();
    if (sms <= 0) return GRIFFIN_ERR_CUDA;
    if (p.ws == nullptr) return GRIFFIN_ERR_WORKSPACE;  // the meeting point's counters live in the header
    const bool overlap = (flags & GRIFFIN_DECODE_OVERLAP_WEIGHT_PREFETCH) != 0;
    FusedPlan fp;
    fp.gu = make_plan(p.d, p.d * 2, MMA_STAGE_TARGET, MMA_BLOCKS_PER_WARP);
    fp.dn = make_plan(p.ldk, p.ldk * 4, GRIFFIN_DEC_DOWN_STAGE_KB * 1024, MMA_BLOCKS_PER_WARP_DOWN);
    fp.slot_bytes = max(fp.gu.stage_bytes, fp.dn.stage_bytes);
    fp.vec_bytes = fp.dn.n_chunks > 1 ? p.ldk * (Z_LO ? 4 : 2) : 16;  // only rows of several chunks stage z in shared memory
    int n = ((int)MMA_SMEM_TARGET - fp.vec_bytes - (int)mma_fixed_smem(8)) / fp.slot_bytes;
    fp.n_stages = (n < 2 ? 2 : (n > 8 ? 8 : n)) & ~1;  // two halves, one per consumer group
    p.n_slices = slices_for(p.k, sms);
    p.n_slices_dn = slices_for(p.d, sms);
    // every CTA of the grid must be able to run at the same time (they meet half-way): one per SM
    const int grid = sms;
    const size_t smem = (size_t)fp.n_stages * fp.slot_bytes + fp.vec_bytes + mma_fixed_smem(fp.n_stages);
    if (smem > 227 * 1024) return GRIFFIN_ERR_UNSUPPORTED;
    const void *fn = (const void *)decode_fused_kernel;
    if (ensure_dynamic_smem(fn, smem) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    void *args[] = {&p, &fp, &act};
    if (launch_maybe_overlapped(fn, dim3(grid), dim3(DEC_THREADS), smem, stream, overlap, args) != cudaSuccess)
        return GRIFFIN_ERR_CUDA;
    return GRIFFIN_OK;
}

}  // namespace griffin
