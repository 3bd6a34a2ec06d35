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
#include "decode_mma.cuh"

namespace griffin {

// The two halves of a decode call share one kernel, one ring and one stage counter:
//   DOWN = false: gate_up, z[b, j] = sigma(gate_j . x + b_gate_j) * (up_j . x + b_up_j);
//                 item = (sequence, slice of neurons), pair = neuron.
//   DOWN = true : down, y[b, c] = w_down_c[c, :] . z[b] + b_down[c];
//                 item = (sequence, chunk of output rows), pair = two consecutive rows.
// A block without a gate (Eq. 2) has a first half of its own, z[b, j] = sigma(up_j . x + b_up_j):
// item = (sequence, slice of neurons), pair = two consecutive rows of W_1_hat, as in the down half.
// The three are the MODEs below.
constexpr int MODE_GATE_UP = 0, MODE_DOWN = 1, MODE_UP = 2;
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
template <int MODE>
__device__ __forceinline__ bool produce_half(const DecodeParams &p, const MmaPlan &plan, const MmaSmem &s, int n_stages,
                                             int slot_bytes, int n_slices, RingPos (&pos)[2], uint32_t &pgc, int lane) {
    constexpr bool DOWN = MODE == MODE_DOWN;
    constexpr bool CONSEC = MODE != MODE_GATE_UP;  // a pair is two consecutive rows of one matrix
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
        const int n_pairs = CONSEC ? (r1 - r0 + 1) / 2 : r1 - r0;
        const uint8_t *mat = static_cast<const uint8_t *>(
            DOWN ? p.seq[b].w_down : ((MODE == MODE_UP || my_row) ? p.seq[b].w_up : p.seq[b].w_gate));
        for (int pg = 0; pg < n_pairs; pg += pl.R, ++pgc) {
            // consumer group (pgc & 1) owns this pair group; each group has its own half of the
            // ring and its own count of stage uses, so that every barrier sees one strictly
            // sequential user (a group skipping over the other's stages would otherwise wait on
            // a parity that an older phase already satisfies)
            const int grp = pgc & 1;
            const int pair = pg + my_pair;
            const int grow = CONSEC ? r0 + 2 * pair + my_row : r0 + pair;  // row in the matrix
            const bool mine = lane < 2 * pl.R && pair < n_pairs && grow < r1;
            // rows copied in this stage (the same for every chunk of the group)
            const int rows_in_stage = CONSEC ? min(2 * pl.R, r1 - r0 - 2 * pg) : 2 * min(pl.R, n_pairs - pg);
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

// Consumer side of one half (all 8 consumer warps).  Returns false after a give-up.
// VREG: a row is one chunk, so every stage of an item meets the same units of the vector and
// each lane keeps its units of it in registers (read straight from global memory, once per
// item); otherwise (rows longer than MMA_CHUNK_UNITS_MAX units, down only) the vector is
// staged in shared memory and read from there block by block.
template <int MODE, bool VREG, int WPG>
__device__ __forceinline__ bool consume_half(const DecodeParams &p, const MmaPlan &plan, const MmaSmem &s, int n_stages,
                                             int slot_bytes, int n_slices, RingPos &pos, uint32_t &pgc,
                                             int &item_parity, int act, int tid, int warp, int lane) {
    constexpr bool DOWN = MODE == MODE_DOWN;
    constexpr bool CONSEC = MODE != MODE_GATE_UP;  // a pair is two consecutive rows of one matrix
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
        const int n_pairs = CONSEC ? (r1 - r0 + 1) / 2 : r1 - r0;
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
        const int my_rows_pair = CONSEC ? my_row >> 1 : my_row;
        if (ok && my_row < r1 - r0 && (int)((pgc0 + my_rows_pair / pl.R) & 1) == group) {
            const int pair = my_rows_pair;
            float a0 = 0.f, a1 = 0.f;
            for (int w = 0; w < wpg; ++w) {
                const float2 v = part[pair * DEC_CONSUMER_WARPS + w];
                a0 += v.x;
                a1 += v.y;
            }
            if (MODE == MODE_UP) {
                const int j = r0 + my_row;
                float u = (my_row & 1) ? a1 : a0;
                if (p.seq[b].b_up) u += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[b].b_up)[j]);
                const float zv = sigma_rt(act, u);
                const __nv_bfloat16 h = __float2bfloat16_rn(zv);
                zbits[(size_t)b * 2 * p.ldk + j] = h;
                if (Z_LO) zbits[(size_t)b * 2 * p.ldk + p.ldk + j] = __float2bfloat16_rn(zv - __bfloat162float(h));
            } else if (!DOWN) {
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
template <bool GATED>
__global__ void __launch_bounds__(DEC_THREADS, GRIFFIN_DEC_MIN_CTAS) decode_fused_kernel(const __grid_constant__ DecodeParams p,
                                                                   const __grid_constant__ FusedPlan fp, int act) {
    constexpr int FIRST = GATED ? MODE_GATE_UP : MODE_UP;
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
        if (produce_half<FIRST>(p, fp.gu, s, fp.n_stages, fp.slot_bytes, p.n_slices, pos, pgc, lane))
            produce_half<MODE_DOWN>(p, fp.dn, s, fp.n_stages, fp.slot_bytes, p.n_slices_dn, pos, pgc, lane);
        const uint32_t issued[2] = {pos[0].uses, pos[1].uses};
        if (lane == 0) producer_drain_mma(s, fp.n_stages, issued);
        return;
    }

    // ---- consumers
    pdl_wait_prior_grids();  // x, the z scratch and the outputs belong to earlier work on the stream
    RingPos pos = {0, 0, 0};  // of this warp's group
    uint32_t pgc = 0;         // pair groups seen by everybody
    int item_parity = 0;
#define GRIFFIN_CONSUME(MODE_, VREG_, WPG_, PLAN_, SLICES_) \
    consume_half<MODE_, VREG_, WPG_>(p, PLAN_, s, fp.n_stages, fp.slot_bytes, SLICES_, pos, pgc, item_parity, act, tid, warp, lane)
    // warps per pair as a compile-time constant: block offsets become immediates.  A row of
    // W_g_hat or W_1_hat (d <= GRIFFIN_MAX_D elements) is always one chunk.
    switch (fp.gu.R) {
        case 4: GRIFFIN_CONSUME(FIRST, true, 1, fp.gu, p.n_slices); break;
        case 2: GRIFFIN_CONSUME(FIRST, true, 2, fp.gu, p.n_slices); break;
        default: GRIFFIN_CONSUME(FIRST, true, 4, fp.gu, p.n_slices); break;
    }
    // each group reports on its own: 2 arrivals per CTA
    const int group = warp / DEC_GROUP_WARPS;
    group_barrier(group);  // this group's z entries are written (the thread that reports in makes them visible device-wide)
    if ((tid & (DEC_GROUP_WARPS * 32 - 1)) == 0)
        grid_meet(&static_cast<WsHeader *>(p.ws)->meet_warp, 2 * gridDim.x, s.abort, p.ws);
    group_barrier(group);  // the group has seen everybody: z is complete
    if (fp.dn.n_chunks == 1) {
        switch (fp.dn.R) {
            case 4: GRIFFIN_CONSUME(MODE_DOWN, true, 1, fp.dn, p.n_slices_dn); break;
            case 2: GRIFFIN_CONSUME(MODE_DOWN, true, 2, fp.dn, p.n_slices_dn); break;
            default: GRIFFIN_CONSUME(MODE_DOWN, true, 4, fp.dn, p.n_slices_dn); break;
        }
    } else {  // chunks of 8 KB or more: at most two pairs per stage
        if (fp.dn.R == 2) GRIFFIN_CONSUME(MODE_DOWN, false, 2, fp.dn, p.n_slices_dn);
        else GRIFFIN_CONSUME(MODE_DOWN, false, 4, fp.dn, p.n_slices_dn);
    }
#undef GRIFFIN_CONSUME
}

griffin_status decode_bf16_mma(DecodeParams &p, int act, bool gated, uint32_t flags, cudaStream_t stream) {
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
    const void *fn = gated ? (const void *)decode_fused_kernel<true> : (const void *)decode_fused_kernel<false>;
    if (ensure_dynamic_smem(fn, smem) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    if (!grid_can_meet(fn, DEC_THREADS, smem, grid)) return GRIFFIN_ERR_UNSUPPORTED;
    void *args[] = {&p, &fp, &act};
    if (launch_maybe_overlapped(fn, dim3(grid), dim3(DEC_THREADS), smem, stream, overlap, args) != cudaSuccess)
        return GRIFFIN_ERR_CUDA;
    return GRIFFIN_OK;
}

}  // namespace griffin
