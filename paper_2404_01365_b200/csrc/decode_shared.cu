// Generation-phase pruned FF (Eqs. 4 and 5 of the GRIFFIN paper) for a batch that shares ONE expert set
// (the batch statistic of Eq. 7): bf16 storage, 2..8 vectors per pass, one kernel per pass.
//
//   first half   z_hat[n] = sigma(W_g_hat x[n] + b_g_hat) * (W_1_hat x[n] + b_1_hat)   for every vector n
//   meeting      every CTA has written its z entries; all CTAs wait for each other (bounded)
//   second half  y_hat[n] = W_2_hat z_hat[n] + b_2
//
// The weights are streamed once for all the vectors, so the call costs what a single vector costs: the
// bytes of the compact set.  Same skeleton as the single-vector kernel (decode_mma.cu): one persistent CTA
// per SM, a producer warp that fills a ring of shared-memory stages with 1-D bulk copies (TMA, no
// multicast) and runs ahead of the previous kernel on the stream and of the meeting point, two groups of
// four consumer warps that take alternate row groups, a wrap-around counter in the workspace header as the
// meeting point.  What differs is how a stage meets the vectors in mma.sync.m16n8k16:
//   * the A operand's rows are the (up to) 8 VECTORS (rows 8..15 are zero), the B operand's 8 columns are 8
//     staged WEIGHT ROWS, so every product of the upper half of the tile is used (the single-vector kernel
//     uses a diagonal only).  A stage is a "row group": 4 gate rows and the 4 up rows of the same neurons, or
//     8 rows of W_1_hat (a block without a gate), or 8 rows of W_2_hat; long rows are cut into chunks of at
//     most 4 KB, one chunk of all 8 rows per stage.  (Measured: a bulk copy costs the SM 55-65 ns whatever its
//     size, so 2 KB pieces cap the stream at 4.7-4.9 TB/s; with 16 weight rows on the A operand a stage of 4 KB
//     pieces would be 64 KB and the ring too shallow, hence the weights sit on the 8-wide operand.)
//   * lane (g, t) of a warp (g = lane / 4, t = lane % 4) reads one 16-byte unit of weight row g and of vector
//     g: unit 4 b + t of block b (a block is 64 bytes of every row).  The unit's first four elements feed one
//     MMA and the last four a second one; the MMA sums over K, so any assignment of elements to K positions
//     works as long as all rows and all vectors agree, and here lane t supplies the same unit of each.  Staged
//     rows and vectors lie at a pitch of 64 bytes modulo 128, so the two rows (or vectors) that a quarter warp
//     reads together fall into different banks.  C[v][r] = vector v . row r sits in lane (v, r / 2).
//   * the four warps of a group share a stage by blocks; their partial 8 x 8 tiles meet in shared memory
//     after the last chunk of the row group, in a fixed order: results are bitwise reproducible.
//   * the vectors stay in shared memory for a whole half (x, then z, which every CTA reads back from L2
//     after the meeting), brought in by bulk copies.  When 8 vectors and a ring of four stages do not fit
//     together, the chunks get shorter, and beyond that the batch is split into passes of fewer vectors.
#include "decode_mma.cuh"

namespace griffin {

constexpr int SH_ROWS = 8;     // weight rows per stage = N of the MMA
constexpr int SH_MAX_VEC = 8;  // vectors per pass (rows 0..7 of the MMA's M = 16)
constexpr int SH_PAD = 64;     // bytes that shift consecutive rows / vectors to other banks
constexpr int SH_BATCH = 4;    // blocks whose loads are issued before their MMAs
constexpr int SH_THREADS = DEC_CONSUMERS + 2 * 32;  // 8 consumer warps + one producer warp per consumer group
constexpr int SH_PART_FLOATS = SH_ROWS * SH_MAX_VEC;                          // one warp's partial tile
constexpr int SH_PART_BYTES = 2 * 2 * DEC_GROUP_WARPS * SH_PART_FLOATS * 4;  // [group][parity][warp][8 x 8]
constexpr int MODE_GATE_UP = 0, MODE_DOWN = 1, MODE_UP = 2;

struct SharedPlan {
    int n_vec;         // vectors of this pass
    int vec_pitch;     // bytes between vectors in shared memory
    int vec_bytes;
    int n_stages;      // even: one half of the ring per consumer group
    int row_pitch;     // bytes between staged rows
    int stage_bytes;   // SH_ROWS * row_pitch
    int cu[2];         // units (16 bytes) per chunk, per half; a multiple of 8
    int n_chunks[2];
    int row_units[2];  // units per weight row: d / 8, ldk / 8
    int n_slices[2];   // work items per half
};

struct ShSmem {
    uint8_t *stages;
    uint8_t *vec;
    uint64_t *full, *empty;
    uint64_t *vfull;  // [2]: the vectors' first chunk has landed / the rest has
    float *part;
    volatile int *abort;
};
__device__ __forceinline__ ShSmem carve_shared(uint8_t *smem, const SharedPlan &pl) {
    ShSmem s;
    s.stages = smem;
    s.vec = smem + (size_t)pl.n_stages * pl.stage_bytes;
    s.part = reinterpret_cast<float *>(s.vec + pl.vec_bytes);
    s.full = reinterpret_cast<uint64_t *>(s.part + SH_PART_BYTES / 4);
    s.empty = s.full + pl.n_stages;
    s.vfull = s.empty + pl.n_stages;
    s.abort = reinterpret_cast<volatile int *>(s.vfull + 2);
    return s;
}
static inline size_t shared_smem_bytes(const SharedPlan &pl) {
    return (size_t)pl.n_stages * pl.stage_bytes + pl.vec_bytes + SH_PART_BYTES + (2 * pl.n_stages + 2) * sizeof(uint64_t) + 16;
}

// Producer side of one half.  There are two producer warps, one per consumer group: consecutive row groups
// belong to the two consumer groups in turn, each group has its own half of the ring, and producer warp `grp`
// feeds that half with the row groups of its group.  Lane l < 8 copies row l of the row group (weights only).
// (Measured: a bulk copy costs the issuing warp 55-65 ns whatever its size, so one warp issuing the 16 copies
// of every stage would pace the kernel; two warps issue side by side.)
template <int MODE>
__device__ __forceinline__ bool sh_produce_half(const DecodeParams &p, const SharedPlan &plan, const ShSmem &s, int grp,
                                                RingPos &pos, uint32_t &rgc, int lane) {
    constexpr bool DOWN = MODE == MODE_DOWN;
    constexpr int H = DOWN ? 1 : 0;
    constexpr int RG = MODE == MODE_GATE_UP ? SH_ROWS / 2 : SH_ROWS;  // neurons / output rows per row group
    const SharedPlan pl = plan;  // in registers: the asm statements in the loops clobber memory
    void *const ws = p.ws;
    const int cu = pl.cu[H], n_chunks = pl.n_chunks[H], row_units = pl.row_units[H], n_slices = pl.n_slices[H];
    const int total_rows = DOWN ? p.d : p.k;
    const int ns2 = pl.n_stages >> 1;
    const size_t row_bytes = (size_t)row_units * 16;
    const uint8_t *const wg = static_cast<const uint8_t *>(p.seq[0].w_gate);
    const uint8_t *const wu = static_cast<const uint8_t *>(p.seq[0].w_up);
    const uint8_t *const wd = static_cast<const uint8_t *>(p.seq[0].w_down);
    for (int item = blockIdx.x; item < n_slices; item += gridDim.x) {
        const int r0 = (int)((long long)item * total_rows / n_slices);
        const int r1 = (int)((long long)(item + 1) * total_rows / n_slices);
        for (int g0 = r0; g0 < r1; g0 += RG, ++rgc) {
            if ((int)(rgc & 1) != grp) continue;  // the other producer's row group
            const int nrows = min(RG, r1 - g0);
            const uint8_t *src = nullptr;
            if (MODE == MODE_GATE_UP) {
                if (lane < SH_ROWS && (lane & 3) < nrows) src = (lane < 4 ? wg : wu) + (size_t)(g0 + (lane & 3)) * row_bytes;
            } else if (lane < nrows) {
                src = (DOWN ? wd : wu) + (size_t)(g0 + lane) * row_bytes;
            }
            const int rows_in_stage = MODE == MODE_GATE_UP ? 2 * nrows : nrows;
            for (int c = 0; c < n_chunks; ++c, pos.advance(ns2)) {
                const int units = min(cu, row_units - c * cu);
                const int stage = grp * ns2 + pos.slot;
                const uint32_t use = pos.round;
                int go = 1;
                if (lane == 0) {
                    if (use > 0 && !wait_or_abort(&s.empty[stage], (use - 1) & 1, s.abort, ws, DOWN ? 47 : 45)) go = 0;
                    if (go) mbar_arrive_expect_tx(&s.full[stage], (uint32_t)(rows_in_stage * units * 16));
                }
                go = __shfl_sync(0xffffffffu, go, 0);
                if (!go) return false;
                if (src != nullptr)
                    bulk_g2s(s.stages + (size_t)stage * pl.stage_bytes + (size_t)lane * pl.row_pitch,
                             src + (size_t)c * cu * 16, (uint32_t)units * 16, &s.full[stage]);
            }
        }
    }
    return true;
}

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

// One thread: starts the bulk copies of the pass's vectors (x, or z) from global memory into shared memory.
// The first chunk of every vector completes vfull[0], the rest of every vector vfull[1]: the consumers need
// chunk 0 first and can start on it while the rest is still on its way.  `units` 16-byte units per vector.
__device__ __forceinline__ void sh_issue_vectors(const ShSmem &s, const SharedPlan &pl, const void *src, size_t src_stride_bytes,
                                                 int units, int cu) {
    // what comes before on this thread -- the other CTAs' z entries acquired at the meeting point, this CTA's
    // own reads of the vectors that are about to be overwritten -- is ordered before the copies, which act
    // through the asynchronous proxy
    fence_proxy_async();
    const uint32_t head = (uint32_t)min(cu, units) * 16, tail = (uint32_t)units * 16 - head;
    mbar_arrive_expect_tx(&s.vfull[0], (uint32_t)pl.n_vec * head);
    for (int n = 0; n < pl.n_vec; ++n)
        bulk_g2s(s.vec + (size_t)n * pl.vec_pitch, static_cast<const uint8_t *>(src) + (size_t)n * src_stride_bytes, head, &s.vfull[0]);
    if (tail > 0) {
        mbar_arrive_expect_tx(&s.vfull[1], (uint32_t)pl.n_vec * tail);
        for (int n = 0; n < pl.n_vec; ++n)
            bulk_g2s(s.vec + (size_t)n * pl.vec_pitch + head, static_cast<const uint8_t *>(src) + (size_t)n * src_stride_bytes + head,
                     tail, &s.vfull[1]);
    } else {
        mbar_arrive(&s.vfull[1]);  // (the phase ends all the same)
    }
}

// One block: the lane's unit of its vector (A operand, rows 8..15 zero) against its unit of its weight row (B operand).
__device__ __forceinline__ void sh_mma_block(float (&acc)[4][4], int i, const uint4 &v, const uint4 &w) {
    mma_bf16(acc[(2 * i) & 3], v.x, 0u, v.y, 0u, w.x, w.y);
    mma_bf16(acc[(2 * i + 1) & 3], v.z, 0u, v.w, 0u, w.z, w.w);
}

// Consumer side of one half (all 8 consumer warps).  Returns false after a give-up.
template <int MODE>
__device__ __forceinline__ bool sh_consume_half(const DecodeParams &p, const SharedPlan &plan, const ShSmem &s, RingPos &pos,
                                                uint32_t &rgc, int &parity, int act, int tid, int warp, int lane) {
    constexpr bool DOWN = MODE == MODE_DOWN;
    constexpr int H = DOWN ? 1 : 0;
    constexpr int RG = MODE == MODE_GATE_UP ? SH_ROWS / 2 : SH_ROWS;
    const SharedPlan pl = plan;
    void *const ws = p.ws;
    const int cu = pl.cu[H], n_chunks = pl.n_chunks[H], row_units = pl.row_units[H], n_slices = pl.n_slices[H];
    const int total_rows = DOWN ? p.d : p.k;
    const int ns2 = pl.n_stages >> 1;
    const int group = warp / DEC_GROUP_WARPS, q = warp - group * DEC_GROUP_WARPS;
    const int g = lane >> 2, t = lane & 3;
    const int tig = tid - group * (DEC_GROUP_WARPS * 32);
    const bool has_vec = g < pl.n_vec;
    // this lane's unit of block 0: of its vector, and (added per stage) of row g
    const uint4 *const vec_lane = reinterpret_cast<const uint4 *>(s.vec + (size_t)(has_vec ? g : 0) * pl.vec_pitch) + t;
    const int row_lane_off = g * pl.row_pitch + t * 16;
    float *const part_grp = s.part + group * (2 * DEC_GROUP_WARPS * SH_PART_FLOATS);
    __nv_bfloat16 *zbits = reinterpret_cast<__nv_bfloat16 *>(p.z);  // per vector: z [ldk] in bf16, 2 ldk elements apart
    const uint4 zero = make_uint4(0, 0, 0, 0);
    bool ok = !*s.abort;
    for (int item = blockIdx.x; item < n_slices; item += gridDim.x) {
        const int r0 = (int)((long long)item * total_rows / n_slices);
        const int r1 = (int)((long long)(item + 1) * total_rows / n_slices);
        for (int g0 = r0; g0 < r1; g0 += RG, ++rgc) {
            if ((int)(rgc & 1) != group) continue;  // the other group's row group
            const int nrows = min(RG, r1 - g0);
            float acc[4][4] = {};
            // After a give-up anywhere in the CTA the work is skipped, but the group still meets at every
            // barrier below, so that nobody is left waiting.
            if (ok) {
                for (int c = 0; c < n_chunks; ++c, pos.advance(ns2)) {
                    const int stage = group * ns2 + pos.slot;
                    if (!wait_or_abort(&s.full[stage], pos.round & 1, s.abort, ws, DOWN ? 48 : 46)) {
                        ok = false;
                        break;
                    }
                    if (c < 2 && !wait_or_abort(&s.vfull[c], H, s.abort, ws, DOWN ? 50 : 49)) {  // this half's vectors
                        ok = false;
                        break;
                    }
                    const int units = min(cu, row_units - c * cu);
                    const int whole = units >> 2;          // blocks whose four units all exist
                    const int nblk = (units + 3) >> 2;     // ... and counting the cut one
                    const uint4 *const w_lane =
                        reinterpret_cast<const uint4 *>(s.stages + (size_t)stage * pl.stage_bytes + row_lane_off);
                    const uint4 *const v_lane = vec_lane + c * cu;
                    // this warp's blocks: q, q + 4, q + 8, ...; a batch is four of them
#pragma unroll 1
                    for (int b0 = q; b0 < nblk; b0 += DEC_GROUP_WARPS * SH_BATCH) {
                        uint4 wr[SH_BATCH], vr[SH_BATCH];
                        if (b0 + DEC_GROUP_WARPS * (SH_BATCH - 1) < whole) {  // warp-uniform: four whole blocks
#pragma unroll
                            for (int i = 0; i < SH_BATCH; ++i) {
                                const int u = 4 * (b0 + DEC_GROUP_WARPS * i);
                                wr[i] = w_lane[u];
                                vr[i] = has_vec ? v_lane[u] : zero;
                            }
#pragma unroll
                            for (int i = 0; i < SH_BATCH; ++i) sh_mma_block(acc, i, vr[i], wr[i]);
                        } else {  // the chunk ends inside this batch: units past the end count as zeros
#pragma unroll
                            for (int i = 0; i < SH_BATCH; ++i) {
                                const int blk = b0 + DEC_GROUP_WARPS * i;
                                const int u = 4 * blk;
                                const bool in = u + t < units;  // (stale bytes behind a row's end could be NaN)
                                wr[i] = in ? w_lane[u] : zero;
                                vr[i] = in && has_vec ? v_lane[u] : zero;
                            }
#pragma unroll
                            for (int i = 0; i < SH_BATCH; ++i)
                                if (b0 + DEC_GROUP_WARPS * i < nblk) sh_mma_block(acc, i, vr[i], wr[i]);  // warp-uniform
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&s.empty[stage]);
                }
            }
            // this warp's partial tile: lane (g, t) holds C[vector g][rows 2t, 2t+1]
            float *const part = part_grp + parity * (DEC_GROUP_WARPS * SH_PART_FLOATS);
            {
                float2 lo;  // (a fixed order: results are reproducible)
                lo.x = (acc[0][0] + acc[1][0]) + (acc[2][0] + acc[3][0]);
                lo.y = (acc[0][1] + acc[1][1]) + (acc[2][1] + acc[3][1]);
                *reinterpret_cast<float2 *>(part + q * SH_PART_FLOATS + g * SH_ROWS + 2 * t) = lo;
            }
            group_barrier(group);
            if (*s.abort) ok = false;
            // thread (v, r) of the group's first 64 finishes row r of the row group for vector v
            const int v = tig >> 3, r = tig & 7;
            if (ok && tig < SH_MAX_VEC * SH_ROWS && v < pl.n_vec && r < nrows) {
                float a0 = 0.f;
#pragma unroll
                for (int w = 0; w < DEC_GROUP_WARPS; ++w) a0 += part[w * SH_PART_FLOATS + v * SH_ROWS + r];
                const int j = g0 + r;
                if (MODE == MODE_GATE_UP) {  // (r < nrows <= 4: the gate rows; the up row of the same neuron is row r + 4)
                    float a1 = 0.f;
#pragma unroll
                    for (int w = 0; w < DEC_GROUP_WARPS; ++w) a1 += part[w * SH_PART_FLOATS + v * SH_ROWS + r + 4];
                    if (p.seq[0].b_gate) a0 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[0].b_gate)[j]);
                    if (p.seq[0].b_up) a1 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[0].b_up)[j]);
                    zbits[(size_t)v * 2 * p.ldk + j] = __float2bfloat16_rn(sigma_rt(act, a0) * a1);
                } else if (MODE == MODE_UP) {
                    if (p.seq[0].b_up) a0 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[0].b_up)[j]);
                    zbits[(size_t)v * 2 * p.ldk + j] = __float2bfloat16_rn(sigma_rt(act, a0));
                } else {
                    if (p.b_down) a0 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.b_down)[j]);
                    static_cast<__nv_bfloat16 *>(p.y)[(size_t)v * p.d + j] = __float2bfloat16_rn(a0);
                }
            }
            parity ^= 1;
        }
        if (!DOWN && item == n_slices - 1 && group == 0)  // the last slice also clears the padding of z
            for (int e = tig; e < pl.n_vec * (p.ldk - p.k); e += DEC_GROUP_WARPS * 32) {
                const int n = e / (p.ldk - p.k), j = p.k + e - n * (p.ldk - p.k);
                zbits[(size_t)n * 2 * p.ldk + j] = __float2bfloat16_rn(0.f);
            }
    }
    return ok && !*s.abort;
}

template <bool GATED>
__global__ void __launch_bounds__(SH_THREADS, 1) decode_shared_kernel(const __grid_constant__ DecodeParams p,
                                                                      const __grid_constant__ SharedPlan pl, int act) {
    constexpr int FIRST = GATED ? MODE_GATE_UP : MODE_UP;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const ShSmem s = carve_shared(smem_raw, pl);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < pl.n_stages; ++i) {
            mbar_init(&s.full[i], 1);
            mbar_init(&s.empty[i], DEC_GROUP_WARPS);  // the group that owns the stage hands it back
        }
        mbar_init(&s.vfull[0], 1);
        mbar_init(&s.vfull[1], 1);
        *s.abort = 0;
        mbar_fence_init();
    }
    __syncthreads();
    pdl_launch_dependents();

    if (warp >= DEC_CONSUMER_WARPS) {
        // ---- producer warps: weights only, so they wait neither for the previous grid nor for the meeting point
        const int grp = warp - DEC_CONSUMER_WARPS;
        const int ns2 = pl.n_stages >> 1;
        RingPos pos = {0, 0, 0};
        uint32_t rgc = 0;
        if (sh_produce_half<FIRST>(p, pl, s, grp, pos, rgc, lane)) sh_produce_half<MODE_DOWN>(p, pl, s, grp, pos, rgc, lane);
        if (lane == 0) {
            // stay until every copy that was started has landed (only matters after a give-up: normally the
            // consumers have waited for every stage), so that shared memory is never released under a copy
            const uint32_t first = pos.uses > (uint32_t)ns2 ? pos.uses - ns2 : 0;
            for (uint32_t it = first; it < pos.uses; ++it) {
                const int stage = grp * ns2 + (int)(it % ns2);
                const long long t0 = clock64();
                while (!mbar_try_wait(&s.full[stage], (it / ns2) & 1))
                    if (clock64() - t0 > WAIT_LIMIT_CYCLES) break;
            }
        }
        return;
    }

    // ---- consumers
    pdl_wait_prior_grids();  // x, the z scratch and the outputs belong to earlier work on the stream
    if (tid == 0) sh_issue_vectors(s, pl, p.x, (size_t)p.d * 2, pl.row_units[0], pl.cu[0]);
    RingPos pos = {0, 0, 0};  // of this warp's group
    uint32_t rgc = 0;         // row groups seen by everybody
    int parity = 0;           // of this group's partial-tile buffers
    sh_consume_half<FIRST>(p, pl, s, pos, rgc, parity, act, tid, warp, lane);
    // each group reports on its own: 2 arrivals per CTA (always, also after a give-up: the counter is never reset)
    const int group = warp / DEC_GROUP_WARPS;
    group_barrier(group);  // this group's z entries are written (the thread that reports in makes them visible device-wide)
    if ((tid & (DEC_GROUP_WARPS * 32 - 1)) == 0)
        grid_meet(&static_cast<WsHeader *>(p.ws)->meet_warp, 2 * gridDim.x, s.abort, p.ws);
    consumer_barrier();  // both groups have seen everybody (z is complete) and are done with x
    const bool second = !*s.abort;
    if (tid == 0 && second) sh_issue_vectors(s, pl, p.z, (size_t)p.ldk * 4, pl.row_units[1], pl.cu[1]);  // (2 ldk bf16 entries per vector)
    sh_consume_half<MODE_DOWN>(p, pl, s, pos, rgc, parity, act, tid, warp, lane);
    if (tid == 0) {
        // stay until the copies of the vectors have landed (only matters after a give-up: normally every
        // consumer has waited for them), so that shared memory is never released under a copy in flight
        const uint32_t last = second ? 1 : 0;
        for (int i = 0; i < 2; ++i) {
            const long long t0 = clock64();
            while (!mbar_try_wait(&s.vfull[i], last))
                if (clock64() - t0 > WAIT_LIMIT_CYCLES) break;
        }
    }
}

// All sequences of the call name the same compact buffers.
bool decode_shared_set(const DecodeParams &p) {
    if (p.B < 2) return false;
    for (int b = 1; b < p.B; ++b)
        if (p.seq[b].w_gate != p.seq[0].w_gate || p.seq[b].w_up != p.seq[0].w_up || p.seq[b].w_down != p.seq[0].w_down ||
            p.seq[b].b_gate != p.seq[0].b_gate || p.seq[b].b_up != p.seq[0].b_up)
            return false;
    return true;
}

// Chunk length and ring depth for n_vec vectors; false if even the smallest ring does not fit beside them.
// Measured on B200 (Llama-2-7B shape): what counts is the bytes the ring keeps in flight (six stages of 32 KB:
// 25.8 us per call, four: 28.4 us) and the size of a copy (4 KB pieces: 25.8 us, 2 KB: 29.5 us; a bulk copy
// costs the SM 55-65 ns whatever its size); a prefetch of later rows into L2 made every case slower.
static bool shared_plan(SharedPlan &pl, int d, int ldk, int k, int n_vec, int sms) {
    pl.n_vec = n_vec;
    pl.vec_pitch = ((max(d, ldk) * 2 + 127) & ~127) + SH_PAD;
    pl.vec_bytes = n_vec * pl.vec_pitch;
    pl.row_units[0] = d / 8;
    pl.row_units[1] = ldk / 8;
    pl.n_slices[0] = slices_for(k, sms);
    pl.n_slices[1] = slices_for(d, sms);
    // {longest chunk in units, stages}, best first: deep rings of long pieces, then shallower, then shorter
    static const int cand[][2] = {{320, 6}, {256, 6}, {320, 4}, {256, 4}, {192, 6}, {192, 4}, {128, 6}, {128, 4}, {64, 4}, {32, 4}};
    for (const auto &c : cand) {
        // (chunks shorter than 2 KB are only taken for a single vector: with more, two passes of half as many
        // vectors at full speed beat one pass of short copies)
        if (c[0] < 128 && n_vec > 1) continue;
        int longest = 0;
        for (int h = 0; h < 2; ++h) {  // a row is cut into equal chunks, a multiple of 128 bytes each
            pl.n_chunks[h] = (pl.row_units[h] + c[0] - 1) / c[0];
            pl.cu[h] = ((pl.row_units[h] + pl.n_chunks[h] - 1) / pl.n_chunks[h] + 7) & ~7;
            if (pl.cu[h] > c[0]) pl.cu[h] = c[0];  // (c[0] is itself a multiple of 8)
            longest = max(longest, pl.cu[h]);
        }
        pl.row_pitch = longest * 16 + SH_PAD;
        pl.stage_bytes = SH_ROWS * pl.row_pitch;
        pl.n_stages = c[1];
        if (shared_smem_bytes(pl) <= 227 * 1024) return true;
    }
    return false;
}

griffin_status decode_bf16_shared(DecodeParams &p, int act, bool gated, uint32_t flags, cudaStream_t stream) {
    const int sms = device_sm_count();
    if (sms <= 0) return GRIFFIN_ERR_CUDA;
    if (p.ws == nullptr) return GRIFFIN_ERR_WORKSPACE;  // the meeting point's counters live in the header
    SharedPlan pl;
    int n_vec = p.B < SH_MAX_VEC ? p.B : SH_MAX_VEC;
    while (!shared_plan(pl, p.d, p.ldk, p.k, n_vec, sms)) {
        if (n_vec == 1) return GRIFFIN_ERR_UNSUPPORTED;
        n_vec = (n_vec + 1) / 2;  // fewer vectors per pass: the weights are streamed once per pass
    }
    const void *fn = gated ? (const void *)decode_shared_kernel<true> : (const void *)decode_shared_kernel<false>;
    bool overlap = (flags & GRIFFIN_DECODE_OVERLAP_WEIGHT_PREFETCH) != 0;
    for (int s0 = 0; s0 < p.B; s0 += n_vec) {
        DecodeParams q = p;
        q.B = p.B - s0 < n_vec ? p.B - s0 : n_vec;
        q.x = static_cast<const __nv_bfloat16 *>(p.x) + (size_t)s0 * p.d;
        q.y = static_cast<__nv_bfloat16 *>(p.y) + (size_t)s0 * p.d;
        q.z = p.z + (size_t)s0 * p.ldk;  // (z of a sequence: 2 ldk bf16 entries = ldk floats)
        SharedPlan ql = pl;
        ql.n_vec = q.B;
        const size_t smem = shared_smem_bytes(pl);
        if (ensure_dynamic_smem(fn, smem) != cudaSuccess) return GRIFFIN_ERR_CUDA;
        if (!grid_can_meet(fn, SH_THREADS, smem, sms)) return GRIFFIN_ERR_UNSUPPORTED;
        void *args[] = {&q, &ql, &act};
        // every CTA of the grid must be able to run at the same time (they meet half-way): one per SM
        if (launch_maybe_overlapped(fn, dim3(sms), dim3(SH_THREADS), smem, stream, overlap, args) != cudaSuccess)
            return GRIFFIN_ERR_CUDA;
        overlap = true;  // a later pass only follows a pass of this call, which writes no weights
    }
    return GRIFFIN_OK;
}

}  // namespace griffin
