// Generation-phase pruned FF (Eqs. 4 and 5 of the GRIFFIN paper) straight from the FULL weights:
// the expert rows are read in place through the index list E, so no compact copy is ever made.
// bf16 storage, neuron-major weights: W_g, W_1 and the TRANSPOSE of W_2, each [d_ff, d].
//
// With W_2 transposed, neuron j owns one contiguous row in each of the three matrices and
//   y_hat = sum over j in E of z_j * W_2^T[j, :],   z_j = sigma(W_g[j, :] . x + b_g[j]) * (W_1[j, :] . x + b_1[j]).
// A CTA therefore needs nothing from the other CTAs until the very end: it takes a slice of E,
// forms its z entries, adds its multiples of the W_2^T rows into a private y, and only the
// partial y vectors (one per CTA and sequence, fp32) meet, through the workspace.
//
// One persistent CTA per SM, built like the compact-set kernel: a producer warp streams rows
// into a ring of shared-memory stages with 1-D bulk copies (TMA, no multicast), one copy per
// row, the source row taken from E; two groups of four consumer warps take alternate stages.
// A stage holds 2R rows in both halves of a work item (a slice of at most DEC_MAX_ROWS experts
// of one sequence):
//   first half   R pairs (gate row, up row); each pair meets x in the warp-level MMA exactly
//                as in the compact-set kernel ("virtual rows"); z of the slice goes to shared
//                memory in fp32;
//   second half  2R rows of W_2^T; consumer thread t of a group owns columns 8u..8u+7 for
//                u = t, t + 128, ...: no reduction across lanes is needed, so plain FMAs on
//                the unpacked bf16 pairs are far below the issue limit.
// After every item the two groups' shares of y are added through shared memory and join the
// CTA's partial y of that sequence in the workspace.  After its last item a CTA reports in; the
// last few to do so wait (bounded) for the rest and sum the columns over all CTAs' partials in
// a fixed order, add b_2 and write bf16, while the others have already left their SMs to the
// next kernel on the stream.  Results are bitwise reproducible.
#include "decode_mma.cuh"

namespace griffin {

struct IndexedParams {
    const void *w_gate, *w_up, *w_down_t;  // [d_ff, d] each
    const void *b_gate, *b_up, *b_down;    // [d_ff], [d_ff], [d] or null
    const int32_t *idx;                    // [B, k]
    const void *x;                         // [B, d]
    void *y;                               // [B, d]
    float *ypart;                          // [B, grid, d] fp32 partial sums
    void *ws;
    int d, d_ff, k, B;
    int n_slices;   // work items per sequence (a multiple of the grid)
    int n_stages;   // ring slots (even: one half per consumer group)
    int red_vec;    // columns per lane in the final reduction: 1 or 4
    int n_red;      // CTAs that share the final reduction (the last ones to finish their items)
};

struct IdxSmem {
    uint8_t *stages;
    float *ysm;   // [d] exchange of the second group's partial y
    float *zs;    // [DEC_MAX_ROWS] z of the current item
    float *red;   // [DEC_CONSUMER_WARPS][128] final reduction
    uint64_t *full, *empty;
    float2 *part;  // [2 parities][DEC_MAX_ROWS pairs][8 warps]
    volatile int *abort;
};
static inline size_t idx_fixed_smem(int d, int n_stages) {
    return (size_t)d * 4 + DEC_MAX_ROWS * 4 + DEC_CONSUMER_WARPS * 128 * 4 + mma_fixed_smem(n_stages);
}
__device__ __forceinline__ IdxSmem carve_idx(uint8_t *smem, int n_stages, int stage_bytes, int d) {
    IdxSmem s;
    s.stages = smem;
    s.ysm = reinterpret_cast<float *>(smem + (size_t)n_stages * stage_bytes);
    s.zs = s.ysm + d;
    s.red = s.zs + DEC_MAX_ROWS;
    s.full = reinterpret_cast<uint64_t *>(s.red + DEC_CONSUMER_WARPS * 128);
    s.empty = s.full + n_stages;
    s.part = reinterpret_cast<float2 *>(s.empty + n_stages);
    s.abort = reinterpret_cast<volatile int *>(s.part + 2 * DEC_MAX_ROWS * DEC_CONSUMER_WARPS);
    return s;
}

// Expert index of row `row` (0..63) of the item, from the two registers every lane holds.
__device__ __forceinline__ int item_expert(int e0, int e1, int row) {
    const int a = __shfl_sync(0xffffffffu, e0, row & 31);
    const int b = __shfl_sync(0xffffffffu, e1, row & 31);
    return row < 32 ? a : b;
}

// Producer: claims the next slot of consumer group `grp` and starts this lane's copy into it.
// Returns false after a give-up.
__device__ __forceinline__ bool ring_put(const IdxSmem &s, int stage_bytes, int ns2, int grp, RingPos &cur,
                                         uint32_t expect_bytes, bool mine, const uint8_t *src, uint32_t row_bytes,
                                         int lane, void *ws, int where) {
    const int stage = grp * ns2 + cur.slot;
    int go = 1;
    if (lane == 0) {
        if (cur.round > 0 && !wait_or_abort(&s.empty[stage], (cur.round - 1) & 1, s.abort, ws, where)) go = 0;
        if (go) mbar_arrive_expect_tx(&s.full[stage], expect_bytes);
    }
    go = __shfl_sync(0xffffffffu, go, 0);
    if (!go) return false;
    if (mine) bulk_g2s(s.stages + (size_t)stage * stage_bytes + (size_t)lane * row_bytes, src, row_bytes, &s.full[stage]);
    cur.advance(ns2);
    return true;
}

// WPG: consumer warps of a group per (gate, up) pair = 4 / R; NU: 16-byte units of a row per
// consumer thread of a group in the second half (row_units <= 128 * NU).  GATED = false: the block
// has no gate (Eq. 2), z_j = sigma(W_1[j, :] . x + b_1[j]); a pair of the first half is then two
// consecutive experts' rows of W_1, staged like the rows of W_2^T.
template <int WPG, int NU, bool GATED>
__global__ void __launch_bounds__(DEC_THREADS, 1) decode_indexed_kernel(const __grid_constant__ IndexedParams p, int act) {
    constexpr int R = DEC_GROUP_WARPS / WPG;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    // (in registers: the asm statements in the loops clobber memory, and a reload of a kernel
    // parameter costs a round trip)
    const int d = p.d, k = p.k, B = p.B, n_slices = p.n_slices, n_stages = p.n_stages;
    void *const ws = p.ws;
    const int row_units = d >> 3;
    const uint32_t row_bytes = (uint32_t)row_units * 16;
    const int stage_bytes = 2 * R * (int)row_bytes;
    const int ns2 = n_stages >> 1;
    const IdxSmem s = carve_idx(smem_raw, n_stages, stage_bytes, d);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < n_stages; ++i) {
            mbar_init(&s.full[i], 1);
            mbar_init(&s.empty[i], DEC_GROUP_WARPS);
        }
        *s.abort = 0;
        mbar_fence_init();
    }
    __syncthreads();
    pdl_launch_dependents();
    const int n_items = B * n_slices;

    if (warp == DEC_CONSUMER_WARPS) {
        // ---- producer warp: weights and E only
        const uint8_t *const wg = static_cast<const uint8_t *>(p.w_gate);
        const uint8_t *const wu = static_cast<const uint8_t *>(p.w_up);
        const uint8_t *const wd = static_cast<const uint8_t *>(p.w_down_t);
        const int32_t *const idx = p.idx;
        const unsigned d_ff = (unsigned)p.d_ff;
        RingPos pos0 = {0, 0, 0}, pos1 = {0, 0, 0};
        uint32_t pgc = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
            const int b = item / n_slices, sl = item - b * n_slices;
            const int r0 = (int)((long long)sl * k / n_slices);
            const int n = (int)((long long)(sl + 1) * k / n_slices) - r0;
            // an index outside [0, d_ff) is never dereferenced: row 0 stands in (the consumers
            // give that neuron z = 0 and raise the status word)
            int e0 = lane < n ? __ldg(idx + (size_t)b * k + r0 + lane) : 0;
            int e1 = lane + 32 < n ? __ldg(idx + (size_t)b * k + r0 + 32 + lane) : 0;
            if ((unsigned)e0 >= d_ff) e0 = 0;
            if ((unsigned)e1 >= d_ff) e1 = 0;
            for (int rg = 0; !GATED && ok && rg < n; rg += 2 * R, ++pgc) {  // no gate: rows of W_1, two per pair
                const int row = rg + lane;
                const int e = item_expert(e0, e1, row & 63);
                const bool mine = lane < 2 * R && row < n;
                const uint32_t rows = (uint32_t)min(2 * R, n - rg);
                const uint8_t *src = wu + (size_t)e * row_bytes;
                RingPos cur = (pgc & 1) ? pos1 : pos0;
                ok = ring_put(s, stage_bytes, ns2, pgc & 1, cur, rows * row_bytes, mine, src, row_bytes, lane, ws, 20);
                if (pgc & 1) pos1 = cur; else pos0 = cur;
            }
            for (int pg = 0; GATED && ok && pg < n; pg += R, ++pgc) {  // (gate, up) pairs
                const int pair = pg + (lane >> 1);
                const int e = item_expert(e0, e1, pair & 63);
                const bool mine = lane < 2 * R && pair < n;
                const uint32_t rows = 2 * (uint32_t)min(R, n - pg);
                const uint8_t *src = ((lane & 1) ? wu : wg) + (size_t)e * row_bytes;
                RingPos cur = (pgc & 1) ? pos1 : pos0;
                ok = ring_put(s, stage_bytes, ns2, pgc & 1, cur, rows * row_bytes, mine, src, row_bytes, lane, ws, 20);
                if (pgc & 1) pos1 = cur; else pos0 = cur;
            }
            for (int rg = 0; ok && rg < n; rg += 2 * R, ++pgc) {  // rows of W_2^T
                const int row = rg + lane;
                const int e = item_expert(e0, e1, row & 63);
                const bool mine = lane < 2 * R && row < n;
                const uint32_t rows = (uint32_t)min(2 * R, n - rg);
                const uint8_t *src = wd + (size_t)e * row_bytes;
                RingPos cur = (pgc & 1) ? pos1 : pos0;
                ok = ring_put(s, stage_bytes, ns2, pgc & 1, cur, rows * row_bytes, mine, src, row_bytes, lane, ws, 21);
                if (pgc & 1) pos1 = cur; else pos0 = cur;
            }
        }
        if (lane == 0) {  // stay until every copy has landed (only matters after a give-up)
            MmaSmem ms;
            ms.full = s.full;
            const uint32_t issued[2] = {pos0.uses, pos1.uses};
            producer_drain_mma(ms, n_stages, issued);
        }
        return;
    }

    // ---- consumers
    pdl_wait_prior_grids();  // x, the partial sums and y belong to earlier work on the stream
    const int group = warp / DEC_GROUP_WARPS, wig = warp - group * DEC_GROUP_WARPS;
    const int tig = tid - group * (DEC_GROUP_WARPS * 32);
    const int my_pair = wig / WPG, q = wig - my_pair * WPG;
    const int lane_unit = q * 32 + lane;
    int my_full, tail_lanes;
    my_blocks<WPG>(row_units, q, my_full, tail_lanes);
    RingPos pos = {0, 0, 0};
    uint32_t pgc = 0;
    int item_parity = 0;
    bool ok = true;

    for (int item = blockIdx.x; item < n_items; item += gridDim.x, item_parity ^= 1) {
        const int b = item / n_slices, sl = item - b * n_slices;
        const int r0 = (int)((long long)sl * k / n_slices);
        const int n = (int)((long long)(sl + 1) * k / n_slices) - r0;
        float2 *part = s.part + item_parity * (DEC_MAX_ROWS * DEC_CONSUMER_WARPS);
        const uint32_t pgc0 = pgc;
        // before a further item both groups are done with the previous one (z, partial sums)
        if (item != (int)blockIdx.x) consumer_barrier();
        // x of this sequence, this lane's units of it (read again for every item, so that the
        // registers are free during the second half; the read hits L2)
        uint4 xr[MMA_BLOCKS_PER_WARP];
        {
            const uint4 *src = reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(p.x) + (size_t)b * d);
            const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int i = 0; i < MMA_BLOCKS_PER_WARP; ++i) {
                const int u = i * (WPG * 32) + lane_unit;
                xr[i] = u < row_units ? __ldcg(src + u) : zero;
            }
        }
        // this thread's neuron of the item (used after the first half)
        int my_e = 0;
        if (tig < n) my_e = __ldg(p.idx + (size_t)b * k + r0 + tig);
        if (*s.abort) ok = false;

        // ---- first half: z of the slice
        const int n_pairs = GATED ? n : (n + 1) >> 1;
        for (int pg = 0; pg < n_pairs; pg += R, ++pgc) {
            if (!ok) continue;
            if ((int)(pgc & 1) != group) continue;
            const bool have = pg + my_pair < n_pairs;
            float acc[MMA_ACCS][4] = {};
            const int stage = group * ns2 + pos.slot;
            if (!wait_or_abort(&s.full[stage], pos.round & 1, s.abort, ws, 22)) {
                ok = false;
                continue;
            }
            if (have) {
                const uint4 *p0 = reinterpret_cast<const uint4 *>(s.stages + (size_t)stage * stage_bytes +
                                                                  (size_t)(2 * my_pair) * row_bytes) +
                                  lane_unit;
                pair_mma<false, true, WPG>(acc, p0, p0 + row_units, p0, p0, xr, xr, my_full, tail_lanes, lane);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&s.empty[stage]);
            pos.advance(ns2);
            if (have) {
                float sum[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float lo = (acc[0][e] + acc[1][e]) + (acc[2][e] + acc[3][e]);
                    if (MMA_ACCS == 8)
                        lo += (acc[4 % MMA_ACCS][e] + acc[5 % MMA_ACCS][e]) + (acc[6 % MMA_ACCS][e] + acc[7 % MMA_ACCS][e]);
                    sum[e] = lo;
                }
                const float dsum = diagonal_sum(sum, lane);
                float *slot = reinterpret_cast<float *>(&part[(pg + my_pair) * DEC_CONSUMER_WARPS + q]);
                if (lane == 0) slot[0] = dsum;  // gate row
                if (lane == 4) slot[1] = dsum;  // up row
            }
        }
        group_barrier(group);  // this group's partial sums are in place
        if (*s.abort) ok = false;
        const int my_pair_of_item = GATED ? tig : tig >> 1;  // the pair that holds this thread's neuron
        if (tig < n && (int)((pgc0 + my_pair_of_item / R) & 1) == group) {
            float a0 = 0.f, a1 = 0.f;
            for (int w = 0; w < WPG; ++w) {
                const float2 v = part[my_pair_of_item * DEC_CONSUMER_WARPS + w];
                a0 += v.x;
                a1 += v.y;
            }
            float zv = 0.f;
            if ((unsigned)my_e < (unsigned)p.d_ff) {
                if (GATED) {
                    if (p.b_gate) a0 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.b_gate)[my_e]);
                    if (p.b_up) a1 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.b_up)[my_e]);
                    zv = sigma_rt(act, a0) * a1;
                } else {
                    float u = (tig & 1) ? a1 : a0;
                    if (p.b_up) u += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.b_up)[my_e]);
                    zv = sigma_rt(act, u);
                }
            } else {
                raise_status(ws, DEV_STATUS_BAD_INDEX, 23);
            }
            s.zs[tig] = ok ? zv : 0.f;
        }
        consumer_barrier();  // z of the slice is complete

        // ---- second half: y += z_j * (row j of W_2^T)
        float yacc[NU][8];  // (live in this half only: the first half needs the registers)
#pragma unroll
        for (int i = 0; i < NU; ++i)
#pragma unroll
            for (int e = 0; e < 8; ++e) yacc[i][e] = 0.f;
        for (int rg = 0; rg < n; rg += 2 * R, ++pgc) {
            if (!ok) continue;
            if ((int)(pgc & 1) != group) continue;
            const int stage = group * ns2 + pos.slot;
            if (!wait_or_abort(&s.full[stage], pos.round & 1, s.abort, ws, 24)) {
                ok = false;
                continue;
            }
            const int rows = min(2 * R, n - rg);
            const uint4 *st = reinterpret_cast<const uint4 *>(s.stages + (size_t)stage * stage_bytes) + tig;
#pragma unroll
            for (int r = 0; r < 2 * R; ++r) {
                if (r < rows) {  // warp-uniform
                    const float zr = s.zs[rg + r];
#pragma unroll
                    for (int i0 = 0; i0 < NU; i0 += 4) {  // four loads in flight, then their FMAs
                        uint4 v[4];
#pragma unroll
                        for (int i = i0; i < i0 + 4 && i < NU; ++i)
                            if (tig + 128 * i < row_units) v[i - i0] = st[r * row_units + 128 * i];
#pragma unroll
                        for (int i = i0; i < i0 + 4 && i < NU; ++i)
                            if (tig + 128 * i < row_units) {
                                float f[8];
                                Elem<__nv_bfloat16>::unpack(v[i - i0], f);
#pragma unroll
                                for (int e = 0; e < 8; ++e) yacc[i][e] = fmaf(zr, f[e], yacc[i][e]);
                            }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&s.empty[stage]);
            pos.advance(ns2);
        }

        // ---- the item's share of y joins the CTA's partial y of this sequence in the workspace
        //      (the second group's half goes through shared memory; a CTA's row is its own, so
        //      adding to what an earlier item of the same sequence left there needs no ordering)
        if (group == 1) {
#pragma unroll
            for (int i = 0; i < NU; ++i)
                if (tig + 128 * i < row_units) {
                    float4 *dst = reinterpret_cast<float4 *>(s.ysm) + 2 * (tig + 128 * i);
                    dst[0] = make_float4(yacc[i][0], yacc[i][1], yacc[i][2], yacc[i][3]);
                    dst[1] = make_float4(yacc[i][4], yacc[i][5], yacc[i][6], yacc[i][7]);
                }
        }
        consumer_barrier();
        if (group == 0) {
            const bool first_of_b = item - (int)gridDim.x < b * n_slices;  // no earlier item of this CTA in sequence b
            float4 *out = reinterpret_cast<float4 *>(p.ypart + ((size_t)b * gridDim.x + blockIdx.x) * d);
#pragma unroll
            for (int i = 0; i < NU; ++i)
                if (tig + 128 * i < row_units) {
                    const float4 *o = reinterpret_cast<const float4 *>(s.ysm) + 2 * (tig + 128 * i);
                    float4 a = o[0], c = o[1];
                    if (!first_of_b) {
                        const float4 pa = __ldcg(out + 2 * (tig + 128 * i)), pc = __ldcg(out + 2 * (tig + 128 * i) + 1);
                        a.x += pa.x; a.y += pa.y; a.z += pa.z; a.w += pa.w;
                        c.x += pc.x; c.y += pc.y; c.z += pc.z; c.w += pc.w;
                    }
                    out[2 * (tig + 128 * i)] =
                        make_float4(yacc[i][0] + a.x, yacc[i][1] + a.y, yacc[i][2] + a.z, yacc[i][3] + a.w);
                    out[2 * (tig + 128 * i) + 1] =
                        make_float4(yacc[i][4] + c.x, yacc[i][5] + c.y, yacc[i][6] + c.z, yacc[i][7] + c.w);
                }
        }
    }

    // ---- this CTA's partial sums are written.  The CTAs report in on a counter that runs round
    //      modulo 2 n and is never reset (as at the meeting point of the compact-set kernel); the
    //      order of arrival decides who adds the partial sums up: the last n_red CTAs to arrive
    //      wait (bounded) until everybody has reported and take the column blocks between them,
    //      the earlier ones are done and leave their SM to the next kernel on the stream.
    consumer_barrier();
    volatile int *role = reinterpret_cast<volatile int *>(s.zs);  // (z is not needed any more)
    const int n_red = p.n_red;
    if (tid == 0) {
        unsigned int *counter = &static_cast<WsHeader *>(ws)->meet_idx;
        const unsigned int n = gridDim.x;
        __threadfence();
        const unsigned int old = atomicInc(counter, 2 * n - 1);
        const bool upper = old >= n;
        int mine = (int)(upper ? old - n : old) - ((int)n - n_red);  // >= 0: this CTA's first column block
        if (mine >= 0) {
            const long long t0 = clock64();
            for (;;) {
                const unsigned int v = ld_acquire_u32(counter);
                if (upper ? v < n : v >= n) break;
                if (*s.abort || clock64() - t0 > WAIT_LIMIT_CYCLES) {
                    *s.abort = 1;
                    raise_status(ws, DEV_STATUS_TIMEOUT, 25);
                    mine = -1;
                    break;
                }
            }
        }
        *role = mine;
    }
    consumer_barrier();
    const int first_blk = *role;
    if (first_blk < 0) return;
    const int V = p.red_vec;            // columns per lane: 1 or 4
    const int total = B * d;            // columns of all sequences
    const int blk_cols = 32 * V;
    const int n_blocks = (total + blk_cols - 1) / blk_cols;
    const int grid = (int)gridDim.x;
    for (int blk = first_blk; blk < n_blocks; blk += n_red) {
        const int col = blk * blk_cols + lane * V;  // V divides d: the lane's columns lie in one sequence
        float4 acc4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (col < total) {
            const int b = col / d, c = col - b * d;
            const float *src = p.ypart + (size_t)b * grid * d + c;
            if (V == 4) {
                for (int r = warp; r < grid; r += DEC_CONSUMER_WARPS) {
                    const float4 v = __ldcg(reinterpret_cast<const float4 *>(src + (size_t)r * d));
                    acc4.x += v.x; acc4.y += v.y; acc4.z += v.z; acc4.w += v.w;
                }
            } else {
                for (int r = warp; r < grid; r += DEC_CONSUMER_WARPS) acc4.x += __ldcg(src + (size_t)r * d);
            }
        }
        reinterpret_cast<float4 *>(s.red)[warp * 32 + lane] = acc4;
        consumer_barrier();
        if (warp == 0 && col < total) {
            float4 t = reinterpret_cast<const float4 *>(s.red)[lane];
            for (int w = 1; w < DEC_CONSUMER_WARPS; ++w) {
                const float4 v = reinterpret_cast<const float4 *>(s.red)[w * 32 + lane];
                t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
            }
            const int c = col % d;
            const __nv_bfloat16 *bd = static_cast<const __nv_bfloat16 *>(p.b_down);
            __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(p.y) + col;
            if (V == 4) {
                if (bd) {
                    t.x += __bfloat162float(bd[c]); t.y += __bfloat162float(bd[c + 1]);
                    t.z += __bfloat162float(bd[c + 2]); t.w += __bfloat162float(bd[c + 3]);
                }
                __nv_bfloat162 lo = __floats2bfloat162_rn(t.x, t.y), hi = __floats2bfloat162_rn(t.z, t.w);
                uint2 o;
                o.x = *reinterpret_cast<uint32_t *>(&lo);
                o.y = *reinterpret_cast<uint32_t *>(&hi);
                *reinterpret_cast<uint2 *>(y) = o;
            } else {
                if (bd) t.x += __bfloat162float(bd[c]);
                *y = __float2bfloat16_rn(t.x);
            }
        }
        consumer_barrier();
    }
}

size_t decode_indexed_scratch_bytes(int d, int n_seq) {
    return (size_t)n_seq * IDX_MAX_GRID * (size_t)d * sizeof(float);
}

griffin_status launch_decode_indexed(const griffin_ff_desc *desc, int B, const griffin_ff_weights_nm *w,
                                     const int32_t *idx, int k, const void *x, void *y, float *ypart, void *ws,
                                     uint32_t flags, cudaStream_t stream) {
    const int sms = device_sm_count();
    if (sms <= 0) return GRIFFIN_ERR_CUDA;
    IndexedParams p = {};
    p.w_gate = w->w_gate;
    p.w_up = w->w_up;
    p.w_down_t = w->w_down_t;
    p.b_gate = w->b_gate;
    p.b_up = w->b_up;
    p.b_down = w->b_down;
    p.idx = idx;
    p.x = x;
    p.y = y;
    p.ypart = ypart;
    p.ws = ws;
    p.d = desc->d;
    p.d_ff = desc->d_ff;
    p.k = k;
    p.B = B;
    // every CTA of the grid must be resident (they meet at the end): one per SM, and no more
    // than the partial-sum rows the workspace was sized for
    const int grid = sms < IDX_MAX_GRID ? sms : IDX_MAX_GRID;
    p.n_slices = slices_for(k, grid);
    const MmaPlan pl = make_plan(desc->d, 16, MMA_STAGE_TARGET, MMA_BLOCKS_PER_WARP);
    if (pl.n_chunks != 1) return GRIFFIN_ERR_UNSUPPORTED;
    int n = ((int)MMA_SMEM_TARGET - (int)idx_fixed_smem(p.d, 8)) / pl.stage_bytes;
    p.n_stages = (n > 8 ? 8 : n) & ~1;
    if (p.n_stages < 2) return GRIFFIN_ERR_UNSUPPORTED;
    const long long total = (long long)B * p.d;
    p.red_vec = total > 32ll * grid ? 4 : 1;  // narrow column blocks while every CTA gets at most one of them
    {
        const long long n_blocks = (total + 32 * p.red_vec - 1) / (32 * p.red_vec);
        p.n_red = n_blocks < grid ? (int)n_blocks : grid;
    }
    const int wpg = DEC_GROUP_WARPS / pl.R;
    const int nu = (pl.row_units + 127) / 128;
    const void *fn = nullptr;
    const bool gated = act_gated(desc->act);
    if (wpg == 1 && nu <= 2)
        fn = gated ? (const void *)decode_indexed_kernel<1, 2, true> : (const void *)decode_indexed_kernel<1, 2, false>;
    else if (wpg == 2 && nu <= 4)
        fn = gated ? (const void *)decode_indexed_kernel<2, 4, true> : (const void *)decode_indexed_kernel<2, 4, false>;
    else if (wpg == 4 && nu <= 8)
        fn = gated ? (const void *)decode_indexed_kernel<4, 8, true> : (const void *)decode_indexed_kernel<4, 8, false>;
    else return GRIFFIN_ERR_UNSUPPORTED;
    const size_t smem = (size_t)p.n_stages * pl.stage_bytes + idx_fixed_smem(p.d, p.n_stages);
    if (smem > 227 * 1024) return GRIFFIN_ERR_UNSUPPORTED;
    if (ensure_dynamic_smem(fn, smem) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    if (!grid_can_meet(fn, DEC_THREADS, smem, grid)) return GRIFFIN_ERR_UNSUPPORTED;
    int act = act_sigma(desc->act);
    void *args[] = {&p, &act};
    const bool overlap = (flags & GRIFFIN_DECODE_OVERLAP_WEIGHT_PREFETCH) != 0;
    if (launch_maybe_overlapped(fn, dim3(grid), dim3(DEC_THREADS), smem, stream, overlap, args) != cudaSuccess)
        return GRIFFIN_ERR_CUDA;
    return GRIFFIN_OK;
}

}  // namespace griffin
