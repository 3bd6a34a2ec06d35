// Prompt-phase FF on the 5th-generation tensor cores (Eqs. 1 and 3 of the GRIFFIN paper), bf16
// storage, fp32 accumulation:
//   kernel<KIND = 1> : Z = sigma(X W_g^T + b_g) * (X W_1^T + b_1), also the bf16 residual Z - bf16(Z) and the
//                      per-tile partial sums of squares of its rows (for the statistic)
//   kernel<KIND = 2> : the same for a block without a gate (Eq. 2): Z = sigma(X W_1^T + b_1)
//   kernel<KIND = 0> : Y = Z W_2^T + b_2
//
// One persistent CTA per SM, 320 threads in three roles:
//   warp 0      TMA producer: cp.async.bulk.tensor (2-D tiles, 128-byte swizzle, no multicast)
//               of a 128 x 64 tile of the left operand and a BN x 64 tile of the weights
//               into a ring of shared-memory stages;
//   warp 1      MMA issuer: one elected thread issues tcgen05.mma (M = 128, N = BN, K = 16,
//               operands from shared memory through matrix descriptors, accumulator in TMEM),
//               releases each stage with tcgen05.commit; it also owns the TMEM allocation;
//   warps 2-9   epilogue: tcgen05.ld of the accumulator (one row per thread), activation and
//               gating (or bias), stores.  A warp may read the TMEM lanes 32 (w mod 4) .. + 31, so
//               warps w and w + 4 share a quarter of the rows and take half of the columns each
//               (measured: with four warps the epilogue of a tile took 23 us of dependent
//               latencies, one warp per scheduler, and the last one of a CTA is never hidden).
//               TMEM holds two accumulator stages, so the epilogue of one tile runs under the
//               MMAs of the next.
// For DUAL the gate and up tiles of the same 128 neurons are loaded one behind the other, so
// that a single N = 256 MMA against the shared X tile fills columns 0..127 with the gate
// and 128..255 with the up pre-activations: the epilogue thread that owns a row finds both.
// Without a gate the same two loads take 256 consecutive neurons of W_1, and every accumulator
// column is a neuron of its own.
//
// Every wait is bounded; after a give-up the CTA still frees its TMEM before it returns.
#include <stdlib.h>

#include "prefill_tc.cuh"

namespace griffin {

struct TcSmem {
    uint8_t *stages;
    uint64_t *full, *empty, *acc_full, *acc_empty;
    uint32_t *tmem_slot;
    uint8_t *stg;  // TC_EPI_WARPS staging buffers
    volatile int *abort;
};
constexpr size_t TC_TAIL_BYTES = (2 * TC_STAGES + 4) * sizeof(uint64_t) + 16 + TC_EPI_WARPS * TC_STG_BYTES;

template <int KIND, int BN>
__global__ void __launch_bounds__(TC_THREADS) ff_tc_kernel(const __grid_constant__ CUtensorMap map_a,
                                                           const __grid_constant__ CUtensorMap map_b0,
                                                           const __grid_constant__ CUtensorMap map_b1,
                                                           const __grid_constant__ TcParams p) {
    constexpr bool DUAL = KIND != TC_PLAIN;        // two weight loads of 128 rows per stage, N = 256
    constexpr int NT = DUAL ? 256 : BN;            // MMA N = TMEM columns of one accumulator stage
    constexpr int B_ROWS = DUAL ? 128 : BN;        // rows of one weight tile load
    constexpr int A_BYTES = TC_BM * TC_BK * 2;     // 16 KB
    constexpr int STAGE_BYTES = A_BYTES + NT * TC_BK * 2;
    constexpr uint32_t IDESC = umma_idesc(TC_BM, NT);

    extern __shared__ uint8_t smem_raw[];
    TcSmem s;
    s.stages = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    s.full = reinterpret_cast<uint64_t *>(s.stages + (size_t)TC_STAGES * STAGE_BYTES);
    s.empty = s.full + TC_STAGES;
    s.acc_full = s.empty + TC_STAGES;
    s.acc_empty = s.acc_full + 2;
    s.tmem_slot = reinterpret_cast<uint32_t *>(s.acc_empty + 2);
    s.abort = reinterpret_cast<volatile int *>(s.tmem_slot + 1);
    s.stg = reinterpret_cast<uint8_t *>(s.full) + (2 * TC_STAGES + 4) * sizeof(uint64_t) + 16;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < TC_STAGES; ++i) {
            mbar_init(&s.full[i], 1);
            mbar_init(&s.empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s.acc_full[i], 1);
            mbar_init(&s.acc_empty[i], TC_EPI_WARPS);  // one arrival per epilogue warp
        }
        *s.abort = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(s.tmem_slot, 2 * NT);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();  // a finishing kernel behind this one may take its place on the SMs and wait there
    const uint32_t tmem_base = *s.tmem_slot;

    // work items: (m, n, K split), or whole tiles followed by the parts of the cut ones
    const int n_tiles_total = p.tail_ks > 1 ? p.tail_first + (p.m_tiles * p.n_tiles - p.tail_first) * p.tail_ks
                                            : p.m_tiles * p.n_tiles * p.splits;
    const int kb_total = p.K / TC_BK;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < n_tiles_total; tile += gridDim.x) {
                const TcItem ti = tc_item(p, tile, kb_total);
                const int m = ti.m, n = ti.n, kb0 = ti.kb0, kb1 = ti.kb1;
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int stage = it % TC_STAGES;
                    const uint32_t use = it / TC_STAGES;
                    if (use > 0 && !wait_or_abort(&s.empty[stage], (use - 1) & 1, s.abort, p.ws, 20)) {
                        ok = false;
                        break;
                    }
                    uint8_t *a = s.stages + (size_t)stage * STAGE_BYTES;
                    mbar_arrive_expect_tx(&s.full[stage], STAGE_BYTES);
                    tma_load_2d(a, &map_a, kb * TC_BK, m * TC_BM, &s.full[stage]);
                    tma_load_2d(a + A_BYTES, &map_b0, kb * TC_BK, KIND == TC_WIDE ? n * 256 : n * B_ROWS, &s.full[stage]);
                    if (DUAL)
                        tma_load_2d(a + A_BYTES + B_ROWS * TC_BK * 2, &map_b1, kb * TC_BK,
                                    KIND == TC_WIDE ? n * 256 + 128 : n * B_ROWS, &s.full[stage]);
                }
            }
            // stay until every copy that was started has landed
            const uint32_t first = it > TC_STAGES ? it - TC_STAGES : 0;
            for (uint32_t j = first; j < it; ++j) {
                const long long t0 = clock64();
                while (!mbar_try_wait(&s.full[j % TC_STAGES], (j / TC_STAGES) & 1))
                    if (clock64() - t0 > WAIT_LIMIT_CYCLES) break;
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < n_tiles_total; tile += gridDim.x, ++tcount) {
                const int acc = tcount & 1;
                const uint32_t acc_use = tcount >> 1;
                if (acc_use > 0 && !wait_or_abort(&s.acc_empty[acc], (acc_use - 1) & 1, s.abort, p.ws, 21)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * NT);
                const TcItem ti = tc_item(p, tile, kb_total);
                const int kb0 = ti.kb0, kb1 = ti.kb1;
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int stage = it % TC_STAGES;
                    if (!wait_or_abort(&s.full[stage], (it / TC_STAGES) & 1, s.abort, p.ws, 22)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint8_t *a = s.stages + (size_t)stage * STAGE_BYTES;
#pragma unroll
                    for (int k16 = 0; k16 < TC_BK / 16; ++k16)
                        umma_bf16(d_tmem, smem_desc_sw128(a, k16), smem_desc_sw128(a + A_BYTES, k16), IDESC,
                                  (kb > kb0 || k16 > 0) ? 1u : 0u);
                    umma_commit(&s.empty[stage]);  // the stage may be refilled once these MMAs have read it
                }
                if (ok) umma_commit(&s.acc_full[acc]);
            }
        }
    } else {
        // ---------------- epilogue (warps 2..9) ----------------
        const int wq = warp & 3;                 // the TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;        // which half of the tile's columns this warp takes
        uint8_t *const stg = s.stg + (warp - 2) * TC_STG_BYTES;
        uint32_t tcount = 0;
        for (int tile = blockIdx.x; tile < n_tiles_total; tile += gridDim.x, ++tcount) {
            const TcItem ti = tc_item(p, tile, kb_total);
            const int m = ti.m, n = ti.n, sp = ti.sp;
            const int acc = tcount & 1;
            // (256 threads wait here for most of a tile's main loop: they sleep between polls)
            if (!wait_or_abort_relaxed(&s.acc_full[acc], (tcount >> 1) & 1, s.abort, p.ws, 23)) break;
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16) + (uint32_t)(acc * NT);
            tc_epilogue_item<KIND, BN>(p, m, n, sp, ti.part, taddr, stg, wq, half, lane);
            tc_fence_before_sync();  // this warp's TMEM reads are done
            __syncwarp();
            if (lane == 0) mbar_arrive(&s.acc_empty[acc]);
        }
    }

    // ---------------- teardown: everybody meets, the allocating warp frees TMEM ----------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 2 * NT);
    }
}

// Finishes the cut tiles of the first GEMM: one warp per (cut tile, row), four neurons of the tile per
// lane.  The parts are added in order, then bias, activation and gating as in the epilogue above:
// Z in bf16 and fp32, and the row's sum of squares over the tile's 128 columns (fixed order).
__global__ void __launch_bounds__(128) dual_tail_finish_kernel(TcParams p) {
    pdl_wait_prior_grids();  // (launched to start early: everything it reads comes from the GEMM kernel before it)
    const int w = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    const int tile = p.tail_first + w / TC_BM, r = w % TC_BM, c = lane * 4;
    const int m = tile % p.m_tiles, n = tile / p.m_tiles;
    // with a gate the two halves of a part are the gate and up sums of the same 128 neurons; without
    // one they are 256 neurons of W_1
    const int row = m * TC_BM + r, col = p.gated ? n * 128 + c : n * 256 + c, col2 = p.gated ? col : col + 128;
    float4 g = make_float4(0.f, 0.f, 0.f, 0.f), u = g, a[4], b[4];
#pragma unroll
    for (int sp = 0; sp < 4; ++sp) {  // at most four parts; all loads in flight together
        a[sp] = b[sp] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (sp < p.tail_ks) {
            const float *src = p.tail_part + ((size_t)((tile - p.tail_first) * p.tail_ks + sp) * TC_BM + r) * 256;
            a[sp] = __ldcs(reinterpret_cast<const float4 *>(src + c));
            b[sp] = __ldcs(reinterpret_cast<const float4 *>(src + 128 + c));
        }
    }
#pragma unroll
    for (int sp = 0; sp < 4; ++sp) {  // added in order (absent parts are zeros)
        g.x += a[sp].x; g.y += a[sp].y; g.z += a[sp].z; g.w += a[sp].w;
        u.x += b[sp].x; u.y += b[sp].y; u.z += b[sp].z; u.w += b[sp].w;
    }
    float gv[4] = {g.x, g.y, g.z, g.w}, uv[4] = {u.x, u.y, u.z, u.w}, z[4];
    float sq = 0.f;
    if (!p.gated) {
        float z2[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (p.bias1) {
                gv[i] += __bfloat162float(p.bias1[col + i]);
                uv[i] += __bfloat162float(p.bias1[col2 + i]);
            }
            z[i] = sigma_fast_rt(p.act, gv[i]);
            z2[i] = sigma_fast_rt(p.act, uv[i]);
            sq = fmaf(z[i], z[i], sq);
            sq = fmaf(z2[i], z2[i], sq);
        }
        if (row < p.S) {
            const __nv_bfloat162 h0 = __floats2bfloat162_rn(z2[0], z2[1]), h1 = __floats2bfloat162_rn(z2[2], z2[3]);
            *reinterpret_cast<uint2 *>(p.out + (size_t)row * p.n_total + col2) =
                make_uint2(*reinterpret_cast<const uint32_t *>(&h0), *reinterpret_cast<const uint32_t *>(&h1));
            const __nv_bfloat162 l0 = __floats2bfloat162_rn(z2[0] - __low2float(h0), z2[1] - __high2float(h0));
            const __nv_bfloat162 l1 = __floats2bfloat162_rn(z2[2] - __low2float(h1), z2[3] - __high2float(h1));
            *reinterpret_cast<uint2 *>(p.zlo + (size_t)row * p.n_total + col2) =
                make_uint2(*reinterpret_cast<const uint32_t *>(&l0), *reinterpret_cast<const uint32_t *>(&l1));
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (p.bias0) gv[i] += __bfloat162float(p.bias0[col + i]);
            if (p.bias1) uv[i] += __bfloat162float(p.bias1[col + i]);
            z[i] = sigma_fast_rt(p.act, gv[i]) * uv[i];
            sq = fmaf(z[i], z[i], sq);
        }
    }
    if (row < p.S) {
        const __nv_bfloat162 h0 = __floats2bfloat162_rn(z[0], z[1]), h1 = __floats2bfloat162_rn(z[2], z[3]);
        *reinterpret_cast<uint2 *>(p.out + (size_t)row * p.n_total + col) =
            make_uint2(*reinterpret_cast<const uint32_t *>(&h0), *reinterpret_cast<const uint32_t *>(&h1));
        const __nv_bfloat162 l0 = __floats2bfloat162_rn(z[0] - __low2float(h0), z[1] - __high2float(h0));
        const __nv_bfloat162 l1 = __floats2bfloat162_rn(z[2] - __low2float(h1), z[3] - __high2float(h1));
        *reinterpret_cast<uint2 *>(p.zlo + (size_t)row * p.n_total + col) =
            make_uint2(*reinterpret_cast<const uint32_t *>(&l0), *reinterpret_cast<const uint32_t *>(&l1));
    }
    sq = warp_sum(sq);
    if (lane < 2 && row < p.S) p.rowsq[(size_t)row * (2 * p.n_tiles) + 2 * n + lane] = lane == 0 ? sq : 0.f;
}

// Finishes the cut tiles of the down projection: one warp per (cut tile, row), eight outputs per lane.
// The parts are added in order, then b_2, then rounded to bf16.
__global__ void __launch_bounds__(128) plain_tail_finish_kernel(TcParams p) {
    pdl_wait_prior_grids();
    const int w = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    const int tile = p.tail_first + w / TC_BM, r = w % TC_BM, c = lane * 8;
    const int m = tile % p.m_tiles, n = tile / p.m_tiles;
    const int row = m * TC_BM + r, col = n * 256 + c;
    float4 a[4][2];
#pragma unroll
    for (int sp = 0; sp < 4; ++sp) {  // at most four parts; all loads in flight together
        a[sp][0] = a[sp][1] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (sp < p.tail_ks) {
            const float4 *src = reinterpret_cast<const float4 *>(
                p.tail_part + ((size_t)((tile - p.tail_first) * p.tail_ks + sp) * TC_BM + r) * 256 + c);
            a[sp][0] = __ldcs(src);
            a[sp][1] = __ldcs(src + 1);
        }
    }
    float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int sp = 0; sp < 4; ++sp) {  // added in order (absent parts are zeros)
        v[0] += a[sp][0].x; v[1] += a[sp][0].y; v[2] += a[sp][0].z; v[3] += a[sp][0].w;
        v[4] += a[sp][1].x; v[5] += a[sp][1].y; v[6] += a[sp][1].z; v[7] += a[sp][1].w;
    }
    if (row >= p.S) return;
    uint32_t packed[4];
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
        float y0 = v[i], y1 = v[i + 1];
        if (p.bias0) { y0 += __bfloat162float(p.bias0[col + i]); y1 += __bfloat162float(p.bias0[col + i + 1]); }
        const __nv_bfloat162 h = __floats2bfloat162_rn(y0, y1);
        packed[i >> 1] = *reinterpret_cast<const uint32_t *>(&h);
    }
    *reinterpret_cast<uint4 *>(p.out + (size_t)row * p.n_total + col) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
}

// y = bf16(sum over K splits of part + bias), four columns per thread, splits added in order.
__global__ void splitk_reduce_kernel(const float *__restrict__ part, const __nv_bfloat16 *__restrict__ bias,
                                     __nv_bfloat16 *__restrict__ y, int splits, size_t n_elems, int n_total) {
    pdl_wait_prior_grids();
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= n_elems) return;
    float4 acc = *reinterpret_cast<const float4 *>(part + i);
    for (int s = 1; s < splits; ++s) {
        const float4 v = *reinterpret_cast<const float4 *>(part + (size_t)s * n_elems + i);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    if (bias) {
        const int c = (int)(i % n_total);
        acc.x += __bfloat162float(bias[c]); acc.y += __bfloat162float(bias[c + 1]);
        acc.z += __bfloat162float(bias[c + 2]); acc.w += __bfloat162float(bias[c + 3]);
    }
    const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
    *reinterpret_cast<uint2 *>(y + i) =
        make_uint2(*reinterpret_cast<const uint32_t *>(&lo), *reinterpret_cast<const uint32_t *>(&hi));
}

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
constexpr int TC_TARGET_CTAS = 148;  // SMs of a B200: what a grid should fill

int gemm1_col_tiles(const griffin_ff_desc *desc) {
    return GRIFFIN_ACT_IS_GATED(desc->act) ? desc->d_ff / 128 : desc->d_ff / 256;
}

void gemm1_tail_plan(int S, int d, int n_col_tiles, int *tail_first, int *ks) {
    const int tiles = ((S + TC_BM - 1) / TC_BM) * n_col_tiles;
    const int rem = tiles % TC_TARGET_CTAS;
    *tail_first = tiles;
    *ks = 1;
    // (only where the last round is a large part of the whole: with many rounds the parts cost more than they save)
    if (tiles > TC_TARGET_CTAS && tiles <= 4 * TC_TARGET_CTAS && rem > 0 && 2 * rem <= TC_TARGET_CTAS && d / TC_BK >= 16) {
        const int k = TC_TARGET_CTAS / rem;
        *ks = k > 4 ? 4 : k;
        *tail_first = tiles - rem;
    }
}

size_t gemm1_tail_bytes(int S, int d, int n_col_tiles) {
    int first = 0, ks = 1;
    gemm1_tail_plan(S, d, n_col_tiles, &first, &ks);
    if (ks <= 1) return 0;
    const int tiles = ((S + TC_BM - 1) / TC_BM) * n_col_tiles;
    return (size_t)(tiles - first) * ks * TC_BM * 256 * sizeof(float);
}

void gemm2_plan(int S, int d, int d_ff, int *bn, int *splits) {
    const int m_tiles = (S + TC_BM - 1) / TC_BM;
    *bn = d % 256 == 0 ? 256 : 128;
    const int tiles = m_tiles * (d / *bn);
    // Uniform K splits, 1..4, by a small cost model in microseconds: the rounds that tiles x splits work
    // items need on one CTA per SM, at the measured pace of a long tile (about 10 TFLOP/s per SM), plus,
    // when there is a split, the fp32 partial sums written and read back (about 4 TB/s) and the launch of
    // the kernel that adds them.  A split must win by a tenth to be taken.
    const double tile_us = 2.0 * TC_BM * (double)*bn * (double)d_ff / 10e12 * 1e6;
    double cost1 = 0.0, best_cost = 0.0;
    int best = 1;
    for (int sp = 1; sp <= 4; ++sp) {
        const int rounds = (tiles * sp + TC_TARGET_CTAS - 1) / TC_TARGET_CTAS;
        double cost = rounds * tile_us / sp;
        if (sp > 1) cost += 2.0 * sp * (double)S * (double)d * 4.0 / 4e12 * 1e6 + 3.0;
        if (sp == 1) cost1 = best_cost = cost;
        else if (cost < 0.9 * cost1 && cost < best_cost) {
            best_cost = cost;
            best = sp;
        }
    }
    *splits = best;
}

// The same cut for the down projection when it runs in whole tiles 256 outputs wide: where the last
// round of tiles would leave at least half of the SMs idle, its tiles are cut along K into 2..4 parts.
void gemm2_tail_plan(int S, int d, int d_ff, int *tail_first, int *ks) {
    int bn = 0, splits = 1;
    gemm2_plan(S, d, d_ff, &bn, &splits);
    const int tiles = ((S + TC_BM - 1) / TC_BM) * (d / (bn > 0 ? bn : 1));
    const int rem = tiles % TC_TARGET_CTAS;
    *tail_first = tiles;
    *ks = 1;
    if (bn == 256 && splits == 1 && tiles > TC_TARGET_CTAS && rem > 0 && 2 * rem <= TC_TARGET_CTAS && d_ff / TC_BK >= 16) {
        const int k = TC_TARGET_CTAS / rem;
        *ks = k > 4 ? 4 : k;
        *tail_first = tiles - rem;
    }
}

size_t gemm2_tail_bytes(int S, int d, int d_ff) {
    int first = 0, ks = 1;
    gemm2_tail_plan(S, d, d_ff, &first, &ks);
    if (ks <= 1) return 0;
    const int tiles = ((S + TC_BM - 1) / TC_BM) * (d / 256);
    return (size_t)(tiles - first) * ks * TC_BM * 256 * sizeof(float);
}

// Row-major bf16 matrix [rows, cols] (cols contiguous); box = box_rows x 64 columns, 128-byte swizzle,
// out-of-range elements read as zero.
static bool make_map(CUtensorMap *map, const void *base, int rows, int cols, int box_rows) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (enc == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool prefill_tc_supported(const griffin_ff_desc *desc, int S) {
    if (desc->dtype != GRIFFIN_DT_BF16 || S < 1) return false;
    if (desc->d % 128 != 0 || desc->d_ff % 128 != 0) return false;  // whole tiles in N, whole stages in K
    if (!GRIFFIN_ACT_IS_GATED(desc->act) && desc->d_ff % 256 != 0) return false;  // (tiles of 256 neurons)
    return encode_tiled_fn() != nullptr;
}

template <int KIND, int BN>
static griffin_status launch_tc(const CUtensorMap &ma, const CUtensorMap &mb0, const CUtensorMap &mb1, const TcParams &p,
                                int sms, cudaStream_t stream) {
    constexpr int NT = KIND != TC_PLAIN ? 256 : BN;
    const size_t smem = 1024 + (size_t)TC_STAGES * (TC_BM * TC_BK * 2 + NT * TC_BK * 2) + TC_TAIL_BYTES;
    const void *fn = (const void *)ff_tc_kernel<KIND, BN>;
    if (ensure_dynamic_smem(fn, smem) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    const int tiles = p.tail_ks > 1 ? p.tail_first + (p.m_tiles * p.n_tiles - p.tail_first) * p.tail_ks
                                    : p.m_tiles * p.n_tiles * p.splits;
    ff_tc_kernel<KIND, BN><<<tiles < sms ? tiles : sms, TC_THREADS, smem, stream>>>(ma, mb0, mb1, p);
    count_launches(1);
    return cudaGetLastError() == cudaSuccess ? GRIFFIN_OK : GRIFFIN_ERR_CUDA;
}

griffin_status launch_prefill_tc(const griffin_ff_desc *desc, const griffin_ff_weights *w, const void *x, int S,
                                 void *y, __nv_bfloat16 *z, __nv_bfloat16 *zlo, float *rowsq, float *ypart, int *n_col_tiles,
                                 void *ws, cudaStream_t stream, cudaEvent_t after_ff1) {
    const int d = desc->d, d_ff = desc->d_ff;
    const int sms = device_sm_count();
    if (sms <= 0) return GRIFFIN_ERR_CUDA;
    const int m_tiles = (S + TC_BM - 1) / TC_BM;
    const bool gated = GRIFFIN_ACT_IS_GATED(desc->act);
    CUtensorMap mx, mg, mu;
    if (!make_map(&mx, x, S, d, TC_BM) || !make_map(&mu, w->w_up, d_ff, d, 128) ||
        !make_map(&mg, gated ? w->w_gate : w->w_up, d_ff, d, 128))
        return GRIFFIN_ERR_CUDA;
    TcParams p = {};
    p.S = S;
    p.n_total = d_ff;
    p.K = d;
    p.m_tiles = m_tiles;
    p.n_tiles = gemm1_col_tiles(desc);
    p.gated = gated ? 1 : 0;
    p.bias0 = static_cast<const __nv_bfloat16 *>(gated ? w->b_gate : nullptr);
    p.bias1 = static_cast<const __nv_bfloat16 *>(w->b_up);
    p.out = z;
    p.zlo = zlo;
    p.rowsq = rowsq;
    p.act = act_sigma(desc->act);
    p.ws = ws;
    p.splits = 1;
    gemm1_tail_plan(S, d, p.n_tiles, &p.tail_first, &p.tail_ks);
    p.tail_part = ypart;  // (the down projection's partials use the same scratch, later)
    *n_col_tiles = 2 * p.n_tiles;  // partial row sums per token: one per tile and column half
    // An even number of 128-token tiles: pairs of CTAs on tiles of 256 tokens, each staging half of the weight
    // tile (the environment variable GRIFFIN_TC_NO_PAIRS, set to anything, keeps one CTA per tile).
    static const bool no_pairs = getenv("GRIFFIN_TC_NO_PAIRS") != nullptr;
    const bool pairs = !no_pairs && m_tiles % 2 == 0 && sms >= 2;
    griffin_status st;
    if (pairs) {
        TcParams p2 = p;
        p2.m_tiles = m_tiles / 2;
        p2.tail_first = p.tail_first / 2;  // (a whole number of pairs: the plan cuts a multiple of m_tiles tiles... of an even count)
        st = launch_tc_pairs(gated ? TC_GATED : TC_WIDE, mx, mg, mu, p2, sms, stream);
    } else {
        st = gated ? launch_tc<TC_GATED, 128>(mx, mg, mu, p, sms, stream) : launch_tc<TC_WIDE, 128>(mx, mg, mu, p, sms, stream);
    }
    if (st == GRIFFIN_OK && p.tail_ks > 1) {
        void *args[] = {&p};
        if (launch_maybe_overlapped((const void *)dual_tail_finish_kernel, dim3((p.m_tiles * p.n_tiles - p.tail_first) * (TC_BM / 4)),
                                    dim3(128), 0, stream, true, args) != cudaSuccess)
            st = GRIFFIN_ERR_CUDA;
    }
    if (st == GRIFFIN_OK && after_ff1 != nullptr && cudaEventRecord(after_ff1, stream) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    if (st != GRIFFIN_OK || y == nullptr) return st;

    // Y = Z W_2^T + b_2
    int bn = 128, splits = 1;
    gemm2_plan(S, d, d_ff, &bn, &splits);
    CUtensorMap mz, md;
    if (!make_map(&mz, z, S, d_ff, TC_BM) || !make_map(&md, w->w_down, d, d_ff, bn)) return GRIFFIN_ERR_CUDA;
    TcParams q = {};
    q.S = S;
    q.n_total = d;
    q.K = d_ff;
    q.m_tiles = m_tiles;
    q.n_tiles = d / bn;
    q.bias0 = splits > 1 ? nullptr : static_cast<const __nv_bfloat16 *>(w->b_down);
    q.out = static_cast<__nv_bfloat16 *>(y);
    q.act = desc->act;
    q.ws = ws;
    q.splits = splits;
    q.part = splits > 1 ? ypart : nullptr;
    q.tail_ks = 1;
    gemm2_tail_plan(S, d, d_ff, &q.tail_first, &q.tail_ks);
    q.tail_part = ypart;
    if (q.tail_ks > 1) q.bias0 = static_cast<const __nv_bfloat16 *>(w->b_down);
    if (pairs && bn == 256) {
        CUtensorMap md2;  // the same matrix in boxes of 128 rows: each CTA of a pair stages half of a 256-wide tile
        if (!make_map(&md2, w->w_down, d, d_ff, 128)) return GRIFFIN_ERR_CUDA;
        TcParams q2 = q;
        q2.m_tiles = m_tiles / 2;
        q2.tail_first = q.tail_first / 2;
        st = launch_tc_pairs(TC_PLAIN, mz, md2, md2, q2, sms, stream);
    } else {
        st = bn == 256 ? launch_tc<TC_PLAIN, 256>(mz, md, md, q, sms, stream)
                       : launch_tc<TC_PLAIN, 128>(mz, md, md, q, sms, stream);
    }
    if (st == GRIFFIN_OK && q.tail_ks > 1) {
        void *args[] = {&q};
        // (not as an early, dependent launch: its waiting blocks would take the thread slots beside the GEMM's CTAs
        // that the statistic's kernels on the side stream are meant to run in -- measured, 4.6 us lost per call)
        if (launch_maybe_overlapped((const void *)plain_tail_finish_kernel, dim3((q.m_tiles * q.n_tiles - q.tail_first) * (TC_BM / 4)),
                                    dim3(128), 0, stream, false, args) != cudaSuccess)
            st = GRIFFIN_ERR_CUDA;
    }
    if (st != GRIFFIN_OK || splits == 1) return st;
    const size_t n_elems = (size_t)S * d;
    const float *part_in = ypart;
    const __nv_bfloat16 *bias = static_cast<const __nv_bfloat16 *>(w->b_down);
    __nv_bfloat16 *y_out = static_cast<__nv_bfloat16 *>(y);
    size_t n_el = n_elems;
    int n_total = d;
    void *args[] = {&part_in, &bias, &y_out, &splits, &n_el, &n_total};
    return launch_maybe_overlapped((const void *)splitk_reduce_kernel, dim3((unsigned)((n_elems / 4 + 255) / 256)), dim3(256), 0,
                                   stream, false, args) == cudaSuccess ? GRIFFIN_OK : GRIFFIN_ERR_CUDA;
}

}  // namespace griffin
