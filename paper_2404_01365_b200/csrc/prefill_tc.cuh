// Pieces shared by the two prompt-phase tensor-core kernels: one CTA per 128-token tile (prefill_tc.cu), and a
// pair of CTAs on a 256-token tile (prefill_tc2.cu).
#pragma once

#include "common.cuh"
#include "launch.h"
#include "prefill_tc.h"
#include "tc_common.cuh"

namespace griffin {

constexpr int TC_PLAIN = 0, TC_GATED = 1, TC_WIDE = 2;
// sigma with the fast division (2 ulp) for the epilogues: a warp there pays most of every dependent
// latency in full, and the IEEE division is a long chain (measured: 2 us of 142 on the bench shape).
__device__ __forceinline__ float sigma_fast_rt(int act, float t) {
    switch (act) {
        case GRIFFIN_ACT_SWIGLU: return __fdividef(t, 1.0f + __expf(-t));
        case GRIFFIN_ACT_GEGLU_TANH: {
            const float inner = 0.7978845608028654f * (t + 0.044715f * t * t * t);
            const float th = 1.0f - __fdividef(2.0f, __expf(2.0f * inner) + 1.0f);
            return 0.5f * t * (1.0f + th);
        }
        case GRIFFIN_ACT_GEGLU_ERF: return sigma<GRIFFIN_ACT_GEGLU_ERF>(t);
        default: return fmaxf(t, 0.0f);
    }
}

constexpr int TC_BM = 128;        // rows (tokens) per tile
constexpr int TC_BK = 64;         // K per stage: 64 bf16 = one 128-byte swizzle row
constexpr int TC_EPI_WARPS = 8;   // two per TMEM lane quarter
constexpr int TC_THREADS = 64 + 32 * TC_EPI_WARPS;
#ifndef GRIFFIN_TC_STAGES
#define GRIFFIN_TC_STAGES 4
#endif
constexpr int TC_STAGES = GRIFFIN_TC_STAGES;

struct TcParams {
    int S;            // rows of the left operand and of the output
    int n_total;      // columns of the output (d_ff for DUAL, d otherwise)
    int K;            // reduction length (d for DUAL, d_ff otherwise), multiple of 64
    int m_tiles, n_tiles;
    const __nv_bfloat16 *bias0, *bias1;  // DUAL: b_gate, b_up; otherwise b_down, unused (may be null)
    __nv_bfloat16 *out;                  // Z or Y, [S, n_total]
    __nv_bfloat16 *zlo;                  // DUAL: what Z lost when it was rounded to bf16, itself in bf16: z - bf16(z), [S, n_total]
    float *rowsq;                        // DUAL: [S, 2 n_tiles] partial sums of squares of the fp32 rows (two column halves per tile)
    int splits;                          // K splits (1 unless the plain GEMM has too few tiles)
    float *part;                         // splits > 1: fp32 partial outputs [splits, S, n_total]
    int act;
    void *ws;
    // Tiles 256 columns wide only: tiles from tail_first on are cut along K into tail_ks parts (tail_ks = 1:
    // none is), whose raw accumulators (fp32; gate | up in the first GEMM) go to tail_part [part][128 rows][256 columns]
    int tail_first, tail_ks;
    float *tail_part;
    int gated;  // first GEMM: 1 = gate | up tiles of 128 neurons, 0 = 256 neurons of W_1 (no gate)
};

// Work item -> (row block m, column block n, K blocks [kb0, kb1), index of the cut tile's part or -1).
// Uniform K splits (the down projection) number the items split-major; the cut tiles of the first GEMM
// follow the whole ones.
struct TcItem {
    int m, n, sp, kb0, kb1, part;
};
__device__ __forceinline__ TcItem tc_item(const TcParams &p, int item, int kb_total) {
    TcItem t;
    const int tiles = p.m_tiles * p.n_tiles;
    int tile = item, ks = p.splits;
    t.sp = 0;
    t.part = -1;
    if (p.tail_ks > 1) {
        ks = 1;
        if (item >= p.tail_first) {
            const int j = item - p.tail_first;
            ks = p.tail_ks;
            tile = p.tail_first + j / ks;
            t.sp = j - (j / ks) * ks;
            t.part = j;
        }
    } else if (ks > 1) {
        t.sp = item / tiles;
        tile = item - t.sp * tiles;
    }
    t.m = tile % p.m_tiles;  // tiles sharing weights are neighbours
    t.n = tile / p.m_tiles;
    t.kb0 = t.sp * kb_total / ks;
    t.kb1 = (t.sp + 1) * kb_total / ks;
    return t;
}

// Output staging of the epilogue warps.  A thread of an epilogue warp holds one ROW of the tile, so a
// store straight from its registers scatters every instruction over 32 rows, 16 bytes each; those
// requests queue behind the TMA loads on the SM's way to L2 and made the epilogue of a tile take
// 18-23 us.  Instead the warp passes its 32 rows, 64 bytes of each at a time, through a small buffer
// of its own in shared memory and writes them back so that an instruction covers 8 rows x 64
// contiguous bytes.
constexpr int TC_STG_PITCH = 80;                  // 64 data bytes + 16 of padding per staged row
constexpr int TC_STG_BYTES = 32 * TC_STG_PITCH;   // per epilogue warp
// v: this thread's 64 bytes of its row; g: global address of the block's first row at the wanted
// column; rows at and beyond rows_live are not written.
__device__ __forceinline__ void store_rows64(uint8_t *stg, const uint4 (&v)[4], void *g, size_t row_pitch_bytes,
                                             int rows_live, int lane) {
    uint4 *mine = reinterpret_cast<uint4 *>(stg + lane * TC_STG_PITCH);
#pragma unroll
    for (int i = 0; i < 4; ++i) mine[i] = v[i];
    __syncwarp();
    const int piece = lane & 3, r0 = lane >> 2;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int r = r0 + 8 * j;
        const uint4 t = *reinterpret_cast<const uint4 *>(stg + r * TC_STG_PITCH + piece * 16);
        if (r < rows_live) *reinterpret_cast<uint4 *>(static_cast<uint8_t *>(g) + (size_t)r * row_pitch_bytes + piece * 16) = t;
    }
    __syncwarp();
}
// 32 fp32 values of this thread's row (128 bytes) as two such passes.
__device__ __forceinline__ void store_rows_f32x32(uint8_t *stg, const float (&a)[32], float *g, size_t row_pitch_bytes,
                                                  int rows_live, int lane) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        uint4 v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            v[i] = make_uint4(__float_as_uint(a[16 * h + 4 * i]), __float_as_uint(a[16 * h + 4 * i + 1]),
                              __float_as_uint(a[16 * h + 4 * i + 2]), __float_as_uint(a[16 * h + 4 * i + 3]));
        store_rows64(stg, v, g + 16 * h, row_pitch_bytes, rows_live, lane);
    }
}

// The epilogue of one work item for one epilogue warp: its 32 rows (TMEM lane quarter wq) and its half of the
// tile's columns.  m, n: the tile; part: index of the cut tile's part (-1: the item is a whole tile or a uniform
// split sp); taddr: TMEM address of the accumulator stage at this warp's lanes; stg: the warp's staging buffer.
template <int KIND, int BN>
__device__ __forceinline__ void tc_epilogue_item(const TcParams &p, int m, int n, int sp, int part, uint32_t taddr,
                                                 uint8_t *stg, int wq, int half, int lane) {
    constexpr bool DUAL = KIND != TC_PLAIN;
    const int row_in_tile = wq * 32 + lane;  // one output row per thread
    const int row = m * TC_BM + row_in_tile;
    const bool live = row < p.S;
    const int row0 = m * TC_BM + wq * 32;  // first row of this warp's block of 32
    const int rows_live = p.S - row0;      // rows of the block that exist (may be <= 0 or > 32)
    if ((DUAL || BN == 256) && part >= 0) {
        // a part of a cut tile: the raw accumulators leave in fp32 (gate | up); the finishing
        // kernel adds the parts and does what the epilogue below does
        float *dst = p.tail_part + ((size_t)part * TC_BM + wq * 32) * 256;
#pragma unroll 1
        for (int c = half * 128; c < half * 128 + 128; c += 32) {
            float a[32];
            tmem_ld32(taddr + c, a);
            store_rows_f32x32(stg, a, dst + c, 256 * sizeof(float), 32, lane);
        }
    } else if (KIND == TC_WIDE) {
        // no gate: every one of the 256 accumulator columns is a neuron, Z = sigma(acc + b_1)
        float sq = 0.f;
#pragma unroll 1
        for (int c = half * 128; c < half * 128 + 128; c += 32) {
            float u[32];
            tmem_ld32(taddr + c, u);
            const int col = n * 256 + c;
            uint32_t packed[16], packed_lo[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                float u0 = u[i], u1 = u[i + 1];
                if (p.bias1) { u0 += __bfloat162float(p.bias1[col + i]); u1 += __bfloat162float(p.bias1[col + i + 1]); }
                const float z0 = sigma_fast_rt(p.act, u0), z1 = sigma_fast_rt(p.act, u1);
                sq = fmaf(z0, z0, sq);
                sq = fmaf(z1, z1, sq);
                const __nv_bfloat162 h = __floats2bfloat162_rn(z0, z1);
                packed[i >> 1] = *reinterpret_cast<const uint32_t *>(&h);
                const __nv_bfloat162 l = __floats2bfloat162_rn(z0 - __low2float(h), z1 - __high2float(h));
                packed_lo[i >> 1] = *reinterpret_cast<const uint32_t *>(&l);
            }
            {
                uint4 pk[4];
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    pk[v] = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
                store_rows64(stg, pk, p.out + (size_t)row0 * p.n_total + col, (size_t)p.n_total * 2, rows_live, lane);
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    pk[v] = make_uint4(packed_lo[4 * v], packed_lo[4 * v + 1], packed_lo[4 * v + 2], packed_lo[4 * v + 3]);
                store_rows64(stg, pk, p.zlo + (size_t)row0 * p.n_total + col, (size_t)p.n_total * 2, rows_live, lane);
            }
        }
        if (live) p.rowsq[(size_t)row * (2 * p.n_tiles) + 2 * n + half] = sq;
    } else if (DUAL) {
        float sq = 0.f;
#pragma unroll 1
        for (int c = half * 64; c < half * 64 + 64; c += 32) {
            float g[32], u[32];
            tmem_ld32x2(taddr + c, taddr + 128 + c, g, u);
            const int col = n * 128 + c;
            uint32_t packed[16], packed_lo[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                float g0 = g[i], g1 = g[i + 1], u0 = u[i], u1 = u[i + 1];
                if (p.bias0) { g0 += __bfloat162float(p.bias0[col + i]); g1 += __bfloat162float(p.bias0[col + i + 1]); }
                if (p.bias1) { u0 += __bfloat162float(p.bias1[col + i]); u1 += __bfloat162float(p.bias1[col + i + 1]); }
                const float z0 = sigma_fast_rt(p.act, g0) * u0, z1 = sigma_fast_rt(p.act, g1) * u1;
                sq = fmaf(z0, z0, sq);
                sq = fmaf(z1, z1, sq);
                const __nv_bfloat162 h = __floats2bfloat162_rn(z0, z1);
                packed[i >> 1] = *reinterpret_cast<const uint32_t *>(&h);
                const __nv_bfloat162 l = __floats2bfloat162_rn(z0 - __low2float(h), z1 - __high2float(h));
                packed_lo[i >> 1] = *reinterpret_cast<const uint32_t *>(&l);
            }
            {
                uint4 pk[4];
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    pk[v] = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
                store_rows64(stg, pk, p.out + (size_t)row0 * p.n_total + col, (size_t)p.n_total * 2, rows_live, lane);
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    pk[v] = make_uint4(packed_lo[4 * v], packed_lo[4 * v + 1], packed_lo[4 * v + 2], packed_lo[4 * v + 3]);
                store_rows64(stg, pk, p.zlo + (size_t)row0 * p.n_total + col, (size_t)p.n_total * 2, rows_live, lane);
            }
        }
        if (live) p.rowsq[(size_t)row * (2 * p.n_tiles) + 2 * n + half] = sq;
    } else {
#pragma unroll 1
        for (int c = half * (BN / 2); c < half * (BN / 2) + BN / 2; c += 32) {
            float a[32];
            tmem_ld32(taddr + c, a);
            const int col = n * BN + c;
            if (p.splits > 1) {  // partial sums leave in fp32; bias and rounding happen in the reduction
                store_rows_f32x32(stg, a, p.part + ((size_t)sp * p.S + row0) * p.n_total + col,
                                  (size_t)p.n_total * 4, rows_live, lane);
                continue;
            }
            uint32_t packed[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                float y0 = a[i], y1 = a[i + 1];
                if (p.bias0) { y0 += __bfloat162float(p.bias0[col + i]); y1 += __bfloat162float(p.bias0[col + i + 1]); }
                const __nv_bfloat162 h = __floats2bfloat162_rn(y0, y1);
                packed[i >> 1] = *reinterpret_cast<const uint32_t *>(&h);
            }
            {
                uint4 pk[4];
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    pk[v] = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
                store_rows64(stg, pk, p.out + (size_t)row0 * p.n_total + col, (size_t)p.n_total * 2, rows_live, lane);
            }
        }
    }
}

// The same GEMMs with pairs of CTAs on tiles of 256 tokens (prefill_tc2.cu).  kind: TC_PLAIN (256-wide tiles),
// TC_GATED or TC_WIDE; p as for the one-CTA kernels except that m_tiles and tail_first count PAIRS of
// 128-token tiles; the weight maps have boxes of 128 rows.
griffin_status launch_tc_pairs(int kind, const CUtensorMap &ma, const CUtensorMap &mb0, const CUtensorMap &mb1,
                               const TcParams &p, int sms, cudaStream_t stream);

}  // namespace griffin
