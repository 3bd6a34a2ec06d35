// Prompt-phase FF and selection statistic (Section 4.2, Eqs. 1, 3 and 6 of the GRIFFIN paper).
//
//   1. Z = sigma(X W_g^T + b_g) * (X W_1^T + b_1)          [S, d_ff]  (Eq. 3), stored in the
//      storage dtype as the operand of step 2 and, for bf16 storage, once more in fp32
//      for the statistic (a bf16-rounded Z would move s by up to 2^-8, more than the
//      margin by which neighbouring neurons differ); the same kernel leaves, per token
//      and per column tile, the partial sum of squares of the fp32 row   (for ||Z_i||^2)
//   2. Y = Z W_2^T + b_2                                    [S, d]     (Eq. 1)
//   3. inv_i = 1 / ||Z_i||_2^2  (0 for an all-zero row)
//   4. colpart[chunk, j] = sum over the chunk's tokens of Z_ij^2 * inv_i
//   5. s_j = sqrt(sum over chunks of colpart[chunk, j])                 (Eq. 6)
//
// The row normaliser spans every column tile, so the column sums cannot finish inside
// step 1: steps 3-5 re-read Z (fp32 storage), or Z and the bf16 residual that step 1 wrote beside it (bf16
// storage; both mostly still sit in L2).  All partial sums are kept
// and added in a fixed order, so s is deterministic.
//
// This file holds the fp32-FMA (SIMT) matrix kernels, which serve the fp32 storage type
// and any shape the tensor-core path does not take, plus steps 3-5 and the dispatcher.
#include <stdlib.h>

#include <type_traits>

#include "common.cuh"
#include "launch.h"
#include "prefill_tc.h"

namespace griffin {

constexpr int PF_BM = 64, PF_BN = 64, PF_BK = 16, PF_THREADS = 256, PF_PAD = 4;
constexpr int PF_ROW_CHUNK = 64;  // tokens per partial column sum

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

PrefillScratch prefill_scratch(const griffin_ff_desc *desc, int S) {
    PrefillScratch ps;
    const size_t esz = desc->dtype == GRIFFIN_DT_F32 ? 4 : 2;
    ps.n_col_tiles = (desc->d_ff + PF_BN - 1) / PF_BN;  // the narrowest column tile any path uses
    ps.n_row_chunks = (S + PF_ROW_CHUNK - 1) / PF_ROW_CHUNK;
    size_t off = 0;
    ps.z_off = off;
    off = align_up(off + (size_t)S * desc->d_ff * esz, 256);
    ps.zf_off = off;
    if (desc->dtype != GRIFFIN_DT_F32) off = align_up(off + (size_t)S * desc->d_ff * 2, 256);  // the bf16 residual of Z
    ps.rowsq_off = off;
    off = align_up(off + (size_t)S * ps.n_col_tiles * sizeof(float), 256);
    ps.inv_off = off;
    off = align_up(off + (size_t)S * sizeof(float), 256);
    ps.colpart_off = off;
    off = align_up(off + (size_t)ps.n_row_chunks * desc->d_ff * sizeof(float), 256);
    ps.ypart_off = off;  // fp32 partial outputs of a K-split down projection (bf16 tensor-core path)
    if (desc->dtype != GRIFFIN_DT_F32) {
        int bn = 0, splits = 1;
        gemm2_plan(S, desc->d, desc->d_ff, &bn, &splits);
        size_t need = splits > 1 ? (size_t)splits * S * desc->d * sizeof(float) : 0;
        const size_t tail = gemm1_tail_bytes(S, desc->d, gemm1_col_tiles(desc));  // (used up before the down projection starts)
        if (tail > need) need = tail;
        const size_t tail2 = gemm2_tail_bytes(S, desc->d, desc->d_ff);
        if (tail2 > need) need = tail2;
        if (need > 0) off = align_up(off + need, 256);
    }
    ps.total = off;
    return ps;
}

// Loads a [64 x 16] tile of a row-major [rows, K] matrix (K contiguous) into shared memory
// as fp32, transposed to [k][row].  256 threads; rows/K beyond the matrix read as zero.
template <typename T>
__device__ __forceinline__ void load_tile_t(const T *__restrict__ src, int ld, int rows, int K, int r0, int k0,
                                            float (*dst)[PF_BM + PF_PAD], int tid) {
    constexpr int VEC = Elem<T>::VEC;
    constexpr int VPR = PF_BK / VEC;  // vectors per tile row
    if (tid < PF_BM * VPR) {
        const int r = tid / VPR, kv = tid - r * VPR;
        const int row = r0 + r, kk = k0 + kv * VEC;
        float f[VEC];
        if (row < rows && kk < K) {
            Elem<T>::unpack(*reinterpret_cast<const uint4 *>(src + (size_t)row * ld + kk), f);
        } else {
#pragma unroll
            for (int e = 0; e < VEC; ++e) f[e] = 0.f;
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e) dst[kv * VEC + e][r] = f[e];
    }
}

// Step 1 (SIMT): one CTA = 64 tokens x 64 neurons.  GATED = false: the block has no gate (Eq. 2),
// Z = sigma(X W_1^T + b_1), and w_gate / b_gate are not touched.
template <typename T, bool GATED>
__global__ void __launch_bounds__(PF_THREADS) ff1_simt_kernel(const T *__restrict__ x, const T *__restrict__ w_gate,
                                                              const T *__restrict__ w_up, const T *__restrict__ b_gate,
                                                              const T *__restrict__ b_up, T *__restrict__ z,
                                                              T *__restrict__ zlo,  // bf16 storage: z - bf16(z); else null
                                                              float *__restrict__ rowsq, int S, int d, int d_ff,
                                                              int n_col_tiles, int act) {
    __shared__ float xs[PF_BK][PF_BM + PF_PAD], gs[PF_BK][PF_BN + PF_PAD], us[PF_BK][PF_BN + PF_PAD];
    __shared__ float red[PF_BM][17];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * PF_BM, n0 = blockIdx.x * PF_BN;
    float ga[4][4] = {}, ua[4][4] = {};
    for (int k0 = 0; k0 < d; k0 += PF_BK) {
        load_tile_t<T>(x, d, S, d, m0, k0, xs, tid);
        if (GATED) load_tile_t<T>(w_gate, d, d_ff, d, n0, k0, gs, tid);
        load_tile_t<T>(w_up, d, d_ff, d, n0, k0, us, tid);
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < PF_BK; ++kk) {
            const float4 a = *reinterpret_cast<const float4 *>(&xs[kk][ty * 4]);
            const float4 u = *reinterpret_cast<const float4 *>(&us[kk][tx * 4]);
            const float4 g = GATED ? *reinterpret_cast<const float4 *>(&gs[kk][tx * 4]) : u;
            const float av[4] = {a.x, a.y, a.z, a.w}, gv[4] = {g.x, g.y, g.z, g.w}, uv[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (GATED) ga[i][j] = fmaf(av[i], gv[j], ga[i][j]);
                    ua[i][j] = fmaf(av[i], uv[j], ua[i][j]);
                }
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = m0 + ty * 4 + i;
        float sq = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int col = n0 + tx * 4 + j;
            if (row < S && col < d_ff) {
                float g = ga[i][j], u = ua[i][j];
                if (GATED && b_gate) g += Elem<T>::to_float(b_gate[col]);
                if (b_up) u += Elem<T>::to_float(b_up[col]);
                const float zv = GATED ? sigma_rt(act, g) * u : sigma_rt(act, u);
                const T zh = Elem<T>::from_float(zv);
                z[(size_t)row * d_ff + col] = zh;
                if (zlo) zlo[(size_t)row * d_ff + col] = Elem<T>::from_float(zv - Elem<T>::to_float(zh));
                sq = fmaf(zv, zv, sq);
            }
        }
        red[ty * 4 + i][tx] = sq;
    }
    __syncthreads();
    if (tid < PF_BM && m0 + tid < S) {
        float sq = 0.f;
#pragma unroll
        for (int t = 0; t < 16; ++t) sq += red[tid][t];
        rowsq[(size_t)(m0 + tid) * n_col_tiles + blockIdx.x] = sq;
    }
}

// Step 2 (SIMT): Y = Z W_2^T + b_2, one CTA = 64 tokens x 64 outputs.
template <typename T>
__global__ void __launch_bounds__(PF_THREADS) ff2_simt_kernel(const T *__restrict__ z, const T *__restrict__ w_down,
                                                              const T *__restrict__ b_down, T *__restrict__ y, int S,
                                                              int d, int d_ff) {
    __shared__ float zs[PF_BK][PF_BM + PF_PAD], ws[PF_BK][PF_BN + PF_PAD];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * PF_BM, n0 = blockIdx.x * PF_BN;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < d_ff; k0 += PF_BK) {
        load_tile_t<T>(z, d_ff, S, d_ff, m0, k0, zs, tid);
        load_tile_t<T>(w_down, d_ff, d, d_ff, n0, k0, ws, tid);
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < PF_BK; ++kk) {
            const float4 a = *reinterpret_cast<const float4 *>(&zs[kk][ty * 4]);
            const float4 b = *reinterpret_cast<const float4 *>(&ws[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = m0 + ty * 4 + i;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int col = n0 + tx * 4 + j;
            if (row < S && col < d) {
                float v = acc[i][j];
                if (b_down) v += Elem<T>::to_float(b_down[col]);
                y[(size_t)row * d + col] = Elem<T>::from_float(v);
            }
        }
    }
}

// Step 3: one warp per token.
__global__ void row_inv_kernel(const float *__restrict__ rowsq, int S, int n_col_tiles, float *__restrict__ inv) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= S) return;
    float sq = 0.f;
    for (int t = lane; t < n_col_tiles; t += 32) sq += rowsq[(size_t)row * n_col_tiles + t];
    sq = warp_sum(sq);
    if (lane == 0) inv[row] = sq > 0.f ? 1.0f / sq : 0.f;
}

// Step 4: a CTA owns 128 neighbouring columns of Z over one chunk of tokens; each of its 8 warps takes
// every 8th token of the chunk (four columns per lane, all loads of a warp in flight together) and
// the warps' sums meet in shared memory in a fixed order.  Z comes in fp32 (fp32 storage: zlo null) or
// as two bf16 numbers per entry, z = zhi + zlo (bf16 storage: the Z that the down projection reads, and
// what its rounding lost; together 16 mantissa bits, 4e-6 relative).
__global__ void __launch_bounds__(256) col_partial_kernel(const void *__restrict__ z, const __nv_bfloat16 *__restrict__ zlo,
                                                          const float *__restrict__ inv, int S, int d_ff,
                                                          float *__restrict__ colpart) {
    __shared__ float4 red[8][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int col = (blockIdx.x * 32 + lane) * 4;
    const int r0 = blockIdx.y * PF_ROW_CHUNK, r1 = min(S, r0 + PF_ROW_CHUNK);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (col < d_ff) {
#pragma unroll
        for (int i = 0; i < PF_ROW_CHUNK / 8; ++i) {
            const int r = r0 + warp + 8 * i;
            if (r < r1) {
                float4 f;
                if (zlo == nullptr) {
                    f = *reinterpret_cast<const float4 *>(static_cast<const float *>(z) + (size_t)r * d_ff + col);
                } else {
                    const uint2 h = *reinterpret_cast<const uint2 *>(static_cast<const __nv_bfloat16 *>(z) + (size_t)r * d_ff + col);
                    const uint2 l = *reinterpret_cast<const uint2 *>(zlo + (size_t)r * d_ff + col);
                    f.x = __uint_as_float(h.x << 16) + __uint_as_float(l.x << 16);
                    f.y = __uint_as_float(h.x & 0xffff0000u) + __uint_as_float(l.x & 0xffff0000u);
                    f.z = __uint_as_float(h.y << 16) + __uint_as_float(l.y << 16);
                    f.w = __uint_as_float(h.y & 0xffff0000u) + __uint_as_float(l.y & 0xffff0000u);
                }
                const float w = __ldg(inv + r);
                acc.x = fmaf(f.x * f.x, w, acc.x);
                acc.y = fmaf(f.y * f.y, w, acc.y);
                acc.z = fmaf(f.z * f.z, w, acc.z);
                acc.w = fmaf(f.w * f.w, w, acc.w);
            }
        }
    }
    red[warp][lane] = acc;
    __syncthreads();
    if (warp == 0 && col < d_ff) {
        float4 t = red[0][lane];
#pragma unroll
        for (int w = 1; w < 8; ++w) {
            t.x += red[w][lane].x; t.y += red[w][lane].y; t.z += red[w][lane].z; t.w += red[w][lane].w;
        }
        *reinterpret_cast<float4 *>(colpart + (size_t)blockIdx.y * d_ff + col) = t;
    }
}

// Step 5.
// sumsq (may be NULL): running sum of squares over the pieces of a prompt that is fed piece by
// piece (s_j^2 is a sum over tokens, Eq. 6); `first` starts it afresh.  score may then be NULL.
__global__ void score_finish_kernel(const float *__restrict__ colpart, int n_row_chunks, int d_ff,
                                    float *__restrict__ score, float *__restrict__ sumsq, int first) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d_ff) return;
    float acc = 0.f;
    for (int c = 0; c < n_row_chunks; ++c) acc += colpart[(size_t)c * d_ff + j];
    if (sumsq != nullptr) {
        if (!first) acc += sumsq[j];
        sumsq[j] = acc;
    }
    if (score != nullptr) score[j] = sqrtf(acc);
}

// The statistic only needs Z, the down projection only Z as well: with the tensor-core path the
// statistic kernels run on a stream of the library's own beside the second GEMM (whose
// persistent CTAs leave room for them on every SM) and join the caller's stream at the end.
// One lane per host thread and device, created at first use and kept.  With the environment
// variable GRIFFIN_NO_SIDE_STREAM set there is none: everything stays on the caller's stream.
struct SideLane {
    cudaStream_t stream;
    cudaEvent_t fork, join;
};
static SideLane *side_lane_of_current_device() {
    constexpr int MAX_DEV = 64;
    static thread_local SideLane lanes[MAX_DEV];
    static thread_local int state[MAX_DEV];  // 0 untried, 1 ready, -1 unavailable
    static const bool disabled = getenv("GRIFFIN_NO_SIDE_STREAM") != nullptr;
    if (disabled) return nullptr;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEV) return nullptr;
    if (state[dev] == 0) {
        SideLane &l = lanes[dev];
        state[dev] = (cudaStreamCreateWithFlags(&l.stream, cudaStreamNonBlocking) == cudaSuccess &&
                      cudaEventCreateWithFlags(&l.fork, cudaEventDisableTiming) == cudaSuccess &&
                      cudaEventCreateWithFlags(&l.join, cudaEventDisableTiming) == cudaSuccess)
                         ? 1
                         : -1;
    }
    return state[dev] == 1 ? &lanes[dev] : nullptr;
}

template <typename T>
static griffin_status prefill_typed(const griffin_ff_desc *desc, const griffin_ff_weights *w, const void *x, int S,
                                    void *y, float *score, float *sumsq, int first, uint8_t *scratch, void *ws,
                                    cudaStream_t stream) {
    const int d = desc->d, d_ff = desc->d_ff;
    const PrefillScratch ps = prefill_scratch(desc, S);
    T *z = reinterpret_cast<T *>(scratch + ps.z_off);
    constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
    T *zlo = kBf16 ? reinterpret_cast<T *>(scratch + ps.zf_off) : nullptr;
    float *rowsq = reinterpret_cast<float *>(scratch + ps.rowsq_off);
    float *inv = reinterpret_cast<float *>(scratch + ps.inv_off);
    float *colpart = reinterpret_cast<float *>(scratch + ps.colpart_off);

    int n_col_tiles = 0;
    bool ff2_done = false;
    bool use_tc = false;
    if constexpr (kBf16) use_tc = prefill_tc_supported(desc, S);
    cudaStream_t stat_stream = stream;  // where the statistic kernels go
    SideLane *lane = nullptr;
    if (use_tc) {
        if constexpr (kBf16) {
            if (y != nullptr) lane = side_lane_of_current_device();  // (measured: a gain at every prompt length, 9 % at S = 512)
            griffin_status st = launch_prefill_tc(desc, w, x, S, y, z, zlo, rowsq, reinterpret_cast<float *>(scratch + ps.ypart_off),
                                                  &n_col_tiles, ws, stream, lane ? lane->fork : nullptr);
            if (st != GRIFFIN_OK) return st;
            if (lane != nullptr) {
                if (cudaStreamWaitEvent(lane->stream, lane->fork, 0) != cudaSuccess) return GRIFFIN_ERR_CUDA;
                stat_stream = lane->stream;
            }
        }
        ff2_done = true;
    } else {
        n_col_tiles = (d_ff + PF_BN - 1) / PF_BN;
        const dim3 g1(n_col_tiles, (S + PF_BM - 1) / PF_BM);
        if (act_gated(desc->act)) {
            ff1_simt_kernel<T, true><<<g1, PF_THREADS, 0, stream>>>(
                static_cast<const T *>(x), static_cast<const T *>(w->w_gate), static_cast<const T *>(w->w_up),
                static_cast<const T *>(w->b_gate), static_cast<const T *>(w->b_up), z, zlo, rowsq, S, d, d_ff,
                n_col_tiles, desc->act);
        } else {
            ff1_simt_kernel<T, false><<<g1, PF_THREADS, 0, stream>>>(
                static_cast<const T *>(x), nullptr, static_cast<const T *>(w->w_up), nullptr,
                static_cast<const T *>(w->b_up), z, zlo, rowsq, S, d, d_ff, n_col_tiles, act_sigma(desc->act));
        }
        count_launches(1);
        if (cudaGetLastError() != cudaSuccess) return GRIFFIN_ERR_CUDA;
    }
    if (!ff2_done && y != nullptr) {
        const dim3 g2((d + PF_BN - 1) / PF_BN, (S + PF_BM - 1) / PF_BM);
        ff2_simt_kernel<T><<<g2, PF_THREADS, 0, stream>>>(z, static_cast<const T *>(w->w_down),
                                                          static_cast<const T *>(w->b_down), static_cast<T *>(y), S, d,
                                                          d_ff);
        count_launches(1);
        if (cudaGetLastError() != cudaSuccess) return GRIFFIN_ERR_CUDA;
    }
    griffin_status st = GRIFFIN_OK;
    row_inv_kernel<<<(S + 7) / 8, 256, 0, stat_stream>>>(rowsq, S, n_col_tiles, inv);
    count_launches(1);
    if (cudaGetLastError() != cudaSuccess) st = GRIFFIN_ERR_CUDA;
    const dim3 g4((d_ff + 127) / 128, ps.n_row_chunks);
    if (st == GRIFFIN_OK) {
        col_partial_kernel<<<g4, 256, 0, stat_stream>>>(z, reinterpret_cast<const __nv_bfloat16 *>(zlo), inv, S, d_ff, colpart);
        count_launches(1);
        if (cudaGetLastError() != cudaSuccess) st = GRIFFIN_ERR_CUDA;
    }
    if (st == GRIFFIN_OK) {
        score_finish_kernel<<<(d_ff + 255) / 256, 256, 0, stat_stream>>>(colpart, ps.n_row_chunks, d_ff, score, sumsq,
                                                                                 first);
        count_launches(1);
        if (cudaGetLastError() != cudaSuccess) st = GRIFFIN_ERR_CUDA;
    }
    // whatever went to the side stream rejoins the caller's stream, also when a launch above failed
    if (lane != nullptr &&
        (cudaEventRecord(lane->join, lane->stream) != cudaSuccess || cudaStreamWaitEvent(stream, lane->join, 0) != cudaSuccess))
        return GRIFFIN_ERR_CUDA;
    return st;
}

griffin_status launch_prefill_score(const griffin_ff_desc *desc, const griffin_ff_weights *w, const void *x, int S,
                                    void *y, float *score, float *sumsq, int first, uint8_t *scratch, void *ws,
                                    cudaStream_t stream) {
    if (desc->dtype == GRIFFIN_DT_F32)
        return prefill_typed<float>(desc, w, x, S, y, score, sumsq, first, scratch, ws, stream);
    return prefill_typed<__nv_bfloat16>(desc, w, x, S, y, score, sumsq, first, scratch, ws, stream);
}

}  // namespace griffin
