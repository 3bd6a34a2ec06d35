// Expert compaction (Section 4.2 of the GRIFFIN paper): W_g_hat = W_g[E, :],
// W_1_hat = W_1[E, :], W_2_hat = W_2[:, E], plus the matching bias entries.  Bit copies, so
// elements are moved as raw 16- or 32-bit words.
//
// One launch per call: the CTAs of a grid are split between the three parts below (columns first:
// its CTAs carry the most work each), so that no part waits for another's tail or launch.
//
//   rows part       16-byte vector copy of the selected rows of W_g and W_1; consecutive
//                   threads move consecutive vectors of one row (coalesced both ways).
//   columns part    W_2 is [d, d_ff] row-major, so selecting columns is a gather inside
//                   each row.  One CTA takes four rows; a thread reads 16 bytes' worth of
//                   output columns of E once, picks those elements from each of the four
//                   rows (E is usually ascending and dense, so neighbouring threads hit
//                   neighbouring sectors) and writes one 16-byte vector per row.  Padding
//                   columns k..ldk are written as zeros.  At the usual keep ratios every
//                   32-byte sector of a row holds a selected column, so all of W_2 is read.
//                   (Tried and dropped, measured: whole rows brought into shared memory by bulk
//                   copies, the columns picked there and the output row sent out by a bulk
//                   store -- 68 us against 60 us on the Llama-2-7B shape, 198 against 100 on the
//                   Gemma shape: one row at a time per CTA leaves too little in flight.)
//   transposing     the same W_2_hat from a NEURON-MAJOR source (the transpose of W_2, [d_ff, d], as the
//     part          index-direct decode call holds it): the selected rows are contiguous, so only the k
//                   selected rows are read -- half the bytes at keep 0.5 -- and turned through a
//                   shared-memory tile of 64 experts x 128 columns into rows of W_2_hat.
#include "common.cuh"
#include "launch.h"

namespace griffin {

constexpr int CP_THREADS = 256;
#ifndef GRIFFIN_CP_MINB
#define GRIFFIN_CP_MINB 6          // CTAs per SM the kernel is compiled for (measured best: 6, half of them turning tiles)
#endif
#ifndef GRIFFIN_CP_SHARE_PCT
#define GRIFFIN_CP_SHARE_PCT 50    // share of the resident CTAs that turn tiles when the source is neuron-major
#endif
constexpr int CP_ROWS_PER_CTA = 4;

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4 *p, const uint4 &v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// dst_g[jj, :] = src_g[idx[jj], :], dst_u likewise; nv = 16-byte vectors per row.  n_mats = 1: only
// the first pair of pointers is used (a block without a gate has W_1 alone).
// Block `bid` of `nblocks` that share the work.
__device__ __forceinline__ void compact_rows_part(const uint4 *__restrict__ src_g, const uint4 *__restrict__ src_u,
                                                  uint4 *__restrict__ dst_g, uint4 *__restrict__ dst_u,
                                                  const int32_t *__restrict__ idx, int k, int d_ff, int nv, int n_mats,
                                                  void *ws, int bid, int nblocks) {
    const long long total = (long long)n_mats * k * nv;
    const long long stride = (long long)nblocks * CP_THREADS;
    constexpr int U = 4;
    for (long long v0 = (long long)bid * CP_THREADS + threadIdx.x; v0 < total; v0 += stride * U) {
        uint4 val[U];
        uint4 *dst[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long v = v0 + u * stride;
            dst[u] = nullptr;
            val[u] = make_uint4(0, 0, 0, 0);
            if (v < total) {
                const int row = (int)(v / nv);
                const int col = (int)(v - (long long)row * nv);
                const int m = row >= k;
                const int jj = m ? row - k : row;
                const int e = idx[jj];
                dst[u] = (m ? dst_u : dst_g) + (size_t)jj * nv + col;
                if (e >= 0 && e < d_ff)
                    val[u] = ld_stream((m ? src_u : src_g) + (size_t)e * nv + col);
                else
                    raise_status(ws, DEV_STATUS_BAD_INDEX, 10);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (dst[u]) st_stream(dst[u], val[u]);
    }
}

template <typename U>
__device__ __forceinline__ void compact_bias_part(const U *__restrict__ src_g, const U *__restrict__ src_u,
                                                  U *__restrict__ dst_g, U *__restrict__ dst_u,
                                                  const int32_t *__restrict__ idx, int k, int d_ff, int bid) {
    const int jj = bid * CP_THREADS + threadIdx.x;
    if (jj >= k) return;
    const int e = idx[jj];
    const bool ok = e >= 0 && e < d_ff;
    if (src_g && dst_g) dst_g[jj] = ok ? src_g[e] : (U)0;
    if (src_u && dst_u) dst_u[jj] = ok ? src_u[e] : (U)0;
}

// dst[c, jj] = src[c, idx[jj]] for jj < k, 0 for k <= jj < ldk.  Block `bid` takes rows 4 bid .. 4 bid + 3.
template <typename U>
__device__ __forceinline__ void compact_cols_part(const U *__restrict__ src, U *__restrict__ dst,
                                                  const int32_t *__restrict__ idx, int d, int d_ff, int k, int ldk,
                                                  void *ws, int bid) {
    constexpr int VEC = 16 / (int)sizeof(U);
    const int c0 = bid * CP_ROWS_PER_CTA;
    const int nvec = ldk / VEC;
    for (int v = threadIdx.x; v < nvec; v += CP_THREADS) {
        int e[VEC];
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            const int jj = v * VEC + i;
            e[i] = jj < k ? idx[jj] : -1;
            if (jj < k && (e[i] < 0 || e[i] >= d_ff)) {
                e[i] = -1;
                raise_status(ws, DEV_STATUS_BAD_INDEX, 11);
            }
        }
#pragma unroll
        for (int r = 0; r < CP_ROWS_PER_CTA; ++r) {
            const int c = c0 + r;
            if (c < d) {
                const U *row = src + (size_t)c * d_ff;
                union {
                    uint4 u;
                    U t[VEC];
                } pack;
                pack.u = make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int i = 0; i < VEC; ++i)
                    if (e[i] >= 0) pack.t[i] = row[e[i]];
                st_stream(reinterpret_cast<uint4 *>(dst + (size_t)c * ldk) + v, pack.u);
            }
        }
    }
}

// ---- transposing part: W_2_hat [d, ldk] from the neuron-major W_2^T [d_ff, d] ---------------------------
constexpr int TP_J = 64;    // experts per tile
constexpr int TP_C = 128;   // columns of W_2^T (= rows of W_2_hat) per tile
// Tile (jt, ct): dst[ct*128 + c, jt*64 + j] = src[idx[jt*64 + j], ct*128 + c]; padding columns k..ldk zero.
template <typename U>
__device__ __forceinline__ void compact_transpose_part(const U *__restrict__ src, U *__restrict__ dst,
                                                       const int32_t *__restrict__ idx, int d, int d_ff, int k, int ldk,
                                                       void *ws, int bid, int nblocks, uint8_t *smem) {
    constexpr int VEC = 16 / (int)sizeof(U);       // elements per 16 bytes
    constexpr int PITCH = TP_C + 4 / (int)sizeof(U);  // one 32-bit word of padding per tile row
    U *tile = reinterpret_cast<U *>(smem);                                          // [TP_J][PITCH]
    int *e_tile = reinterpret_cast<int *>(smem + TP_J * PITCH * sizeof(U));          // [TP_J]
    const int tid = threadIdx.x;
    const int n_jt = (ldk + TP_J - 1) / TP_J, n_ct = (d + TP_C - 1) / TP_C;
    for (int t = bid; t < n_jt * n_ct; t += nblocks) {
        const int jt = t / n_ct, ct = t - jt * n_ct;  // (consecutive CTAs share the expert rows' neighbourhood)
        const int j0 = jt * TP_J, c0 = ct * TP_C;
        __syncthreads();  // the previous tile has been written out
        if (tid < TP_J) {
            int e = -1;
            if (j0 + tid < k) {
                e = idx[j0 + tid];
                if (e < 0 || e >= d_ff) {
                    e = -1;
                    raise_status(ws, DEV_STATUS_BAD_INDEX, 13);
                }
            }
            e_tile[tid] = e;
        }
        __syncthreads();
        // read: TP_J row segments of TP_C elements, 16 bytes per thread and step
        constexpr int UPR = TP_C / VEC;  // 16-byte units per row segment
        for (int v = tid; v < TP_J * UPR; v += CP_THREADS) {
            const int r = v / UPR, u = v - r * UPR;
            const int e = e_tile[r];
            uint4 val = make_uint4(0, 0, 0, 0);
            if (e >= 0 && c0 + u * VEC < d) val = ld_stream(reinterpret_cast<const uint4 *>(src + (size_t)e * d + c0) + u);
            uint32_t *w = reinterpret_cast<uint32_t *>(tile + r * PITCH + u * VEC);  // (rows are 4-byte aligned)
            w[0] = val.x; w[1] = val.y; w[2] = val.z; w[3] = val.w;
        }
        __syncthreads();
        // write: for every column c of the tile, TP_J / VEC units of 16 bytes; 8 lanes cover one output row's 128 bytes
        constexpr int UPC = TP_J / VEC;
        for (int v = tid; v < TP_C * UPC; v += CP_THREADS) {
            const int c = v / UPC, u = v - c * UPC;
            const int jj = j0 + u * VEC;
            if (c0 + c < d && jj < ldk) {
                union {
                    uint4 q;
                    U t[VEC];
                } pack;
#pragma unroll
                for (int i = 0; i < VEC; ++i) pack.t[i] = tile[(u * VEC + i) * PITCH + c];
                st_stream(reinterpret_cast<uint4 *>(dst + (size_t)(c0 + c) * ldk + jj), pack.q);
            }
        }
    }
}

struct CompactArgs {
    const void *src_g, *src_u, *src_d, *src_bg, *src_bu;
    void *dst_g, *dst_u, *dst_d, *dst_bg, *dst_bu;
    const int32_t *idx;
    void *ws;
    int d, d_ff, k, ldk, nv, n_mats;
    int cols_mode;  // how W_2_hat is made: COLS_GLOBAL from the row-major W_2, COLS_TRANSPOSE from W_2^T
    int cols_blocks, rows_blocks;  // CTAs [0, cols_blocks) make W_2_hat, the next rows_blocks copy rows, the rest biases
};
constexpr int COLS_GLOBAL = 0, COLS_TRANSPOSE = 2;

template <typename U>
__global__ void __launch_bounds__(CP_THREADS, GRIFFIN_CP_MINB) compact_kernel(const __grid_constant__ CompactArgs a) {
    extern __shared__ __align__(128) uint8_t cp_smem[];
    const int bid = blockIdx.x;
    if (bid < a.cols_blocks) {
        if (a.cols_mode == COLS_TRANSPOSE)
            compact_transpose_part<U>(static_cast<const U *>(a.src_d), static_cast<U *>(a.dst_d), a.idx, a.d, a.d_ff, a.k,
                                      a.ldk, a.ws, bid, a.cols_blocks, cp_smem);
        else
            compact_cols_part<U>(static_cast<const U *>(a.src_d), static_cast<U *>(a.dst_d), a.idx, a.d, a.d_ff, a.k, a.ldk,
                                 a.ws, bid);
    } else if (bid < a.cols_blocks + a.rows_blocks) {
        compact_rows_part(static_cast<const uint4 *>(a.src_g), static_cast<const uint4 *>(a.src_u),
                          static_cast<uint4 *>(a.dst_g), static_cast<uint4 *>(a.dst_u), a.idx, a.k, a.d_ff, a.nv, a.n_mats,
                          a.ws, bid - a.cols_blocks, a.rows_blocks);
    } else {
        compact_bias_part<U>(static_cast<const U *>(a.src_bg), static_cast<const U *>(a.src_bu),
                             static_cast<U *>(a.dst_bg), static_cast<U *>(a.dst_bu), a.idx, a.k, a.d_ff,
                             bid - a.cols_blocks - a.rows_blocks);
    }
}

// w_down: the row-major W_2 [d, d_ff], or (down_transposed) its transpose [d_ff, d].
template <typename U>
static griffin_status compact_typed(const griffin_ff_desc *desc, const void *w_gate, const void *w_up, const void *w_down,
                                    bool down_transposed, const void *b_gate, const void *b_up, const int32_t *idx,
                                    const griffin_ff_compact *out, void *ws, cudaStream_t stream) {
    const int d = desc->d, d_ff = desc->d_ff, k = out->k, ldk = out->ldk;
    const int nv = d * (int)sizeof(U) / 16;
    const int sms = device_sm_count();
    if (sms <= 0) return GRIFFIN_ERR_CUDA;
    const bool gated = w_gate != nullptr;  // (a block without a gate has W_1 alone, Eq. 2)
    CompactArgs a = {};
    a.src_g = gated ? w_gate : w_up;
    a.src_u = w_up;
    a.dst_g = gated ? out->w_gate_c : out->w_up_c;
    a.dst_u = out->w_up_c;
    a.src_d = w_down;
    a.dst_d = out->w_down_c;
    a.src_bg = b_gate;
    a.src_bu = b_up;
    a.dst_bg = out->b_gate_c;
    a.dst_bu = out->b_up_c;
    a.idx = idx;
    a.ws = ws;
    a.d = d;
    a.d_ff = d_ff;
    a.k = k;
    a.ldk = ldk;
    a.nv = nv;
    a.n_mats = gated ? 2 : 1;
    size_t smem = 0;
    int per_sm = 8;  // CTAs of 256 threads that an SM holds
    const long long want = ((gated ? 2ll : 1ll) * k * nv + CP_THREADS * 4 - 1) / (CP_THREADS * 4);
    if (down_transposed) {
        a.cols_mode = COLS_TRANSPOSE;
        smem = (size_t)TP_J * (TP_C + 4 / sizeof(U)) * sizeof(U) + TP_J * sizeof(int);  // the tile and its experts
        // the CTAs that turn tiles and those that copy rows share the SMs one to two, as their bytes do (k d
        // elements read and written against 2 k d), all resident at once (both kinds loop over their work)
        int occ = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, compact_kernel<U>, CP_THREADS, smem) == cudaSuccess && occ > 0)
            per_sm = occ;
        const int share = per_sm * GRIFFIN_CP_SHARE_PCT / 100 > 0 ? per_sm * GRIFFIN_CP_SHARE_PCT / 100 : 1;
        const int tiles = ((ldk + TP_J - 1) / TP_J) * ((d + TP_C - 1) / TP_C);
        a.cols_blocks = min(tiles, sms * share);
        const long long cap = (long long)sms * (per_sm - share > 0 ? per_sm - share : 1);
        a.rows_blocks = (int)(want < cap ? want : cap);
    } else {
        a.cols_mode = COLS_GLOBAL;
        a.cols_blocks = (d + CP_ROWS_PER_CTA - 1) / CP_ROWS_PER_CTA;
        a.rows_blocks = (int)(want < (long long)sms * 8 ? want : (long long)sms * 8);
    }
    if (a.rows_blocks < 1) a.rows_blocks = 1;
    const bool biases = (b_gate && out->b_gate_c) || (b_up && out->b_up_c);
    const int bias_blocks = biases ? (k + CP_THREADS - 1) / CP_THREADS : 0;
    const void *fn = (const void *)compact_kernel<U>;
    if (smem > 0 && ensure_dynamic_smem(fn, smem) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    compact_kernel<U><<<a.cols_blocks + a.rows_blocks + bias_blocks, CP_THREADS, smem, stream>>>(a);
    count_launches(1);
    if (cudaGetLastError() != cudaSuccess) return GRIFFIN_ERR_CUDA;
    return GRIFFIN_OK;
}

griffin_status launch_compact(const griffin_ff_desc *desc, const griffin_ff_weights *w, const int32_t *idx,
                              const griffin_ff_compact *out, void *ws, cudaStream_t stream) {
    if (desc->dtype == GRIFFIN_DT_F32)
        return compact_typed<uint32_t>(desc, w->w_gate, w->w_up, w->w_down, false, w->b_gate, w->b_up, idx, out, ws, stream);
    return compact_typed<uint16_t>(desc, w->w_gate, w->w_up, w->w_down, false, w->b_gate, w->b_up, idx, out, ws, stream);
}

griffin_status launch_compact_nm(const griffin_ff_desc *desc, const griffin_ff_weights_nm *w, const int32_t *idx,
                                 const griffin_ff_compact *out, void *ws, cudaStream_t stream) {
    if (desc->dtype == GRIFFIN_DT_F32)
        return compact_typed<uint32_t>(desc, w->w_gate, w->w_up, w->w_down_t, true, w->b_gate, w->b_up, idx, out, ws, stream);
    return compact_typed<uint16_t>(desc, w->w_gate, w->w_up, w->w_down_t, true, w->b_gate, w->b_up, idx, out, ws, stream);
}

}  // namespace griffin
