// Expert selection (Section 4.2 of the GRIFFIN paper): E = indices of the k largest entries
// of the statistic s, ties to the lower index, written in ascending index order.
//
// One CTA per sequence.  Scores are mapped to order-preserving 32-bit keys; four 8-bit
// radix passes (most significant digit first) find the k-th largest key tau and how many
// of the entries equal to tau are still needed; one ordered sweep then emits every index
// whose key is above tau plus the first `need` indices whose key equals tau.  Integer
// work only after the key mapping, so the result is exact and deterministic.
#include "common.cuh"
#include "launch.h"

namespace griffin {

constexpr int TOPK_THREADS = 1024;

__device__ __forceinline__ uint32_t order_key(float f) {
    f = f + 0.0f;  // -0 -> +0, so equal floats get equal keys
    const uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__global__ void __launch_bounds__(TOPK_THREADS) select_topk_kernel(const float *__restrict__ score, int d_ff, int k,
                                                                   int32_t *__restrict__ idx) {
    const float *s = score + (size_t)blockIdx.x * d_ff;
    int32_t *out = idx + (size_t)blockIdx.x * k;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    __shared__ uint32_t hist[256];
    __shared__ uint32_t sh_prefix, sh_remaining;
    __shared__ uint32_t warp_tot[32];

    uint32_t prefix = 0, mask = 0, remaining = (uint32_t)k;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (int j = tid; j < d_ff; j += TOPK_THREADS) {
            const uint32_t key = order_key(s[j]);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (warp == 0) {
            // lane l owns the 8 bins 255-8l ... 248-8l (descending); find the bin in which
            // the running count from the top first reaches `remaining`
            uint32_t loc[8], tot = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                loc[i] = hist[255 - 8 * lane - i];
                tot += loc[i];
            }
            uint32_t incl = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            uint32_t cum = incl - tot;
            if (cum < remaining && remaining <= incl) {
                bool found = false;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (!found && cum + loc[i] >= remaining) {
                        sh_prefix = prefix | ((uint32_t)(255 - 8 * lane - i) << shift);
                        sh_remaining = remaining - cum;
                        found = true;
                    }
                    cum += loc[i];
                }
            }
        }
        __syncthreads();
        prefix = sh_prefix;
        remaining = sh_remaining;
        mask |= 0xffu << shift;
    }
    const uint32_t tau = prefix;      // key of the k-th largest score
    const uint32_t need = remaining;  // entries equal to tau that belong to E (>= 1)

    uint32_t gt_base = 0, eq_base = 0;
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int base = 0; base < d_ff; base += TOPK_THREADS) {
        const int j = base + tid;
        const bool valid = j < d_ff;
        const uint32_t key = valid ? order_key(s[j]) : 0u;
        const bool gt = valid && key > tau;
        const bool eq = valid && key == tau;
        const uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
        if (lane == 0) warp_tot[warp] = (uint32_t)__popc(bg) | ((uint32_t)__popc(be) << 16);
        __syncthreads();
        const uint32_t v = warp_tot[lane];
        uint32_t incl = v;  // two 16-bit counters packed; a chunk holds at most 1024 entries
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        const uint32_t excl = __shfl_sync(0xffffffffu, incl - v, warp);
        const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
        const uint32_t g_before = gt_base + (excl & 0xffffu) + (uint32_t)__popc(bg & lt_mask);
        const uint32_t e_before = eq_base + (excl >> 16) + (uint32_t)__popc(be & lt_mask);
        if (gt || (eq && e_before < need)) out[g_before + min(e_before, need)] = j;
        gt_base += total & 0xffffu;
        eq_base += total >> 16;
        __syncthreads();
    }
}

// Batch statistic s_bar = sum_i s_i / sqrt(S_i) (Eq. 7); the weights 1/sqrt(S_i) arrive by value.
struct CombineWeights {
    float w[GRIFFIN_MAX_COMBINE];
};
__global__ void combine_scores_kernel(const float *__restrict__ score, const __grid_constant__ CombineWeights cw,
                                      int n_seq, int d_ff, float *__restrict__ out) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d_ff) return;
    float acc = 0.f;
    for (int i = 0; i < n_seq; ++i) acc = fmaf(score[(size_t)i * d_ff + j], cw.w[i], acc);
    out[j] = acc;
}

griffin_status launch_select_topk(const float *score, int n_seq, int d_ff, int k, int32_t *idx, cudaStream_t stream) {
    select_topk_kernel<<<n_seq, TOPK_THREADS, 0, stream>>>(score, d_ff, k, idx);
    count_launches(1);
    return cudaGetLastError() == cudaSuccess ? GRIFFIN_OK : GRIFFIN_ERR_CUDA;
}

griffin_status launch_combine_scores(const float *score, const int32_t *prompt_len_host, int n_seq, int d_ff,
                                     float *out, cudaStream_t stream) {
    CombineWeights cw;
    for (int i = 0; i < n_seq; ++i) cw.w[i] = (float)(1.0 / sqrt((double)prompt_len_host[i]));
    combine_scores_kernel<<<(d_ff + 255) / 256, 256, 0, stream>>>(score, cw, n_seq, d_ff, out);
    count_launches(1);
    return cudaGetLastError() == cudaSuccess ? GRIFFIN_OK : GRIFFIN_ERR_CUDA;
}

}  // namespace griffin
