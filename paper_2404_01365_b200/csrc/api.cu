// C ABI entry points: host-side validation, workspace carve-up, dispatch to the launchers.
#include <math.h>

#include <atomic>
#include <mutex>

#include "common.cuh"
#include "launch.h"

using namespace griffin;

namespace griffin {

static std::atomic<uint64_t> g_launches{0};
void count_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int device_sm_count() {
    static std::atomic<int> cached[64];  // (zero-initialised; two threads that race both store the same value)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
        cached[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

cudaError_t ensure_dynamic_smem(const void *fn, size_t bytes) {
    // remembers, per (device, kernel), the largest limit already granted
    struct Entry {
        const void *fn;
        int dev;
        size_t bytes;
    };
    static Entry table[128];
    static int n_entries = 0;
    static std::mutex table_mutex;  // entry points may be called from several host threads
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(table_mutex);
    for (int i = 0; i < n_entries; ++i)
        if (table[i].fn == fn && table[i].dev == dev) {
            if (table[i].bytes >= bytes) return cudaSuccess;
            e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
            if (e == cudaSuccess) table[i].bytes = bytes;
            return e;
        }
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess && n_entries < 128) table[n_entries++] = Entry{fn, dev, bytes};
    return e;
}

bool grid_can_meet(const void *fn, int threads, size_t smem, int grid) {
    // remembers, per (device, kernel, shared memory), how many CTAs an SM holds
    struct Entry {
        const void *fn;
        int dev;
        size_t smem;
        int per_sm;
    };
    static Entry table[128];
    static int n_entries = 0;
    static std::mutex table_mutex;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const int sms = device_sm_count();
    if (sms <= 0) return false;
    std::lock_guard<std::mutex> lock(table_mutex);
    for (int i = 0; i < n_entries; ++i)
        if (table[i].fn == fn && table[i].dev == dev && table[i].smem == smem)
            return (long long)table[i].per_sm * sms >= grid;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, threads, smem) != cudaSuccess) return false;
    if (n_entries < 128) table[n_entries++] = Entry{fn, dev, smem, per_sm};
    return (long long)per_sm * sms >= grid;
}

}  // namespace griffin

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static griffin_status check_desc(const griffin_ff_desc *desc) {
    if (desc == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (desc->d < 8 || desc->d_ff < 8) return GRIFFIN_ERR_INVALID_ARG;
    if (desc->d % 8 != 0 || desc->d_ff % 8 != 0) return GRIFFIN_ERR_ALIGNMENT;
    if (desc->dtype != GRIFFIN_DT_F32 && desc->dtype != GRIFFIN_DT_BF16) return GRIFFIN_ERR_UNSUPPORTED;
    if (desc->act < GRIFFIN_ACT_SWIGLU || desc->act > GRIFFIN_ACT_SILU) return GRIFFIN_ERR_UNSUPPORTED;
    return GRIFFIN_OK;
}

// A gated block (Eq. 3) needs W_g; a block without a gate (Eq. 2) must not name one.
static bool gate_args_ok(const griffin_ff_desc *desc, const void *w_gate, const void *b_gate) {
    return act_gated(desc->act) ? w_gate != nullptr : (w_gate == nullptr && b_gate == nullptr);
}

static size_t decode_scratch_bytes(const griffin_ff_desc *desc, int n_seq) {
    return (size_t)n_seq * (size_t)desc->d_ff * sizeof(float);  // z [B, ldk], ldk <= d_ff
}

extern "C" {

const char *griffin_status_string(griffin_status st) {
    switch (st) {
        case GRIFFIN_OK: return "ok";
        case GRIFFIN_ERR_INVALID_ARG: return "invalid argument";
        case GRIFFIN_ERR_UNSUPPORTED: return "unsupported shape, dtype or activation";
        case GRIFFIN_ERR_ALIGNMENT: return "pointer or leading dimension not 16-byte aligned";
        case GRIFFIN_ERR_WORKSPACE: return "workspace missing or too small";
        case GRIFFIN_ERR_CUDA: return "CUDA runtime or launch error";
        case GRIFFIN_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

int32_t griffin_version(void) { return GRIFFIN_FF_VERSION; }

uint64_t griffin_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int32_t griffin_k_from_keep_ratio(int32_t d_ff, double keep) {
    if (d_ff < 1) return 0;
    double v = floor(keep * (double)d_ff + 0.5);
    if (!(v >= 1.0)) v = 1.0;  // also catches NaN
    if (v > (double)d_ff) v = (double)d_ff;
    return (int32_t)v;
}

int32_t griffin_compact_ldk(int32_t k) { return k < 1 ? 0 : (k + 7) / 8 * 8; }

size_t griffin_workspace_bytes(const griffin_ff_desc *desc, int32_t S_max, int32_t n_seq_max) {
    if (check_desc(desc) != GRIFFIN_OK || S_max < 0 || n_seq_max < 0) return 0;
    size_t need = 0;
    if (S_max > 0) need = prefill_scratch(desc, S_max).total;
    const size_t dec = decode_scratch_bytes(desc, n_seq_max);
    if (dec > need) need = dec;
    if (desc->dtype == GRIFFIN_DT_BF16 && desc->d <= GRIFFIN_MAX_D) {
        const size_t di = decode_indexed_scratch_bytes(desc->d, n_seq_max);
        if (di > need) need = di;
    }
    return WS_HEADER_BYTES + need;
}

griffin_status griffin_workspace_init(void *workspace, size_t ws_bytes, void *stream) {
    if (workspace == nullptr || ws_bytes < WS_HEADER_BYTES) return GRIFFIN_ERR_WORKSPACE;
    if (!aligned16(workspace)) return GRIFFIN_ERR_ALIGNMENT;
    if (cudaMemsetAsync(workspace, 0, WS_HEADER_BYTES, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return GRIFFIN_ERR_CUDA;
    return GRIFFIN_OK;
}

griffin_status griffin_ff_prefill_score(const griffin_ff_desc *desc, const griffin_ff_weights *w, const void *x,
                                        int32_t S, void *y, float *score, void *workspace, size_t ws_bytes,
                                        void *stream) {
    griffin_status st = check_desc(desc);
    if (st != GRIFFIN_OK) return st;
    if (w == nullptr || w->w_up == nullptr || x == nullptr || score == nullptr || S < 1)
        return GRIFFIN_ERR_INVALID_ARG;
    if (!gate_args_ok(desc, w->w_gate, w->b_gate)) return GRIFFIN_ERR_INVALID_ARG;
    if (y != nullptr && w->w_down == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (!aligned16(w->w_gate) || !aligned16(w->w_up) || !aligned16(w->w_down) || !aligned16(x) || !aligned16(y) ||
        !aligned16(score))
        return GRIFFIN_ERR_ALIGNMENT;
    if (workspace == nullptr) return GRIFFIN_ERR_WORKSPACE;
    if (!aligned16(workspace)) return GRIFFIN_ERR_ALIGNMENT;
    const PrefillScratch ps = prefill_scratch(desc, S);
    if (ws_bytes < WS_HEADER_BYTES + ps.total) return GRIFFIN_ERR_WORKSPACE;
    return launch_prefill_score(desc, w, x, S, y, score, nullptr, 1,
                                static_cast<uint8_t *>(workspace) + WS_HEADER_BYTES, workspace,
                                static_cast<cudaStream_t>(stream));
}

griffin_status griffin_ff_prefill_score_chunk(const griffin_ff_desc *desc, const griffin_ff_weights *w, const void *x,
                                              int32_t S, void *y, float *sumsq, float *score, int32_t first,
                                              void *workspace, size_t ws_bytes, void *stream) {
    griffin_status st = check_desc(desc);
    if (st != GRIFFIN_OK) return st;
    if (w == nullptr || w->w_up == nullptr || x == nullptr || sumsq == nullptr || S < 1)
        return GRIFFIN_ERR_INVALID_ARG;
    if (!gate_args_ok(desc, w->w_gate, w->b_gate)) return GRIFFIN_ERR_INVALID_ARG;
    if (y != nullptr && w->w_down == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (!aligned16(w->w_gate) || !aligned16(w->w_up) || !aligned16(w->w_down) || !aligned16(x) || !aligned16(y) ||
        !aligned16(sumsq) || !aligned16(score))
        return GRIFFIN_ERR_ALIGNMENT;
    if (workspace == nullptr) return GRIFFIN_ERR_WORKSPACE;
    if (!aligned16(workspace)) return GRIFFIN_ERR_ALIGNMENT;
    const PrefillScratch ps = prefill_scratch(desc, S);
    if (ws_bytes < WS_HEADER_BYTES + ps.total) return GRIFFIN_ERR_WORKSPACE;
    return launch_prefill_score(desc, w, x, S, y, score, sumsq, first != 0,
                                static_cast<uint8_t *>(workspace) + WS_HEADER_BYTES, workspace,
                                static_cast<cudaStream_t>(stream));
}

griffin_status griffin_select_topk(const float *score, int32_t n_seq, int32_t d_ff, int32_t k, int32_t *idx,
                                   void *stream) {
    if (score == nullptr || idx == nullptr || n_seq < 1 || d_ff < 1) return GRIFFIN_ERR_INVALID_ARG;
    if (k < 1 || k > d_ff) return GRIFFIN_ERR_INVALID_ARG;
    return launch_select_topk(score, n_seq, d_ff, k, idx, static_cast<cudaStream_t>(stream));
}

griffin_status griffin_combine_scores(const float *score, const int32_t *prompt_len, int32_t n_seq, int32_t d_ff,
                                      float *out, void *stream) {
    if (score == nullptr || prompt_len == nullptr || out == nullptr || n_seq < 1 || d_ff < 1)
        return GRIFFIN_ERR_INVALID_ARG;
    if (n_seq > GRIFFIN_MAX_COMBINE) return GRIFFIN_ERR_UNSUPPORTED;
    for (int i = 0; i < n_seq; ++i)
        if (prompt_len[i] < 1) return GRIFFIN_ERR_INVALID_ARG;
    return launch_combine_scores(score, prompt_len, n_seq, d_ff, out, static_cast<cudaStream_t>(stream));
}

static griffin_status check_compact(const griffin_ff_desc *desc, const griffin_ff_compact *c) {
    if (c->w_up_c == nullptr || c->w_down_c == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (!gate_args_ok(desc, c->w_gate_c, c->b_gate_c)) return GRIFFIN_ERR_INVALID_ARG;
    if (c->k < 1 || c->k > desc->d_ff) return GRIFFIN_ERR_INVALID_ARG;
    if (c->ldk < c->k || c->ldk > desc->d_ff) return GRIFFIN_ERR_INVALID_ARG;
    if (c->ldk % 8 != 0) return GRIFFIN_ERR_ALIGNMENT;
    if (!aligned16(c->w_gate_c) || !aligned16(c->w_up_c) || !aligned16(c->w_down_c)) return GRIFFIN_ERR_ALIGNMENT;
    return GRIFFIN_OK;
}

griffin_status griffin_compact_experts(const griffin_ff_desc *desc, const griffin_ff_weights *w, const int32_t *idx,
                                       const griffin_ff_compact *out, void *workspace, void *stream) {
    griffin_status st = check_desc(desc);
    if (st != GRIFFIN_OK) return st;
    if (w == nullptr || out == nullptr || idx == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (w->w_up == nullptr || w->w_down == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (!gate_args_ok(desc, w->w_gate, w->b_gate)) return GRIFFIN_ERR_INVALID_ARG;
    if (!aligned16(w->w_gate) || !aligned16(w->w_up) || !aligned16(w->w_down)) return GRIFFIN_ERR_ALIGNMENT;
    st = check_compact(desc, out);
    if (st != GRIFFIN_OK) return st;
    if (out->ldk != griffin_compact_ldk(out->k)) return GRIFFIN_ERR_INVALID_ARG;
    return launch_compact(desc, w, idx, out, workspace, static_cast<cudaStream_t>(stream));
}

griffin_status griffin_compact_experts_nm(const griffin_ff_desc *desc, const griffin_ff_weights_nm *w, const int32_t *idx,
                                          const griffin_ff_compact *out, void *workspace, void *stream) {
    griffin_status st = check_desc(desc);
    if (st != GRIFFIN_OK) return st;
    if (w == nullptr || out == nullptr || idx == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (w->w_up == nullptr || w->w_down_t == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (!gate_args_ok(desc, w->w_gate, w->b_gate)) return GRIFFIN_ERR_INVALID_ARG;
    if (!aligned16(w->w_gate) || !aligned16(w->w_up) || !aligned16(w->w_down_t)) return GRIFFIN_ERR_ALIGNMENT;
    st = check_compact(desc, out);
    if (st != GRIFFIN_OK) return st;
    if (out->ldk != griffin_compact_ldk(out->k)) return GRIFFIN_ERR_INVALID_ARG;
    return launch_compact_nm(desc, w, idx, out, workspace, static_cast<cudaStream_t>(stream));
}

griffin_status griffin_ff_decode(const griffin_ff_desc *desc, int32_t B, const griffin_ff_compact *sets,
                                 const void *b_down, const void *x, void *y, void *workspace, size_t ws_bytes,
                                 uint32_t flags, void *stream) {
    griffin_status st = check_desc(desc);
    if (st != GRIFFIN_OK) return st;
    if (sets == nullptr || x == nullptr || y == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (B < 1) return GRIFFIN_ERR_INVALID_ARG;
    if (B > GRIFFIN_MAX_BATCH || desc->d > GRIFFIN_MAX_D) return GRIFFIN_ERR_UNSUPPORTED;
    if (flags & ~(GRIFFIN_DECODE_OVERLAP_WEIGHT_PREFETCH | GRIFFIN_DECODE_TCGEN05 | GRIFFIN_DECODE_RING | GRIFFIN_DECODE_STREAM))
        return GRIFFIN_ERR_INVALID_ARG;
    if ((flags & GRIFFIN_DECODE_RING) && (flags & GRIFFIN_DECODE_STREAM)) return GRIFFIN_ERR_INVALID_ARG;
    for (int b = 0; b < B; ++b) {
        st = check_compact(desc, &sets[b]);
        if (st != GRIFFIN_OK) return st;
        if (sets[b].k != sets[0].k || sets[b].ldk != sets[0].ldk) return GRIFFIN_ERR_INVALID_ARG;
    }
    if (!aligned16(x) || !aligned16(y)) return GRIFFIN_ERR_ALIGNMENT;
    if (workspace == nullptr) return GRIFFIN_ERR_WORKSPACE;
    if (!aligned16(workspace)) return GRIFFIN_ERR_ALIGNMENT;
    if (ws_bytes < WS_HEADER_BYTES + (size_t)B * sets[0].ldk * sizeof(float)) return GRIFFIN_ERR_WORKSPACE;
    float *z = reinterpret_cast<float *>(static_cast<uint8_t *>(workspace) + WS_HEADER_BYTES);
    return launch_decode(desc, B, sets, b_down, x, y, z, workspace, flags, static_cast<cudaStream_t>(stream));
}

griffin_status griffin_ff_decode_indexed(const griffin_ff_desc *desc, int32_t B, const griffin_ff_weights_nm *w,
                                         const int32_t *idx, int32_t k, const void *x, void *y, void *workspace,
                                         size_t ws_bytes, uint32_t flags, void *stream) {
    griffin_status st = check_desc(desc);
    if (st != GRIFFIN_OK) return st;
    if (w == nullptr || idx == nullptr || x == nullptr || y == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (w->w_up == nullptr || w->w_down_t == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (!gate_args_ok(desc, w->w_gate, w->b_gate)) return GRIFFIN_ERR_INVALID_ARG;
    if (B < 1 || k < 1 || k > desc->d_ff) return GRIFFIN_ERR_INVALID_ARG;
    if (flags & ~GRIFFIN_DECODE_OVERLAP_WEIGHT_PREFETCH) return GRIFFIN_ERR_INVALID_ARG;
    if (desc->dtype != GRIFFIN_DT_BF16 || B > GRIFFIN_MAX_BATCH || desc->d > GRIFFIN_MAX_D) return GRIFFIN_ERR_UNSUPPORTED;
    if (!aligned16(w->w_gate) || !aligned16(w->w_up) || !aligned16(w->w_down_t) || !aligned16(x) || !aligned16(y) ||
        (reinterpret_cast<uintptr_t>(idx) & 3u) != 0)
        return GRIFFIN_ERR_ALIGNMENT;
    if (workspace == nullptr) return GRIFFIN_ERR_WORKSPACE;
    if (!aligned16(workspace)) return GRIFFIN_ERR_ALIGNMENT;
    if (ws_bytes < WS_HEADER_BYTES + decode_indexed_scratch_bytes(desc->d, B)) return GRIFFIN_ERR_WORKSPACE;
    float *ypart = reinterpret_cast<float *>(static_cast<uint8_t *>(workspace) + WS_HEADER_BYTES);
    return launch_decode_indexed(desc, B, w, idx, k, x, y, ypart, workspace, flags, static_cast<cudaStream_t>(stream));
}

griffin_status griffin_ff_decode_static(const griffin_ff_desc *desc, int32_t B, const griffin_ff_compact *sets,
                                        const void *b_down, const void *x, void *y, uint32_t flags, void *stream) {
    griffin_status st = check_desc(desc);
    if (st != GRIFFIN_OK) return st;
    if (sets == nullptr || x == nullptr || y == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (B < 1) return GRIFFIN_ERR_INVALID_ARG;
    if (B > GRIFFIN_MAX_BATCH || desc->d > GRIFFIN_MAX_D) return GRIFFIN_ERR_UNSUPPORTED;
    if (flags & ~(GRIFFIN_DECODE_OVERLAP_WEIGHT_PREFETCH | GRIFFIN_DECODE_TCGEN05 | GRIFFIN_DECODE_RING | GRIFFIN_DECODE_STREAM))
        return GRIFFIN_ERR_INVALID_ARG;
    if ((flags & GRIFFIN_DECODE_RING) && (flags & GRIFFIN_DECODE_STREAM)) return GRIFFIN_ERR_INVALID_ARG;
    for (int b = 0; b < B; ++b) {
        st = check_compact(desc, &sets[b]);
        if (st != GRIFFIN_OK) return st;
        if (sets[b].k != sets[0].k || sets[b].ldk != sets[0].ldk) return GRIFFIN_ERR_INVALID_ARG;
    }
    if (!aligned16(x) || !aligned16(y)) return GRIFFIN_ERR_ALIGNMENT;
    // the size check against GRIFFIN_STATIC_SCRATCH_BYTES happens in the launcher, before any CUDA call
    return launch_decode_static(desc, B, sets, b_down, x, y, flags, static_cast<cudaStream_t>(stream));
}

griffin_status griffin_ff_decode_static_status(void *stream) {
    return static_scratch_status(static_cast<cudaStream_t>(stream));
}

griffin_status griffin_check_device_status(const void *workspace, void *stream) {
    if (workspace == nullptr) return GRIFFIN_ERR_WORKSPACE;
    WsHeader h;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&h, workspace, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    if (h.status == DEV_STATUS_TIMEOUT) return GRIFFIN_ERR_TIMEOUT;
    if (h.status == DEV_STATUS_BAD_INDEX) return GRIFFIN_ERR_INVALID_ARG;
    return h.status == DEV_STATUS_OK ? GRIFFIN_OK : GRIFFIN_ERR_CUDA;
}

}  // extern "C"
