// Shared device helpers for the GRIFFIN FF kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "griffin_ff.h"

namespace griffin {

// ---------------------------------------------------------------------------------------
// Workspace layout.  The first WS_HEADER_BYTES hold the device status word; the rest is
// scratch that each entry point carves up for itself (calls sharing a workspace are
// stream-ordered, so the regions may alias between calls).
// ---------------------------------------------------------------------------------------
constexpr size_t WS_HEADER_BYTES = 256;
constexpr int DEV_STATUS_OK = 0;
constexpr int DEV_STATUS_TIMEOUT = 1;    // a bounded wait gave up
constexpr int DEV_STATUS_BAD_INDEX = 2;  // an expert index outside [0, d_ff)

struct WsHeader {
    int status;           // DEV_STATUS_*
    int detail;           // where it happened (kernel-specific code)
    unsigned int meet_warp;  // meeting-point counter of the warp-level fused decode kernel (see grid_meet)
    unsigned int meet_tc;    // ... and of the tcgen05 one (the two have different numbers of parties)
    unsigned int meet_idx;   // ... and of the index-direct one
    unsigned int meet_stream;  // ... and of the register-streaming one
    unsigned int pool_stream;  // that kernel's count of claims on its pool of pairs (runs round once per call)
};

__device__ __forceinline__ void raise_status(void *ws, int status, int detail) {
    if (ws != nullptr) {
        WsHeader *h = reinterpret_cast<WsHeader *>(ws);
        if (atomicCAS(&h->status, DEV_STATUS_OK, status) == DEV_STATUS_OK) h->detail = detail;
    }
}

// ---------------------------------------------------------------------------------------
// Element types: 16-byte vectors of T widened to fp32.
// ---------------------------------------------------------------------------------------
template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int VEC = 4;  // elements per 16 bytes
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&f)[4]) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ float to_float(float v) { return v; }
    static __device__ __forceinline__ float from_float(float v) { return v; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int VEC = 8;
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&f)[8]) {
        // bf16 -> fp32 is a 16-bit shift; the low half of each word is the earlier element
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
        f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
        f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
    }
    static __device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
    static __device__ __forceinline__ __nv_bfloat16 from_float(float v) { return __float2bfloat16_rn(v); }
};

// ---------------------------------------------------------------------------------------
// Gate non-linearity sigma (Eq. 3), fp32.
// ---------------------------------------------------------------------------------------
template <int ACT> __device__ __forceinline__ float sigma(float t) {
    if constexpr (ACT == GRIFFIN_ACT_SWIGLU) {
        return t / (1.0f + __expf(-t));
    } else if constexpr (ACT == GRIFFIN_ACT_GEGLU_TANH) {
        const float c = 0.7978845608028654f;  // sqrt(2/pi)
        const float inner = c * (t + 0.044715f * t * t * t);
        // tanh(a) = 1 - 2 / (exp(2a) + 1); an overflowing exp still gives the right limit
        const float th = 1.0f - 2.0f / (__expf(2.0f * inner) + 1.0f);
        return 0.5f * t * (1.0f + th);
    } else if constexpr (ACT == GRIFFIN_ACT_GEGLU_ERF) {
        return 0.5f * t * (1.0f + erff(t * 0.70710678118654752f));
    } else {
        return fmaxf(t, 0.0f);
    }
}

// The sigma of an activation code, as the code of the gated form that uses the same function: the
// kernels get this (0..3) as `act` plus, separately, whether the block has a gate (Eq. 3) or not
// (Eq. 2).
__host__ __device__ inline int act_sigma(int act) {
    switch (act) {
        case GRIFFIN_ACT_RELU: return GRIFFIN_ACT_REGLU;
        case GRIFFIN_ACT_GELU_TANH: return GRIFFIN_ACT_GEGLU_TANH;
        case GRIFFIN_ACT_GELU_ERF: return GRIFFIN_ACT_GEGLU_ERF;
        case GRIFFIN_ACT_SILU: return GRIFFIN_ACT_SWIGLU;
        default: return act;
    }
}
__host__ __device__ inline bool act_gated(int act) { return GRIFFIN_ACT_IS_GATED(act); }

__device__ __forceinline__ float sigma_rt(int act, float t) {
    switch (act) {
        case GRIFFIN_ACT_SWIGLU: return sigma<GRIFFIN_ACT_SWIGLU>(t);
        case GRIFFIN_ACT_GEGLU_TANH: return sigma<GRIFFIN_ACT_GEGLU_TANH>(t);
        case GRIFFIN_ACT_GEGLU_ERF: return sigma<GRIFFIN_ACT_GEGLU_ERF>(t);
        default: return sigma<GRIFFIN_ACT_REGLU>(t);
    }
}

// ---------------------------------------------------------------------------------------
// mbarrier + bulk-copy (TMA, 1-D, no multicast) primitives.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Every device-side wait gives up after this many SM clock cycles (about 2 s).
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;

// Barrier wait that gives up after `limit` SM clock cycles (WAIT_LIMIT_CYCLES everywhere in the
// library; only the self-test of this primitive passes a shorter one), or as soon as another
// thread of the CTA has given up.  On a give-up the status word is raised and false is returned.
__device__ __forceinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort, void *ws,
                                              int where, long long limit = WAIT_LIMIT_CYCLES) {
    // Fast path: plain polling.  The clock is only consulted every few thousand polls, so a
    // wait that succeeds (every wait of a healthy run) never pays for reading it.
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort) return false;
#pragma unroll 1
    for (int i = 0; i < 4096; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 4096; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort) return false;
        if (clock64() - t0 > limit) {
            *abort = 1;
            raise_status(ws, DEV_STATUS_TIMEOUT, where);
            return false;
        }
    }
}

// The same for many threads that wait long (an epilogue waiting for a whole work item): they
// sleep between polls, so that their polling does not take issue slots and shared-memory
// cycles from the warps that do the work.
__device__ __forceinline__ bool wait_or_abort_relaxed(uint64_t *bar, uint32_t parity, volatile int *abort, void *ws,
                                                      int where) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        __nanosleep(64);
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort) return false;
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
            *abort = 1;
            raise_status(ws, DEV_STATUS_TIMEOUT, where);
            return false;
        }
    }
}

// 1-D bulk copy global -> shared memory of this CTA; completion is counted on `bar` in
// bytes.  dst and src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Programmatic dependent launch controls.
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait_prior_grids() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

}  // namespace griffin
