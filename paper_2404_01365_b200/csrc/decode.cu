// Generation-phase pruned FF (Eqs. 4 and 5 of the GRIFFIN paper):
//   z_hat = sigma(W_g_hat x + b_g_hat) * (W_1_hat x + b_1_hat)        kernel "gate_up"
//   y_hat = W_2_hat z_hat + b_2                                        kernel "down"
//
// This file holds the fp32-FMA kernels (fp32 storage) and the dispatcher; bf16 storage goes
// through the warp-MMA kernels in decode_mma.cu, which share the pipeline design below.
//
// At batch 1..8 both products are matrix-vector products whose cost is the single pass
// over the compact weights, so both kernels are built around keeping HBM busy:
//   * one CTA per SM, persistent over its share of the work items;
//   * a producer warp streams weight rows into a ring of shared-memory stages with 1-D
//     bulk copies (TMA, no multicast) tracked by mbarriers; 8 consumer warps read the
//     stages, keep the vector operand (x, or a tile of z) in registers and reduce with
//     warp shuffles;
//   * with programmatic dependent launch the producer starts streaming weights before
//     the previous kernel on the stream has finished; everything that depends on that
//     kernel (x, z, y) is touched only after griddepcontrol.wait.
// Results are deterministic: every sum has a fixed order.
#include <atomic>

#include "decode_common.cuh"

namespace griffin {

// ---------------------------------------------------------------------------------------
// Kernel gate_up:
//   z[b, j] = sigma(w_gate_c[j,:] . x[b] + b_gate_c[j]) * (w_up_c[j,:] . x[b] + b_up_c[j])
// Work item = (sequence b, slice of neurons).  Stage = gate row j followed by up row j.
// GATED = false (a block without a gate, Eq. 2): z[b, j] = sigma(w_up_c[j,:] . x[b] + b_up_c[j]),
// stage = up row j alone.
// ---------------------------------------------------------------------------------------
template <typename T, int ITER, bool GATED>
__global__ void __launch_bounds__(DEC_THREADS) decode_gate_up_kernel(const __grid_constant__ DecodeParams p, int act) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    constexpr int VEC = Elem<T>::VEC;
    const int row_bytes = p.d * (int)sizeof(T);
    const int stage_bytes = (GATED ? 2 : 1) * row_bytes;
    const DecSmem s = carve(smem_raw, p.n_stages, stage_bytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < p.n_stages; ++i) {
            mbar_init(&s.full[i], 1);
            mbar_init(&s.empty[i], DEC_CONSUMER_WARPS);
        }
        *s.abort = 0;
        mbar_fence_init();
    }
    __syncthreads();
    pdl_launch_dependents();

    const int n_items = p.B * p.n_slices;
    if (warp == DEC_CONSUMER_WARPS) {
        // ---- producer: touches weights only, so it never waits for the previous grid
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
                const int b = item / p.n_slices, sl = item - b * p.n_slices;
                const int j0 = (int)((long long)sl * p.k / p.n_slices);
                const int j1 = (int)((long long)(sl + 1) * p.k / p.n_slices);
                const uint8_t *g = static_cast<const uint8_t *>(p.seq[b].w_gate);
                const uint8_t *u = static_cast<const uint8_t *>(p.seq[b].w_up);
                for (int j = j0; j < j1; ++j, ++it) {
                    const int stage = it % p.n_stages;
                    const uint32_t use = it / p.n_stages;
                    if (use > 0 && !wait_or_abort(&s.empty[stage], (use - 1) & 1, s.abort, p.ws, 1)) {
                        ok = false;
                        break;
                    }
                    uint8_t *dst = s.stages + (size_t)stage * stage_bytes;
                    mbar_arrive_expect_tx(&s.full[stage], stage_bytes);
                    if (GATED) bulk_g2s(dst, g + (size_t)j * row_bytes, row_bytes, &s.full[stage]);
                    bulk_g2s(dst + (GATED ? row_bytes : 0), u + (size_t)j * row_bytes, row_bytes, &s.full[stage]);
                }
            }
            producer_drain(s, p.n_stages, it);
        }
        return;
    }

    // ---- consumers
    pdl_wait_prior_grids();  // x and the z scratch belong to earlier work on the stream
    uint32_t it = 0;
    int item_parity = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, item_parity ^= 1) {
        const int b = item / p.n_slices, sl = item - b * p.n_slices;
        const int j0 = (int)((long long)sl * p.k / p.n_slices);
        const int j1 = (int)((long long)(sl + 1) * p.k / p.n_slices);
        float2 *part = reinterpret_cast<float2 *>(s.part + item_parity * DEC_PART_FLOATS);

        float xr[ITER][VEC];
#pragma unroll
        for (int i = 0; i < ITER; ++i) {
            const int col = (tid + i * DEC_CONSUMERS) * VEC;
            if (col < p.d) {
                const uint4 v = *reinterpret_cast<const uint4 *>(static_cast<const T *>(p.x) + (size_t)b * p.d + col);
                Elem<T>::unpack(v, xr[i]);
            } else {
#pragma unroll
                for (int e = 0; e < VEC; ++e) xr[i][e] = 0.f;
            }
        }

        bool ok = true;
        for (int j = j0; j < j1; ++j, ++it) {
            const int stage = it % p.n_stages;
            if (!wait_or_abort(&s.full[stage], (it / p.n_stages) & 1, s.abort, p.ws, 2)) {
                ok = false;
                break;
            }
            const uint8_t *src = s.stages + (size_t)stage * stage_bytes;
            float ga = 0.f, ua = 0.f;
#pragma unroll
            for (int i = 0; i < ITER; ++i) {
                const int col = (tid + i * DEC_CONSUMERS) * VEC;
                if (col < p.d) {
                    float gf[VEC], uf[VEC];
                    if (GATED) Elem<T>::unpack(*reinterpret_cast<const uint4 *>(src + (size_t)col * sizeof(T)), gf);
                    Elem<T>::unpack(*reinterpret_cast<const uint4 *>(src + (GATED ? row_bytes : 0) + (size_t)col * sizeof(T)), uf);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        if (GATED) ga = fmaf(gf[e], xr[i][e], ga);
                        ua = fmaf(uf[e], xr[i][e], ua);
                    }
                }
            }
            if (GATED) ga = warp_sum(ga);
            ua = warp_sum(ua);
            if (lane == 0) {
                // every lane's shared-memory reads fed the shuffles above, so they are done
                mbar_arrive(&s.empty[stage]);
                part[(j - j0) * DEC_CONSUMER_WARPS + warp] = make_float2(ga, ua);
            }
        }
        consumer_barrier();
        if (!ok || *s.abort) break;
        if (tid < j1 - j0) {
            float ga = 0.f, ua = 0.f;
#pragma unroll
            for (int w = 0; w < DEC_CONSUMER_WARPS; ++w) {
                const float2 v = part[tid * DEC_CONSUMER_WARPS + w];
                ga += v.x;
                ua += v.y;
            }
            const int j = j0 + tid;
            if (GATED && p.seq[b].b_gate) ga += Elem<T>::to_float(static_cast<const T *>(p.seq[b].b_gate)[j]);
            if (p.seq[b].b_up) ua += Elem<T>::to_float(static_cast<const T *>(p.seq[b].b_up)[j]);
            p.z[(size_t)b * p.ldk + j] = GATED ? sigma_rt(act, ga) * ua : sigma_rt(act, ua);
        }
        // the last slice also clears the padding of z (at most 7 entries)
        const int pad = tid - (DEC_CONSUMERS - 8);
        if (sl == p.n_slices - 1 && pad >= 0 && p.k + pad < p.ldk) p.z[(size_t)b * p.ldk + p.k + pad] = 0.f;
    }
}

// ---------------------------------------------------------------------------------------
// Kernel down:  y[b, c] = w_down_c[c, 0:k] . z[b, 0:k] + b_down[c]
// Work item = (sequence b, chunk of output rows).  Rows are cut into k-tiles so that the
// matching tile of z sits in registers; stage = the same k-tile of two consecutive rows.
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(DEC_THREADS) decode_down_kernel(const __grid_constant__ DecodeParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    constexpr int VEC = Elem<T>::VEC;
    constexpr int ITER = DEC_DOWN_ITER;
    const int seg_bytes_max = p.kt_len * (int)sizeof(T);
    const int stage_bytes = 2 * seg_bytes_max;
    const DecSmem s = carve(smem_raw, p.n_stages, stage_bytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < p.n_stages; ++i) {
            mbar_init(&s.full[i], 1);
            mbar_init(&s.empty[i], DEC_CONSUMER_WARPS);
        }
        *s.abort = 0;
        mbar_fence_init();
    }
    __syncthreads();
    pdl_launch_dependents();

    const int n_items = p.B * p.n_slices;
    if (warp == DEC_CONSUMER_WARPS) {
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
                const int b = item / p.n_slices, sl = item - b * p.n_slices;
                const int c0 = (int)((long long)sl * p.d / p.n_slices);
                const int c1 = (int)((long long)(sl + 1) * p.d / p.n_slices);
                const uint8_t *w = static_cast<const uint8_t *>(p.seq[b].w_down);
                for (int kt = 0; ok && kt < p.n_ktiles; ++kt) {
                    const int e0 = kt * p.kt_len;
                    const int len = min(p.kt_len, p.ldk - e0);
                    const uint32_t seg_bytes = (uint32_t)len * sizeof(T);
                    for (int c = c0; c < c1; c += 2, ++it) {
                        const int stage = it % p.n_stages;
                        const uint32_t use = it / p.n_stages;
                        if (use > 0 && !wait_or_abort(&s.empty[stage], (use - 1) & 1, s.abort, p.ws, 3)) {
                            ok = false;
                            break;
                        }
                        uint8_t *dst = s.stages + (size_t)stage * stage_bytes;
                        const bool two = c + 1 < c1;
                        mbar_arrive_expect_tx(&s.full[stage], two ? 2 * seg_bytes : seg_bytes);
                        bulk_g2s(dst, w + ((size_t)c * p.ldk + e0) * sizeof(T), seg_bytes, &s.full[stage]);
                        if (two)
                            bulk_g2s(dst + seg_bytes_max, w + ((size_t)(c + 1) * p.ldk + e0) * sizeof(T), seg_bytes,
                                     &s.full[stage]);
                    }
                }
            }
            producer_drain(s, p.n_stages, it);
        }
        return;
    }

    pdl_wait_prior_grids();  // z comes from the gate_up kernel
    uint32_t it = 0;
    int item_parity = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, item_parity ^= 1) {
        const int b = item / p.n_slices, sl = item - b * p.n_slices;
        const int c0 = (int)((long long)sl * p.d / p.n_slices);
        const int c1 = (int)((long long)(sl + 1) * p.d / p.n_slices);
        float *part = s.part + item_parity * DEC_PART_FLOATS;
        bool ok = true;
        for (int kt = 0; ok && kt < p.n_ktiles; ++kt) {
            const int e0 = kt * p.kt_len;
            const int len = min(p.kt_len, p.ldk - e0);
            float zr[ITER][VEC];
#pragma unroll
            for (int i = 0; i < ITER; ++i) {
                const int col = (tid + i * DEC_CONSUMERS) * VEC;
#pragma unroll
                for (int e = 0; e < VEC; ++e) zr[i][e] = 0.f;
                if (col < len) {
                    const float4 *zp = reinterpret_cast<const float4 *>(p.z + (size_t)b * p.ldk + e0 + col);
#pragma unroll
                    for (int q = 0; q < VEC / 4; ++q) {
                        const float4 v = zp[q];
                        zr[i][4 * q + 0] = v.x; zr[i][4 * q + 1] = v.y;
                        zr[i][4 * q + 2] = v.z; zr[i][4 * q + 3] = v.w;
                    }
                }
            }
            for (int c = c0; c < c1; c += 2, ++it) {
                const int stage = it % p.n_stages;
                if (!wait_or_abort(&s.full[stage], (it / p.n_stages) & 1, s.abort, p.ws, 4)) {
                    ok = false;
                    break;
                }
                const uint8_t *src = s.stages + (size_t)stage * stage_bytes;
                const bool two = c + 1 < c1;
                float a0 = 0.f, a1 = 0.f;
#pragma unroll
                for (int i = 0; i < ITER; ++i) {
                    const int col = (tid + i * DEC_CONSUMERS) * VEC;
                    if (col < len) {
                        float w0[VEC];
                        Elem<T>::unpack(*reinterpret_cast<const uint4 *>(src + (size_t)col * sizeof(T)), w0);
#pragma unroll
                        for (int e = 0; e < VEC; ++e) a0 = fmaf(w0[e], zr[i][e], a0);
                        if (two) {
                            float w1[VEC];
                            Elem<T>::unpack(
                                *reinterpret_cast<const uint4 *>(src + seg_bytes_max + (size_t)col * sizeof(T)), w1);
#pragma unroll
                            for (int e = 0; e < VEC; ++e) a1 = fmaf(w1[e], zr[i][e], a1);
                        }
                    }
                }
                a0 = warp_sum(a0);
                a1 = warp_sum(a1);
                if (lane == 0) {
                    mbar_arrive(&s.empty[stage]);
                    float *q = part + (c - c0) * DEC_CONSUMER_WARPS + warp;  // rows c and c+1
                    if (kt == 0) {
                        q[0] = a0;
                        q[DEC_CONSUMER_WARPS] = a1;
                    } else {
                        q[0] += a0;
                        q[DEC_CONSUMER_WARPS] += a1;
                    }
                }
            }
        }
        consumer_barrier();
        if (!ok || *s.abort) break;
        if (tid < c1 - c0) {
            float acc = 0.f;
#pragma unroll
            for (int w = 0; w < DEC_CONSUMER_WARPS; ++w) acc += part[tid * DEC_CONSUMER_WARPS + w];
            const int c = c0 + tid;
            if (p.b_down) acc += Elem<T>::to_float(static_cast<const T *>(p.b_down)[c]);
            static_cast<T *>(p.y)[(size_t)b * p.d + c] = Elem<T>::from_float(acc);
        }
    }
}

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
cudaError_t launch_maybe_overlapped(const void *func, dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                           bool overlap, void **args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = overlap ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launches(1);
    return cudaLaunchKernelExC(&cfg, func, args);
}

#ifndef GRIFFIN_DEC_STAGE_KB
#define GRIFFIN_DEC_STAGE_KB 96
#endif
static int pick_stages(int stage_bytes) {
    // about 96 KB of stages: deep enough to cover HBM latency, small enough that the next
    // kernel's CTA fits beside this one on the SM and can prefetch its own weights
    int n = (GRIFFIN_DEC_STAGE_KB * 1024) / stage_bytes;
    if (n < 2) n = 2;
    if (n > 12) n = 12;
    return n;
}

int slices_for(int rows, int grid) {
    // a multiple of the grid, fine enough that one item has at most DEC_MAX_ROWS rows
    int per = (rows + grid * DEC_MAX_ROWS - 1) / (grid * DEC_MAX_ROWS);
    if (per < 1) per = 1;
    return grid * per;
}

template <typename T, bool GATED>
static const void *gate_up_fn(int iter) {
    switch (iter) {
        case 1: return (const void *)decode_gate_up_kernel<T, 1, GATED>;
        case 2: return (const void *)decode_gate_up_kernel<T, 2, GATED>;
        case 3: return (const void *)decode_gate_up_kernel<T, 3, GATED>;
        case 4: return (const void *)decode_gate_up_kernel<T, 4, GATED>;
        case 5: case 6: return (const void *)decode_gate_up_kernel<T, 6, GATED>;
        case 7: case 8: return (const void *)decode_gate_up_kernel<T, 8, GATED>;
        default: return nullptr;
    }
}

// act: the code of sigma (0..3); gated: whether the block has a gate (Eq. 3) or not (Eq. 2)
template <typename T>
static griffin_status decode_simt(DecodeParams &p, int act, bool gated, uint32_t flags, cudaStream_t stream) {
    constexpr int VEC = Elem<T>::VEC;
    const int B = p.B;
    const int sms = device_sm_count();
    if (sms <= 0) return GRIFFIN_ERR_CUDA;
    const bool overlap = (flags & GRIFFIN_DECODE_OVERLAP_WEIGHT_PREFETCH) != 0;

    {  // gate_up
        const int stage_bytes = (gated ? 2 : 1) * p.d * (int)sizeof(T);
        p.n_stages = pick_stages(stage_bytes);
        p.n_slices = slices_for(p.k, sms);
        const int grid = min(sms, B * p.n_slices);
        const size_t smem = dec_smem_bytes(p.n_stages, stage_bytes);
        const int iter = (p.d + DEC_CONSUMERS * VEC - 1) / (DEC_CONSUMERS * VEC);
        const void *fn = gated ? gate_up_fn<T, true>(iter) : gate_up_fn<T, false>(iter);
        if (fn == nullptr) return GRIFFIN_ERR_UNSUPPORTED;
        if (ensure_dynamic_smem(fn, smem) != cudaSuccess) return GRIFFIN_ERR_CUDA;
        void *args[] = {&p, &act};
        if (launch_maybe_overlapped(fn, dim3(grid), dim3(DEC_THREADS), smem, stream, overlap, args) != cudaSuccess)
            return GRIFFIN_ERR_CUDA;
    }
    {  // down: may always start early, since gate_up never writes weights
        const int kt_max = DEC_CONSUMERS * VEC * DEC_DOWN_ITER;
        p.n_ktiles = (p.ldk + kt_max - 1) / kt_max;
        const int kt_len = (p.ldk + p.n_ktiles - 1) / p.n_ktiles;
        p.kt_len = (kt_len + 7) / 8 * 8;
        const int stage_bytes = 2 * p.kt_len * (int)sizeof(T);
        p.n_stages = pick_stages(stage_bytes);
        p.n_slices = slices_for(p.d, sms);
        const int grid = min(sms, B * p.n_slices);
        const size_t smem = dec_smem_bytes(p.n_stages, stage_bytes);
        const void *fn = (const void *)decode_down_kernel<T>;
        if (ensure_dynamic_smem(fn, smem) != cudaSuccess) return GRIFFIN_ERR_CUDA;
        void *args[] = {&p};
        if (launch_maybe_overlapped(fn, dim3(grid), dim3(DEC_THREADS), smem, stream, true, args) != cudaSuccess)
            return GRIFFIN_ERR_CUDA;
    }
    return GRIFFIN_OK;
}

// Weight bytes of a call from which the register-streaming kernel is the default.
#ifndef GRIFFIN_STREAM_MIN_MB
#define GRIFFIN_STREAM_MIN_MB 150
#endif
griffin_status launch_decode(const griffin_ff_desc *desc, int B, const griffin_ff_compact *sets, const void *b_down,
                             const void *x, void *y, float *z, void *ws, uint32_t flags, cudaStream_t stream) {
    DecodeParams p = {};
    for (int b = 0; b < B; ++b) {
        p.seq[b].w_gate = sets[b].w_gate_c;
        p.seq[b].w_up = sets[b].w_up_c;
        p.seq[b].w_down = sets[b].w_down_c;
        p.seq[b].b_gate = sets[b].b_gate_c;
        p.seq[b].b_up = sets[b].b_up_c;
    }
    p.b_down = b_down;
    p.x = x;
    p.y = y;
    p.z = z;
    p.ws = ws;
    p.d = desc->d;
    p.k = sets[0].k;
    p.ldk = sets[0].ldk;
    p.B = B;
    const int act = act_sigma(desc->act);
    const bool gated = act_gated(desc->act);
    if (desc->dtype == GRIFFIN_DT_F32) return decode_simt<float>(p, act, gated, flags, stream);
    const bool want_tc = gated && (flags & GRIFFIN_DECODE_TCGEN05) != 0;  // (the tcgen05 kernels are built for gated blocks)
    // one expert set for several sequences (Eq. 7): streamed once for up to 8 of them at a time
    if (decode_shared_set(p) && !(want_tc && decode_tc_shared(p))) {
        const griffin_status st = decode_bf16_shared(p, act, gated, flags, stream);
        if (st != GRIFFIN_ERR_UNSUPPORTED) return st;
    }
    // sequences with their own sets: the register stream once every warp has enough to do, else the ring
    // (a shape that the stream kernel cannot place goes to the ring kernel after all)
    bool use_stream = (flags & GRIFFIN_DECODE_STREAM) != 0;
    if (!use_stream && !(flags & GRIFFIN_DECODE_RING) && !want_tc)
        use_stream = (size_t)B * 3 * p.k * p.d * 2 >= (size_t)GRIFFIN_STREAM_MIN_MB * 1000 * 1000;
    if (use_stream) {
        const griffin_status st = decode_bf16_stream(p, act, gated, flags, stream);
        if (st != GRIFFIN_ERR_UNSUPPORTED) return st;
    }
    if (!gated) return decode_bf16_mma(p, act, false, flags, stream);
    // (a shape that the tcgen05 plan cannot place in shared memory or TMEM after all goes to the warp-level kernel)
    if (want_tc && decode_tc_supported(p)) {
        const griffin_status st = decode_bf16_tc(p, act, flags, stream);
        if (st != GRIFFIN_ERR_UNSUPPORTED) return st;
    }
    return decode_bf16_mma(p, act, true, flags, stream);
}

// ---------------------------------------------------------------------------------------
// Decode without a caller-provided workspace: z lives in a static device array that is part
// of this library's image (one copy per GPU that loads it).  In host code the array's name
// is only a stand-in; the address a kernel may use comes from cudaGetSymbolAddress, asked
// once per device with that device current.
// ---------------------------------------------------------------------------------------
// 256 bytes of header (what a workspace starts with; zero at load time and self-cleaning) + the scratch proper
static __device__ __align__(256) unsigned char g_static_decode_scratch[256 + GRIFFIN_STATIC_SCRATCH_BYTES];

static unsigned char *static_scratch_of_current_device() {
    static std::atomic<unsigned char *> addr[64];  // (zero-initialised; two threads that race both store the same address)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    unsigned char *a = addr[dev].load(std::memory_order_acquire);
    if (a == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_decode_scratch) != cudaSuccess) return nullptr;
        a = static_cast<unsigned char *>(p);
        addr[dev].store(a, std::memory_order_release);
    }
    return a;
}

griffin_status static_scratch_status(cudaStream_t stream) {
    unsigned char *base = static_scratch_of_current_device();
    if (base == nullptr) return GRIFFIN_ERR_CUDA;
    WsHeader h;
    if (cudaMemcpyAsync(&h, base, sizeof(h), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    if (h.status == DEV_STATUS_OK) return GRIFFIN_OK;
    if (cudaMemsetAsync(base, 0, WS_HEADER_BYTES, stream) != cudaSuccess || cudaStreamSynchronize(stream) != cudaSuccess)
        return GRIFFIN_ERR_CUDA;
    if (h.status == DEV_STATUS_TIMEOUT) return GRIFFIN_ERR_TIMEOUT;
    return h.status == DEV_STATUS_BAD_INDEX ? GRIFFIN_ERR_INVALID_ARG : GRIFFIN_ERR_CUDA;
}

griffin_status launch_decode_static(const griffin_ff_desc *desc, int B, const griffin_ff_compact *sets,
                                    const void *b_down, const void *x, void *y, uint32_t flags, cudaStream_t stream) {
    if ((size_t)B * (size_t)sets[0].ldk * sizeof(float) > (size_t)GRIFFIN_STATIC_SCRATCH_BYTES)
        return GRIFFIN_ERR_UNSUPPORTED;
    unsigned char *base = static_scratch_of_current_device();
    if (base == nullptr) return GRIFFIN_ERR_CUDA;
    // same launcher as the workspace variant: header first, z behind it
    return launch_decode(desc, B, sets, b_down, x, y, reinterpret_cast<float *>(base + 256), base, flags, stream);
}

}  // namespace griffin
