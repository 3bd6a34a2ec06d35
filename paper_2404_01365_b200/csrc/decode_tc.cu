// Generation-phase pruned FF (Eqs. 4 and 5 of the GRIFFIN paper) for bf16 storage on the
// 5th-generation tensor cores, as ONE kernel per call:
//   first half   z_hat = sigma(W_g_hat x + b_g_hat) * (W_1_hat x + b_1_hat)
//   meeting      every CTA has written its z entries; all CTAs wait for each other (bounded)
//   second half  y_hat = W_2_hat z_hat + b_2
//
// The products are matrix-vector products, bound by the HBM stream of the weights.  What the
// tensor cores buy here is not FLOPs: tcgen05.mma reads its operands from shared memory by
// itself, so the bytes that the copy engine lands are multiplied without a single load,
// unpack or FMA instruction in any warp, and one thread issues everything.
//
// One persistent CTA per SM, 192 threads in three roles:
//   warp 0      producer: 1-D bulk copies (TMA, no multicast) of pieces of weight rows into
//               a ring of shared-memory stages.  Weights only, so it runs ahead of the
//               previous kernel on the stream (programmatic dependent launch) and of the
//               meeting point.
//   warp 1      MMA issuer (one thread) and owner of the TMEM allocation.
//   warps 2-5   vector staging (x, then z), epilogues, the meeting point.
//
// How contiguous rows are fed to an M = 128, N = 16, K = 16 MMA without rearranging a byte:
//   * The canonical K-major operand layout WITHOUT swizzle is made of "core matrices" of 8
//     rows x 16 bytes stored as 128 contiguous bytes.  Read the other way round, 128
//     contiguous bytes of a weight row ARE a core matrix: its 8 rows are the row's eight
//     consecutive 16-byte units.  The second core matrix of a K = 16 step lies 128 bytes
//     further (leading byte offset), and the next group of 8 MMA rows is the next weight row
//     (stride byte offset = the distance between staged rows).  One MMA thus takes a "window"
//     of 256 bytes (128 elements) of up to 16 weight rows: MMA row 8 r + i is unit i (and
//     unit 8 + i) of weight row r.
//   * The vector is described in exactly the same way: B row n is unit n (and 8 + n) of the
//     matching 256-byte window of x, and in the second half B rows 8..15 are the units of
//     z_lo (z crosses the halves as two bf16 numbers z_hi + z_lo per entry, so 16 bits of z
//     survive; same scratch layout as the warp-level kernel).
//   * D[8 r + i][n] pairs unit i of the weight row with unit n of the vector: the dot product
//     of the window is the diagonal i = n (plus n = 8 + i for z_lo).  The epilogue thread that
//     owns TMEM lane 8 r + i reads columns i and 8 + i, and three shuffles add the 8 lanes of
//     a weight row.  Everything else in D is computed and never read, which is free here.
//   * A stage holds one piece (at most a few KB per row) of the S rows of a "set" (S = 8 or
//     16 consecutive rows of the work item); every set has its own 16 accumulator columns.
//     Rows of A beyond the set only reach accumulator lanes that nobody reads.
//
// Every wait is bounded; after a give-up every role leaves its loops, the producer waits
// (bounded) for its copies in flight and the CTA frees its TMEM before it returns.
#include "decode_common.cuh"
#include "tc_common.cuh"

namespace griffin {

constexpr int DTC_THREADS = 192;
constexpr int DTC_EPI_THREADS = 128;
constexpr int DTC_WINDOW = 256;            // bytes of a row that one MMA takes (two K steps of 8 units)
constexpr int DTC_SLOT_BYTES = 32 * 1024;  // one stage of the ring
constexpr int DTC_MAX_STAGES = 7;
constexpr int DTC_MAX_SETS = 16;           // sets per work item (128 rows of 8)
constexpr int DTC_TMEM_COLS = 512;         // 32 accumulators of 16 columns
constexpr int DTC_STAGING_DEPTH_SHARED = 32;  // 16-byte loads a thread keeps in flight while it stages the up to 8 vectors that share a set
constexpr int DTC_MAX_VEC = 8;             // vectors that may share one expert set in a call
#ifndef GRIFFIN_DTC_SET_ROWS_0
#define GRIFFIN_DTC_SET_ROWS_0 16
#endif
#ifndef GRIFFIN_DTC_SET_ROWS_1
#define GRIFFIN_DTC_SET_ROWS_1 16
#endif

struct DtcHalf {
    int n_rows;    // rows of the matrix (k, or d)
    int n_slices;  // work items per sequence
    int set_rows;  // weight rows per MMA (8 or 16)
    int windows;   // 256-byte windows of a row
    int n_chunks;  // pieces a row is cut into (one per stage)
    int wpc;       // windows per piece (the last may be shorter)
    int sbo_b;     // bytes from the vector to its second copy (z_lo), 0 if there is none
    int n_acc;     // accumulators per set (a power of two), taken in turn by the windows of a row
    int acc_cols;  // columns of one accumulator = N of the MMA: 8 per group of B rows, at least 16
};
struct DtcPlan {
    DtcHalf h[2];
    int n_stages;
    int vec_bytes;   // shared memory set aside for the vector(s)
    int n_vec;       // 1: every sequence has its own expert set; B: one set for the B vectors of the call
    int vec_stride;  // bytes between the vectors in shared memory (n_vec > 1)
};

struct DtcSmem {
    uint8_t *ring, *vec;
    float *part;  // [DTC_MAX_VEC][DTC_MAX_SETS * 16]
    uint64_t *full, *empty, *vec_full, *acc_full;
    uint32_t *tmem_slot;
    volatile int *abort;
};
// An MMA always reads 16 staged rows: with sets of 8 rows the other 8 lie beyond the stage, so
// what follows the ring must be at least that long (what is read there is never used).
static size_t dtc_smem_bytes(const DtcPlan &pl) {
    size_t tail = pl.vec_bytes + DTC_MAX_VEC * DTC_MAX_SETS * 16 * sizeof(float) + (2 * DTC_MAX_STAGES + 2) * sizeof(uint64_t) + 16;
    for (int i = 0; i < 2; ++i) {
        const size_t beyond = (size_t)(16 - pl.h[i].set_rows) * pl.h[i].wpc * DTC_WINDOW;
        if (beyond > tail) tail = beyond;
    }
    return 1024 + (size_t)pl.n_stages * DTC_SLOT_BYTES + tail;
}

// Descriptor of a K-major operand without swizzle: core matrices of 8 rows x 16 bytes (128
// contiguous bytes); lbo = bytes between the two core matrices of a K = 16 step, sbo = bytes
// between groups of 8 rows.
__device__ __forceinline__ uint64_t smem_desc_plain(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// 32 lanes x 16 columns of fp32: thread i of the warp receives row (lane base + i)
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// D[tmem] += A[smem] * B[smem]
__device__ __forceinline__ void umma_bf16_acc(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.eq.u32 p, 1, 1;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc)
        : "memory");
}
// Barrier among the 128 epilogue threads that also ORs a flag, so that all of them take the
// same way out after a give-up.
__device__ __forceinline__ bool epi_barrier_or(bool flag) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)flag)
        : "memory");
    return r != 0;
}

// Rows [r0, r1) of work item `sl` (the same split as the other decode kernels).
__device__ __forceinline__ void dtc_item_rows(const DtcHalf &h, int sl, int &r0, int &r1) {
    r0 = (int)((long long)sl * h.n_rows / h.n_slices);
    r1 = (int)((long long)(sl + 1) * h.n_rows / h.n_slices);
}

// Issuing an MMA keeps the issuing thread busy for about as long as the MMA keeps the tensor
// core busy, and every instruction between two MMAs adds to that: the windows of a piece are
// therefore issued in batches of eight with every offset a compile-time constant.  Window j of
// a batch goes to accumulator j % NACC of the set (an MMA into the accumulator of the one just
// before it would wait for its result); the batch starts at a multiple of 8 windows of the
// row, so this is also the window's number in the row modulo NACC.
//   first : these are the first windows of the row (accumulators 0 .. NACC-1 are overwritten)
template <int NACC>
__device__ __forceinline__ void mma_batch8(const uint32_t (&dacc)[NACC], uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                           bool first) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t d = dacc[j % NACC];
        const uint64_t a = a_desc + (uint64_t)(j * (DTC_WINDOW >> 4)), b = b_desc + (uint64_t)(j * (DTC_WINDOW >> 4));
        if (j < NACC)
            umma_bf16(d, a, b, idesc, first ? 0u : 1u);
        else
            umma_bf16_acc(d, a, b, idesc);
    }
}

// The MMA issuer's part of one half.  Returns false after a give-up.
template <int NACC>
__device__ __forceinline__ bool dtc_issue_half(const DecodeParams &p, const DtcPlan &pl, const DtcSmem &s, int half,
                                               uint32_t tmem_base, uint32_t &it, uint32_t &n_item) {
    const DtcHalf h = half ? pl.h[1] : pl.h[0];  // (a copy in registers: the asm statements below clobber memory)
    const uint32_t IDESC = umma_idesc(128, h.acc_cols);
    const int n_stages = pl.n_stages;
    const int n_items = (pl.n_vec > 1 ? 1 : p.B) * h.n_slices;
    const uint32_t piece_max = (uint32_t)h.wpc * DTC_WINDOW;
    const uint64_t a_desc0 = smem_desc_plain(smem_u32(s.ring), 128u, piece_max);
    const uint64_t b_desc0 = smem_desc_plain(smem_u32(s.vec), 128u, (uint32_t)h.sbo_b);
    int stage = (int)(it % (uint32_t)n_stages);
    uint32_t round = it / (uint32_t)n_stages;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n_item) {
        const int sl = item % h.n_slices;
        int r0, r1;
        dtc_item_rows(h, sl, r0, r1);
        const int n_rows_item = half ? r1 - r0 : 2 * (r1 - r0);
        // the vector is in place, and the previous item's accumulators have been read
        if (!wait_or_abort(s.vec_full, n_item & 1, s.abort, p.ws, 32 + half)) return false;
        tc_fence_after_sync();
        uint32_t d_set = tmem_base;
        for (int row_s = 0; row_s < n_rows_item; row_s += h.set_rows, d_set += NACC * (uint32_t)h.acc_cols) {
            uint32_t dacc[NACC];
#pragma unroll
            for (int a = 0; a < NACC; ++a) dacc[a] = d_set + (uint32_t)(a * h.acc_cols);
            for (int c = 0; c < h.n_chunks; ++c, ++it) {
                if (!wait_or_abort(&s.full[stage], round & 1, s.abort, p.ws, 34 + half)) return false;
                tc_fence_after_sync();
                const int nw = min(h.wpc, h.windows - c * h.wpc);
                // (a window further = 16 in the address field of the descriptor's low word)
                uint64_t a_desc = a_desc0 + (uint64_t)((uint32_t)stage * (DTC_SLOT_BYTES >> 4));
                uint64_t b_desc = b_desc0 + (uint64_t)((uint32_t)(c * h.wpc) * (DTC_WINDOW >> 4));
                int w = 0;
                for (; w + 8 <= nw; w += 8) {
                    mma_batch8<NACC>(dacc, a_desc, b_desc, IDESC, c == 0 && w == 0);
                    a_desc += 8 * (DTC_WINDOW >> 4);
                    b_desc += 8 * (DTC_WINDOW >> 4);
                }
                for (int j = 0; w < nw; ++w, ++j)  // what is left of the row's last piece
                    umma_bf16(d_set + (uint32_t)((j % NACC) * h.acc_cols), a_desc + (uint64_t)(j * (DTC_WINDOW >> 4)),
                              b_desc + (uint64_t)(j * (DTC_WINDOW >> 4)), IDESC, (c * h.wpc + w) >= NACC ? 1u : 0u);
                umma_commit(&s.empty[stage]);  // the stage may be refilled once these MMAs have read it
                if (++stage == n_stages) {
                    stage = 0;
                    ++round;
                }
            }
        }
        umma_commit(s.acc_full);
    }
    return true;
}

// SHARED: one expert set for all the vectors of the call (see decode_tc_shared); otherwise one
// vector per work item.
template <bool SHARED>
__global__ void __launch_bounds__(DTC_THREADS, 1) decode_tc_kernel(const __grid_constant__ DecodeParams p,
                                                                const __grid_constant__ DtcPlan pl, int act) {
    extern __shared__ uint8_t smem_raw[];
    DtcSmem s;
    s.ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    s.vec = s.ring + (size_t)pl.n_stages * DTC_SLOT_BYTES;
    s.part = reinterpret_cast<float *>(s.vec + pl.vec_bytes);
    s.full = reinterpret_cast<uint64_t *>(s.part + DTC_MAX_VEC * DTC_MAX_SETS * 16);
    s.empty = s.full + DTC_MAX_STAGES;
    s.vec_full = s.empty + DTC_MAX_STAGES;
    s.acc_full = s.vec_full + 1;
    s.tmem_slot = reinterpret_cast<uint32_t *>(s.acc_full + 1);
    s.abort = reinterpret_cast<volatile int *>(s.tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < pl.n_stages; ++i) {
            mbar_init(&s.full[i], 1);
            mbar_init(&s.empty[i], 1);
        }
        mbar_init(s.vec_full, 1);
        mbar_init(s.acc_full, 1);
        *s.abort = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(s.tmem_slot, DTC_TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();
    const uint32_t tmem_base = *s.tmem_slot;

    if (warp == 0) {
        // ---------------- producer: lane l copies row l of the set ----------------
        uint32_t it = 0;
        bool ok = true;
        for (int half = 0; ok && half < 2; ++half) {
            const DtcHalf h = half ? pl.h[1] : pl.h[0];  // (a copy in registers: the asm statements below clobber memory)
            const int n_items = (pl.n_vec > 1 ? 1 : p.B) * h.n_slices;  // (one shared set: the slices of that one set)
            const size_t row_bytes = (size_t)h.windows * DTC_WINDOW;
            const uint32_t piece_max = (uint32_t)h.wpc * DTC_WINDOW;
            for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
                const int b = item / h.n_slices, sl = item - b * h.n_slices;
                int r0, r1;
                dtc_item_rows(h, sl, r0, r1);
                const int n_rows_item = half ? r1 - r0 : 2 * (r1 - r0);  // first half: gate rows, then up rows
                for (int row_s = 0; ok && row_s < n_rows_item; row_s += h.set_rows) {
                    const int rows_here = min(h.set_rows, n_rows_item - row_s);
                    const int idx = row_s + lane;  // this lane's row of the item
                    const uint8_t *src = nullptr;
                    if (lane < rows_here) {
                        if (half) {
                            src = static_cast<const uint8_t *>(p.seq[b].w_down) + (size_t)(r0 + idx) * row_bytes;
                        } else {
                            const int R = r1 - r0;
                            src = static_cast<const uint8_t *>(idx < R ? p.seq[b].w_gate : p.seq[b].w_up) +
                                  (size_t)(r0 + (idx < R ? idx : idx - R)) * row_bytes;
                        }
                    }
                    for (int c = 0; c < h.n_chunks; ++c, ++it) {
                        const int stage = it % pl.n_stages;
                        const uint32_t use = it / pl.n_stages;
                        const uint32_t bytes = (uint32_t)min(h.wpc, h.windows - c * h.wpc) * DTC_WINDOW;
                        int go = 1;
                        if (lane == 0) {
                            if (use > 0 && !wait_or_abort(&s.empty[stage], (use - 1) & 1, s.abort, p.ws, 30 + half)) go = 0;
                            if (go) mbar_arrive_expect_tx(&s.full[stage], (uint32_t)rows_here * bytes);
                        }
                        go = __shfl_sync(0xffffffffu, go, 0);
                        if (!go) {
                            ok = false;
                            break;
                        }
                        if (src != nullptr)
                            bulk_g2s(s.ring + (size_t)stage * DTC_SLOT_BYTES + (size_t)lane * piece_max,
                                     src + (size_t)c * piece_max, bytes, &s.full[stage]);
                    }
                }
            }
        }
        if (lane == 0) {  // stay until every copy that was started has landed
            const uint32_t first = it > (uint32_t)pl.n_stages ? it - pl.n_stages : 0;
            for (uint32_t j = first; j < it; ++j) {
                const long long t0 = clock64();
                while (!mbar_try_wait(&s.full[j % pl.n_stages], (j / pl.n_stages) & 1))
                    if (clock64() - t0 > WAIT_LIMIT_CYCLES) break;
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            uint32_t it = 0, n_item = 0;
            bool ok = true;
            for (int half = 0; ok && half < 2; ++half) {
                switch (pl.h[half].n_acc) {  // (a compile-time constant inside: see mma_batch8)
                    case 8: ok = dtc_issue_half<8>(p, pl, s, half, tmem_base, it, n_item); break;
                    case 4: ok = dtc_issue_half<4>(p, pl, s, half, tmem_base, it, n_item); break;
                    case 2: ok = dtc_issue_half<2>(p, pl, s, half, tmem_base, it, n_item); break;
                    default: ok = dtc_issue_half<1>(p, pl, s, half, tmem_base, it, n_item); break;
                }
            }
        }
    } else {
        // ---------------- vector staging, epilogue, meeting (warps 2..5) ----------------
        const int et = tid - 64;       // 0..127
        const int wq = warp & 3;       // the TMEM lane quarter this warp may read
        const int m = wq * 32 + lane;  // TMEM lane = 8 * (row of the set) + unit
        const int unit = m & 7, row_in_set = m >> 3;
        __nv_bfloat16 *zbits = reinterpret_cast<__nv_bfloat16 *>(p.z);
        pdl_wait_prior_grids();  // x, the z scratch and the outputs belong to earlier work on the stream
        uint32_t n_item = 0;
        bool stop = false;
        for (int half = 0; !stop && half < 2; ++half) {
            const DtcHalf h = half ? pl.h[1] : pl.h[0];  // (a copy in registers: the asm statements below clobber memory)
            const int n_vec = pl.n_vec;                    // vectors that meet every staged row
            const int n_groups = n_vec > 1 ? n_vec : (half ? 2 : 1);  // groups of 8 B rows with data: vectors, or z_hi and z_lo
            const int n_items = (n_vec > 1 ? 1 : p.B) * h.n_slices;
            int cur_b = -1;
            for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n_item) {
                const int b = item / h.n_slices, sl = item - b * h.n_slices;
                int r0, r1;
                dtc_item_rows(h, sl, r0, r1);
                const int R = r1 - r0;
                const int n_rows_item = half ? R : 2 * R;
                const int n_sets = (n_rows_item + h.set_rows - 1) / h.set_rows;
                if constexpr (!SHARED) {
                if (b != cur_b) {
                    // the vector, read through L2 (x comes from earlier work on the stream, z from
                    // other CTAs of this grid): x, or z_hi then z_lo, as they lie in memory
                    const int n_units = h.windows * (DTC_WINDOW / 16) * (half ? 2 : 1);
                    const uint4 *src = half ? reinterpret_cast<const uint4 *>(zbits + (size_t)b * 2 * p.ldk)
                                            : reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(p.x) +
                                                                              (size_t)b * p.d);
                    uint4 *dst = reinterpret_cast<uint4 *>(s.vec);
                    for (int u0 = et; u0 < n_units; u0 += 4 * DTC_EPI_THREADS) {
                        uint4 v[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {  // all loads of a round are in flight together
                            const int u = u0 + j * DTC_EPI_THREADS;
                            v[j] = u < n_units ? __ldcg(src + u) : make_uint4(0, 0, 0, 0);
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int u = u0 + j * DTC_EPI_THREADS;
                            if (u < n_units) dst[u] = v[j];
                        }
                    }
                    fence_proxy_async_smem();  // the MMA reads shared memory through the async proxy
                    cur_b = b;
                }
                tc_fence_before_sync();
                if (epi_barrier_or(*s.abort != 0)) {
                    stop = true;
                    break;
                }
                if (et == 0) mbar_arrive(s.vec_full);
                const bool got = __all_sync(
                    0xffffffffu, wait_or_abort_relaxed(s.acc_full, n_item & 1, s.abort, p.ws, 36 + half));  // (tcgen05.ld is warp-wide)
                tc_fence_after_sync();
                if (got) {
                    const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16);
#pragma unroll 1
                    for (int set = 0; set < n_sets; ++set) {
                        float val = 0.f;
                        for (int a = 0; a < h.n_acc; ++a) {  // (a fixed order: results are reproducible)
                            float v[16];
                            tmem_ld16(taddr + (uint32_t)(set * h.n_acc + a) * 16u, v);
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                if (c == unit) val += half ? v[c] + v[8 + c] : v[c];
                        }
                        // the 8 units of a weight row sit in 8 consecutive lanes
                        val += __shfl_xor_sync(0xffffffffu, val, 1);
                        val += __shfl_xor_sync(0xffffffffu, val, 2);
                        val += __shfl_xor_sync(0xffffffffu, val, 4);
                        if (unit == 0) s.part[set * 16 + row_in_set] = val;
                    }
                }
                tc_fence_before_sync();
                if (epi_barrier_or(!got)) {
                    stop = true;
                    break;
                }
                // thread t finishes row r0 + t of the item
                if (et < R) {
                    const int row = r0 + et;
                    if (!half) {
                        const int iu = R + et;  // the up row's place in the item
                        float a0 = s.part[(et / h.set_rows) * 16 + et % h.set_rows];
                        float a1 = s.part[(iu / h.set_rows) * 16 + iu % h.set_rows];
                        if (p.seq[b].b_gate) a0 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[b].b_gate)[row]);
                        if (p.seq[b].b_up) a1 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[b].b_up)[row]);
                        const float zv = sigma_rt(act, a0) * a1;
                        const __nv_bfloat16 hi = __float2bfloat16_rn(zv);
                        zbits[(size_t)b * 2 * p.ldk + row] = hi;
                        zbits[(size_t)b * 2 * p.ldk + p.ldk + row] = __float2bfloat16_rn(zv - __bfloat162float(hi));
                    } else {
                        float acc = s.part[(et / h.set_rows) * 16 + et % h.set_rows];
                        if (p.b_down) acc += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.b_down)[row]);
                        static_cast<__nv_bfloat16 *>(p.y)[(size_t)b * p.d + row] = __float2bfloat16_rn(acc);
                    }
                }
                if (!half && sl == h.n_slices - 1)  // the last slice also clears the padding of z
                    for (int j = p.k + et; j < p.ldk; j += DTC_EPI_THREADS) {
                        zbits[(size_t)b * 2 * p.ldk + j] = __float2bfloat16_rn(0.f);
                        zbits[(size_t)b * 2 * p.ldk + p.ldk + j] = __float2bfloat16_rn(0.f);
                    }
                } else {
                if (b != cur_b) {
                    // the vector(s), read through L2 (x comes from earlier work on the stream, z from
                    // other CTAs of this grid).  One vector: x, or z_hi then z_lo, as they lie in
                    // memory.  A shared set: x (or z_hi) of every sequence, vec_stride bytes apart.
                    const int row_units = h.windows * (DTC_WINDOW / 16);
                    const int n_units = n_vec > 1 ? row_units : row_units * (half ? 2 : 1);
                    // (plain loads: a bulk copy would queue behind the producer's weight copies; the
                    // units of all vectors are shared out together so that many loads are in flight)
                    const size_t src_stride = half ? (size_t)2 * p.ldk * 2 : (size_t)p.d * 2;  // bytes between sequences
                    const uint8_t *src0 = half ? reinterpret_cast<const uint8_t *>(zbits) : static_cast<const uint8_t *>(p.x);
                    const int total = n_vec * n_units;
                    for (int e0 = et; e0 < total; e0 += DTC_STAGING_DEPTH_SHARED * DTC_EPI_THREADS) {
                        uint4 t[DTC_STAGING_DEPTH_SHARED];
                        int v = e0 / n_units, u = e0 - v * n_units;  // (vector, unit) of this thread's first load of the round
                        const int v0 = v, u0 = u;
#pragma unroll
                        for (int j = 0; j < DTC_STAGING_DEPTH_SHARED; ++j) {  // all loads of a round are in flight together
                            t[j] = e0 + j * DTC_EPI_THREADS < total
                                       ? __ldcg(reinterpret_cast<const uint4 *>(src0 + (size_t)v * src_stride) + u)
                                       : make_uint4(0, 0, 0, 0);
                            for (u += DTC_EPI_THREADS; u >= n_units; u -= n_units) ++v;
                        }
                        v = v0, u = u0;
#pragma unroll
                        for (int j = 0; j < DTC_STAGING_DEPTH_SHARED; ++j) {
                            if (e0 + j * DTC_EPI_THREADS < total) reinterpret_cast<uint4 *>(s.vec + (size_t)v * pl.vec_stride)[u] = t[j];
                            for (u += DTC_EPI_THREADS; u >= n_units; u -= n_units) ++v;
                        }
                    }
                    fence_proxy_async_smem();  // the MMA reads shared memory through the async proxy
                    cur_b = b;
                }
                tc_fence_before_sync();
                if (epi_barrier_or(*s.abort != 0)) {
                    stop = true;
                    break;
                }
                if (et == 0) mbar_arrive(s.vec_full);
                const bool got = __all_sync(
                    0xffffffffu, wait_or_abort_relaxed(s.acc_full, n_item & 1, s.abort, p.ws, 36 + half));  // (tcgen05.ld is warp-wide)
                tc_fence_after_sync();
                if (got) {
                    const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16);
#pragma unroll 1
                    for (int set = 0; set < n_sets; ++set) {
                        float val[DTC_MAX_VEC];  // per group of B rows: this lane's diagonal entry
#pragma unroll
                        for (int g = 0; g < DTC_MAX_VEC; ++g) val[g] = 0.f;
                        for (int a = 0; a < h.n_acc; ++a) {  // (a fixed order: results are reproducible)
                            const uint32_t acc_addr = taddr + (uint32_t)((set * h.n_acc + a) * h.acc_cols);
#pragma unroll
                            for (int g2 = 0; g2 < DTC_MAX_VEC / 2; ++g2) {  // 16 columns = two groups at a time
                                if (2 * g2 < n_groups) {               // warp-uniform
                                    float t[16];
                                    tmem_ld16(acc_addr + (uint32_t)g2 * 16u, t);
#pragma unroll
                                    for (int c = 0; c < 8; ++c)
                                        if (c == unit) {
                                            val[2 * g2] += t[c];
                                            if (2 * g2 + 1 < n_groups) val[2 * g2 + 1] += t[8 + c];
                                        }
                                }
                            }
                        }
                        if (n_vec == 1 && half) val[0] += val[1];  // z_hi and z_lo belong to the same output
#pragma unroll
                        for (int g = 0; g < DTC_MAX_VEC; ++g)
                            if (g < n_vec) {  // the 8 units of a weight row sit in 8 consecutive lanes
                                float t = val[g];
                                t += __shfl_xor_sync(0xffffffffu, t, 1);
                                t += __shfl_xor_sync(0xffffffffu, t, 2);
                                t += __shfl_xor_sync(0xffffffffu, t, 4);
                                if (unit == 0) s.part[g * (DTC_MAX_SETS * 16) + set * 16 + row_in_set] = t;
                            }
                    }
                }
                tc_fence_before_sync();
                if (epi_barrier_or(!got)) {
                    stop = true;
                    break;
                }
                // the (vector, row) results of the item are shared out among the threads
                for (int task = et; task < n_vec * R; task += DTC_EPI_THREADS) {
                    const int v = task / R, rr = task - v * R;
                    const int row = r0 + rr;
                    const int ig = (rr / h.set_rows) * 16 + rr % h.set_rows;  // where the (gate) row's result is
                    {
                        const int seq = n_vec > 1 ? v : b;
                        const float *part = s.part + v * (DTC_MAX_SETS * 16);
                        if (!half) {
                            const int iu = R + rr;  // the up row's place in the item
                            float a0 = part[ig];
                            float a1 = part[(iu / h.set_rows) * 16 + iu % h.set_rows];
                            if (p.seq[b].b_gate) a0 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[b].b_gate)[row]);
                            if (p.seq[b].b_up) a1 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[b].b_up)[row]);
                            const float zv = sigma_rt(act, a0) * a1;
                            const __nv_bfloat16 hi = __float2bfloat16_rn(zv);
                            zbits[(size_t)seq * 2 * p.ldk + row] = hi;
                            if (n_vec == 1) zbits[(size_t)seq * 2 * p.ldk + p.ldk + row] = __float2bfloat16_rn(zv - __bfloat162float(hi));
                        } else {
                            float acc = part[ig];
                            if (p.b_down) acc += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.b_down)[row]);
                            static_cast<__nv_bfloat16 *>(p.y)[(size_t)seq * p.d + row] = __float2bfloat16_rn(acc);
                        }
                    }
                }
                if (!half && sl == h.n_slices - 1)  // the last slice also clears the padding of z
                    for (int v = 0; v < n_vec; ++v) {
                        const int seq = n_vec > 1 ? v : b;
                        for (int j = p.k + et; j < p.ldk; j += DTC_EPI_THREADS) {
                            zbits[(size_t)seq * 2 * p.ldk + j] = __float2bfloat16_rn(0.f);
                            zbits[(size_t)seq * 2 * p.ldk + p.ldk + j] = __float2bfloat16_rn(0.f);
                        }
                    }
                }
            }
            if (half == 0) {
                // ---- the meeting point: this CTA's z entries are written; the thread that reports in makes them visible.
                // (`stop` is the same in every epilogue thread: it only changes behind epi_barrier_or.)  After a give-up
                // the CTA still reports in, without waiting: the counter runs round modulo twice the number of
                // CTAs and is never reset, so every CTA must add exactly one arrival per launch, or every later
                // call on this workspace would meet out of phase.
                if (stop) {
                    if (et == 0) grid_arrive_only(&static_cast<WsHeader *>(p.ws)->meet_tc, gridDim.x);
                } else {
                    bool bad = epi_barrier_or(false);
                    if (et == 0) bad = !grid_meet(&static_cast<WsHeader *>(p.ws)->meet_tc, gridDim.x, s.abort, p.ws);
                    if (epi_barrier_or(bad)) stop = true;
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, DTC_TMEM_COLS);
}

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
bool decode_tc_supported(const DecodeParams &p) {
    if (p.B < 1 || p.ws == nullptr) return false;
    // whole 256-byte windows (the bytes after a shorter row would be multiplied too)
    if (p.d % 128 != 0 || p.ldk % 128 != 0 || p.d > GRIFFIN_MAX_D) return false;
    if ((size_t)p.ldk * 4 > 48 * 1024) return false;  // the vector must leave room for the ring
    for (int b = 0; b < p.B; ++b)
        if ((reinterpret_cast<uintptr_t>(p.seq[b].w_gate) | reinterpret_cast<uintptr_t>(p.seq[b].w_up) |
             reinterpret_cast<uintptr_t>(p.seq[b].w_down)) & 15)
            return false;
    return true;
}

// One expert set for all the sequences of the call (entries of `sets` that all name the same
// buffers): the weights are streamed once and every staged row meets all B vectors in one MMA.
bool decode_tc_shared(const DecodeParams &p) {
    if (p.B < 2 || p.B > DTC_MAX_VEC || !decode_tc_supported(p)) return false;
    for (int b = 1; b < p.B; ++b)
        if (p.seq[b].w_gate != p.seq[0].w_gate || p.seq[b].w_up != p.seq[0].w_up || p.seq[b].w_down != p.seq[0].w_down ||
            p.seq[b].b_gate != p.seq[0].b_gate || p.seq[b].b_up != p.seq[0].b_up)
            return false;
    const int groups = ((8 * p.B + 15) / 16) * 2;
    const size_t stride = ((size_t)max(p.d, p.ldk) * 2 + 255) & ~(size_t)255;
    return groups * stride <= 112 * 1024;  // the vectors must leave room for a ring of three stages
}

static void dtc_plan_half(DtcHalf &h, int n_rows, int mats, int row_elems, int set_rows, int acc_cols, int sms) {
    h.n_rows = n_rows;
    h.n_slices = slices_for(n_rows, sms);
    h.set_rows = set_rows;
    h.windows = row_elems * 2 / DTC_WINDOW;
    h.wpc = DTC_SLOT_BYTES / set_rows / DTC_WINDOW;  // what a stage can hold per row: 8 or 16 windows
    h.n_chunks = (h.windows + h.wpc - 1) / h.wpc;
    h.sbo_b = 0;
    // all sets of the largest item keep their accumulators until its epilogue
    const int rows_max = (n_rows + h.n_slices - 1) / h.n_slices;
    const int sets_max = (rows_max * mats + set_rows - 1) / set_rows;
    h.acc_cols = acc_cols;
    h.n_acc = 8;
    while (h.n_acc > 1 && (sets_max * h.n_acc * acc_cols > DTC_TMEM_COLS || h.n_acc > h.windows)) h.n_acc >>= 1;  // (each is written at least once)
}

griffin_status decode_bf16_tc(DecodeParams &p, int act, uint32_t flags, cudaStream_t stream) {
    const int sms = device_sm_count();
    if (sms <= 0) return GRIFFIN_ERR_CUDA;
    if (!decode_tc_supported(p)) return GRIFFIN_ERR_UNSUPPORTED;
    const bool overlap = (flags & GRIFFIN_DECODE_OVERLAP_WEIGHT_PREFETCH) != 0;
    DtcPlan pl;
    const bool shared = decode_tc_shared(p);
    pl.n_vec = shared ? p.B : 1;
    pl.vec_stride = (max(p.d, p.ldk) * 2 + 255) & ~255;
    const int acc_cols = shared ? ((8 * p.B + 15) / 16) * 16 : 16;
    dtc_plan_half(pl.h[0], p.k, 2, p.d, GRIFFIN_DTC_SET_ROWS_0, acc_cols, sms);
    dtc_plan_half(pl.h[1], p.d, 1, p.ldk, GRIFFIN_DTC_SET_ROWS_1, acc_cols, sms);
    if (shared) {
        pl.h[0].sbo_b = pl.h[1].sbo_b = pl.vec_stride;  // the next 8 rows of B are the next vector
        pl.vec_bytes = (acc_cols / 8) * pl.vec_stride;   // (an odd number of vectors: the MMA reads one more, unused)
    } else {
        pl.h[1].sbo_b = p.ldk * 2;  // z_lo lies behind z_hi
        pl.vec_bytes = (max(p.d * 2, p.ldk * 4) + 127) & ~127;
    }
    // every set of the largest item keeps its accumulators until the item's epilogue
    for (int i = 0; i < 2; ++i)
        if (((pl.h[i].n_rows + pl.h[i].n_slices - 1) / pl.h[i].n_slices * (i ? 1 : 2) + pl.h[i].set_rows - 1) / pl.h[i].set_rows *
                pl.h[i].n_acc * acc_cols > DTC_TMEM_COLS)
            return GRIFFIN_ERR_UNSUPPORTED;
    pl.n_stages = 0;
    for (int n = DTC_MAX_STAGES; n >= 2; --n) {
        pl.n_stages = n;
        if (dtc_smem_bytes(pl) <= 227 * 1024) break;
    }
    const size_t smem = dtc_smem_bytes(pl);
    if (smem > 227 * 1024) return GRIFFIN_ERR_UNSUPPORTED;
    // every CTA of the grid must be able to run at the same time (they meet half-way): one per SM
    const void *fn = shared ? (const void *)decode_tc_kernel<true> : (const void *)decode_tc_kernel<false>;
    if (ensure_dynamic_smem(fn, smem) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    if (!grid_can_meet(fn, DTC_THREADS, smem, sms)) return GRIFFIN_ERR_UNSUPPORTED;
    void *args[] = {&p, &pl, &act};
    if (launch_maybe_overlapped(fn, dim3(sms), dim3(DTC_THREADS), smem, stream, overlap, args) != cudaSuccess)
        return GRIFFIN_ERR_CUDA;
    return GRIFFIN_OK;
}

}  // namespace griffin
