// Prompt-phase FF on the 5th-generation tensor cores with PAIRS of SMs on one tile (Eqs. 1 and 3 of the
// GRIFFIN paper), bf16 storage, fp32 accumulation.  Same three kernels as prefill_tc.cu (gated first GEMM,
// first GEMM without a gate, down projection with 256-wide tiles) and the same epilogues; what differs is the
// main loop: two CTAs of a cluster share a tile of 256 tokens x 256 columns through tcgen05.mma.cta_group::2.
//
// Why: with one CTA per 128 x 256 tile a K step of 64 needs 48 KB from L2 (16 KB of the left operand, 32 KB
// of weights) for 4.2 MFLOP, and the SM's path from L2 into shared memory, not the tensor core, set the pace
// (measured: the tile stream alone took 56 of the first GEMM's 76 us on the Llama-2-7B shape at 512 tokens).
// In a pair each CTA stages its own 128 tokens and only HALF of the weight tile -- 32 KB per K step for the
// same flops -- and the MMA reads both halves.
//
// The pair (cluster of 2; rank 0 is the leader):
//   warp 0 of both   TMA producer: cp.async.bulk.tensor (2-D, 128-byte swizzle, no multicast) of this CTA's
//                    128 x 64 tile of the left operand and of its 128 x 64 half of the weight tile into its
//                    OWN shared memory; the bytes are counted on the LEADER's full barrier of the stage, which
//                    the leader's producer arms for both CTAs' bytes.  Each producer waits on its own CTA's
//                    empty barrier.
//   warp 1, leader   MMA issuer: tcgen05.mma.cta_group::2 (M = 256, N = 256, K = 16); the accumulator rows of
//                    the first 128 tokens land in the leader's TMEM, the others in the follower's.  A stage is
//                    released by one tcgen05.commit per CTA (its own barrier and, through its address in the
//                    cluster's shared window, the follower's), an accumulator stage is announced the same way.
//   warp 1, both     owns the TMEM allocation (tcgen05.alloc.cta_group::2, issued by both CTAs).
//   warps 2-9, both  epilogue of the CTA's own 128 rows from its own TMEM, exactly as with one CTA per tile;
//                    an accumulator stage is handed back on the leader's barrier (16 arrivals: the follower's
//                    warps arrive through the cluster's shared window).
// Every wait on a barrier is bounded; the two cluster-wide barriers (after set-up, so that no CTA touches a
// peer's barrier before it is initialised, and before TMEM is freed, so that no CTA leaves while its peer may
// still read its shared memory or write its TMEM) are reached by every thread of both CTAs on every path.
#include "prefill_tc.cuh"

namespace griffin {

#ifndef GRIFFIN_TC2_STAGES
#define GRIFFIN_TC2_STAGES 6
#endif
constexpr int TC2_STAGES = GRIFFIN_TC2_STAGES;
constexpr int TC2_NT = 256;                                  // columns of the pair's tile = TMEM columns of a stage
constexpr int TC2_A_BYTES = TC_BM * TC_BK * 2;               // this CTA's 128 rows of the left operand: 16 KB
constexpr int TC2_B_BYTES = (TC2_NT / 2) * TC_BK * 2;        // this CTA's half of the weight tile: 16 KB
constexpr int TC2_STAGE_BYTES = TC2_A_BYTES + TC2_B_BYTES;   // per CTA
constexpr size_t TC2_TAIL_BYTES = (2 * TC2_STAGES + 4) * sizeof(uint64_t) + 16 + TC_EPI_WARPS * TC_STG_BYTES;

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory location in the CTA of the given rank, in the cluster's shared window
__device__ __forceinline__ uint32_t map_to_rank(const void *p, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load of a CTA of a pair: into its own shared memory, bytes counted on the barrier at bar_cluster_addr
// (the leader's).  No multicast.
__device__ __forceinline__ void tma_load_2d_pair(void *dst, const CUtensorMap *map, int x, int y, uint32_t bar_cluster_addr) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_u32(dst)),
        "l"(map), "r"(x), "r"(y), "r"(bar_cluster_addr)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t *dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// the barrier at this address of the cluster's shared window gets one arrival once every MMA issued so far by
// this thread has completed
__device__ __forceinline__ void umma_commit_pair(uint32_t bar_cluster_addr) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_cluster_addr)
                 : "memory");
}

struct Tc2Smem {
    uint8_t *stages;
    uint64_t *full, *empty, *acc_full, *acc_empty;
    uint32_t *tmem_slot;
    uint8_t *stg;
    volatile int *abort;
};

// p.m_tiles counts PAIRS of 128-token tiles here (tile m of the work-item arithmetic is tokens 256 m .. 256 m + 255);
// p.tail_first likewise counts pair tiles.  KIND as in prefill_tc.cu; the plain kernel has 256-wide tiles.
template <int KIND>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS)
    ff_tc2_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b0,
                  const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ TcParams p) {
    constexpr uint32_t IDESC = umma_idesc(2 * TC_BM, TC2_NT);
    extern __shared__ uint8_t smem_raw[];
    Tc2Smem s;
    s.stages = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    s.full = reinterpret_cast<uint64_t *>(s.stages + (size_t)TC2_STAGES * TC2_STAGE_BYTES);
    s.empty = s.full + TC2_STAGES;
    s.acc_full = s.empty + TC2_STAGES;
    s.acc_empty = s.acc_full + 2;
    s.tmem_slot = reinterpret_cast<uint32_t *>(s.acc_empty + 2);
    s.abort = reinterpret_cast<volatile int *>(s.tmem_slot + 1);
    s.stg = reinterpret_cast<uint8_t *>(s.full) + (2 * TC2_STAGES + 4) * sizeof(uint64_t) + 16;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();  // 0: leader
    const bool leader = rank == 0;
    if (tid == 0) {
        for (int i = 0; i < TC2_STAGES; ++i) {
            mbar_init(&s.full[i], 1);   // (used in the leader only: its producer's arrival, both CTAs' bytes)
            mbar_init(&s.empty[i], 1);  // one commit from the leader's MMA issuer, in each CTA
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s.acc_full[i], 1);                   // one commit, in each CTA
            mbar_init(&s.acc_empty[i], 2 * TC_EPI_WARPS);   // (used in the leader only: every epilogue warp of the pair)
        }
        *s.abort = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc_pair(s.tmem_slot, 2 * TC2_NT);
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers are initialised before anything of this CTA reaches them
    tc_fence_after_sync();
    pdl_launch_dependents();  // a finishing kernel behind this one may take its place on the SMs and wait there
    const uint32_t tmem_base = *s.tmem_slot;

    const int n_clusters = gridDim.x >> 1, cluster_id = blockIdx.x >> 1;
    const int n_items = p.tail_ks > 1 ? p.tail_first + (p.m_tiles * p.n_tiles - p.tail_first) * p.tail_ks
                                      : p.m_tiles * p.n_tiles * p.splits;
    const int kb_total = p.K / TC_BK;

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int item = cluster_id; ok && item < n_items; item += n_clusters) {
                const TcItem ti = tc_item(p, item, kb_total);
                const int m = 2 * ti.m + (int)rank, n = ti.n;
                // this CTA's half of the weight tile: with a gate the leader stages the 128 gate rows and the
                // follower the 128 up rows of the tile's neurons (accumulator columns 0..127 | 128..255);
                // otherwise rows 256 n + 128 rank .. + 127 of the one weight matrix
                const CUtensorMap *mb = (KIND == TC_GATED && rank) ? &map_b1 : &map_b0;
                const int b_row = KIND == TC_GATED ? n * 128 : n * 256 + (int)rank * 128;
                for (int kb = ti.kb0; kb < ti.kb1; ++kb, ++it) {
                    const int stage = it % TC2_STAGES;
                    const uint32_t use = it / TC2_STAGES;
                    if (use > 0 && !wait_or_abort(&s.empty[stage], (use - 1) & 1, s.abort, p.ws, 60)) {
                        ok = false;
                        break;
                    }
                    uint8_t *a = s.stages + (size_t)stage * TC2_STAGE_BYTES;
                    const uint32_t bar = map_to_rank(&s.full[stage], 0);
                    if (leader) mbar_arrive_expect_tx(&s.full[stage], 2 * TC2_STAGE_BYTES);
                    tma_load_2d_pair(a, &map_a, kb * TC_BK, m * TC_BM, bar);
                    tma_load_2d_pair(a + TC2_A_BYTES, mb, kb * TC_BK, b_row, bar);
                }
            }
            if (leader) {
                // stay until every copy of the pair that was started has landed (the follower leaves only after
                // the cluster-wide barrier below, which the leader reaches after this)
                const uint32_t first = it > TC2_STAGES ? it - TC2_STAGES : 0;
                for (uint32_t j = first; j < it; ++j) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&s.full[j % TC2_STAGES], (j / TC2_STAGES) & 1))
                        if (clock64() - t0 > WAIT_LIMIT_CYCLES) break;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader only) ----------------
        if (leader && lane == 0) {
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int item = cluster_id; ok && item < n_items; item += n_clusters, ++tcount) {
                const int acc = tcount & 1;
                const uint32_t acc_use = tcount >> 1;
                if (acc_use > 0 && !wait_or_abort(&s.acc_empty[acc], (acc_use - 1) & 1, s.abort, p.ws, 61)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * TC2_NT);
                const TcItem ti = tc_item(p, item, kb_total);
                for (int kb = ti.kb0; kb < ti.kb1; ++kb, ++it) {
                    const int stage = it % TC2_STAGES;
                    if (!wait_or_abort(&s.full[stage], (it / TC2_STAGES) & 1, s.abort, p.ws, 62)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint8_t *a = s.stages + (size_t)stage * TC2_STAGE_BYTES;
#pragma unroll
                    for (int k16 = 0; k16 < TC_BK / 16; ++k16)
                        umma_bf16_pair(d_tmem, smem_desc_sw128(a, k16), smem_desc_sw128(a + TC2_A_BYTES, k16), IDESC,
                                       (kb > ti.kb0 || k16 > 0) ? 1u : 0u);
                    // the stage may be refilled, in both CTAs, once these MMAs have read it
                    umma_commit_pair(map_to_rank(&s.empty[stage], 0));
                    umma_commit_pair(map_to_rank(&s.empty[stage], 1));
                }
                if (ok) {
                    umma_commit_pair(map_to_rank(&s.acc_full[acc], 0));
                    umma_commit_pair(map_to_rank(&s.acc_full[acc], 1));
                }
            }
        }
    } else {
        // ---------------- epilogue (warps 2..9 of both CTAs): this CTA's 128 rows of the pair's tile ----------------
        const int wq = warp & 3;
        const int half = (warp - 2) >> 2;
        uint8_t *const stg = s.stg + (warp - 2) * TC_STG_BYTES;
        uint32_t tcount = 0;
        for (int item = cluster_id; item < n_items; item += n_clusters, ++tcount) {
            const TcItem ti = tc_item(p, item, kb_total);
            const int m = 2 * ti.m + (int)rank;
            const int acc = tcount & 1;
            if (!wait_or_abort_relaxed(&s.acc_full[acc], (tcount >> 1) & 1, s.abort, p.ws, 63)) break;
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16) + (uint32_t)(acc * TC2_NT);
            // a part of a cut tile goes where the finishing kernel, which counts 128-token tiles, looks for it
            const int part = ti.part >= 0 ? (2 * (ti.part / p.tail_ks) + (int)rank) * p.tail_ks + ti.sp : -1;
            tc_epilogue_item<KIND, TC2_NT>(p, m, ti.n, ti.sp, part, taddr, stg, wq, half, lane);
            tc_fence_before_sync();  // this warp's TMEM reads are done
            __syncwarp();
            if (lane == 0) {
                if (leader) mbar_arrive(&s.acc_empty[acc]);
                else mbar_arrive_cluster(map_to_rank(&s.acc_empty[acc], 0));
            }
        }
    }

    // ---------------- teardown: the pair meets, then each CTA's allocating warp frees TMEM ----------------
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, 2 * TC2_NT);
    }
}

// p counts pair tiles (see the kernel).  Grid: two CTAs per work item, at most one pair per two SMs.
template <int KIND>
static griffin_status launch_tc2(const CUtensorMap &ma, const CUtensorMap &mb0, const CUtensorMap &mb1, const TcParams &p,
                                 int sms, cudaStream_t stream) {
    const size_t smem = 1024 + (size_t)TC2_STAGES * TC2_STAGE_BYTES + TC2_TAIL_BYTES;
    const void *fn = (const void *)ff_tc2_kernel<KIND>;
    if (ensure_dynamic_smem(fn, smem) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    const int items = p.tail_ks > 1 ? p.tail_first + (p.m_tiles * p.n_tiles - p.tail_first) * p.tail_ks
                                    : p.m_tiles * p.n_tiles * p.splits;
    const int clusters = items < sms / 2 ? items : sms / 2;
    ff_tc2_kernel<KIND><<<2 * clusters, TC_THREADS, smem, stream>>>(ma, mb0, mb1, p);
    count_launches(1);
    return cudaGetLastError() == cudaSuccess ? GRIFFIN_OK : GRIFFIN_ERR_CUDA;
}

griffin_status launch_tc_pairs(int kind, const CUtensorMap &ma, const CUtensorMap &mb0, const CUtensorMap &mb1,
                               const TcParams &p, int sms, cudaStream_t stream) {
    switch (kind) {
        case TC_GATED: return launch_tc2<TC_GATED>(ma, mb0, mb1, p, sms, stream);
        case TC_WIDE: return launch_tc2<TC_WIDE>(ma, mb0, mb1, p, sms, stream);
        default: return launch_tc2<TC_PLAIN>(ma, mb0, mb1, p, sms, stream);
    }
}

}  // namespace griffin
