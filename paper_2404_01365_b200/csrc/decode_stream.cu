// Generation-phase pruned FF (Eqs. 4 and 5 of the GRIFFIN paper) for bf16 storage, streamed
// through registers: ONE kernel per call, one persistent CTA of 16 warps per SM, no shared-memory
// ring, no producer warp, no barriers on the way.
//   first half   z_hat = sigma(W_g_hat x + b_g_hat) * (W_1_hat x + b_1_hat)
//   meeting      every CTA has written its z entries; all CTAs wait for each other (bounded)
//   second half  y_hat = W_2_hat z_hat + b_2
//
// Both halves are matrix-vector products whose cost is the single pass over the compact weights,
// and a read-only stream of HBM runs fastest (measured on B200: 6.8-7.2 TB/s, against 6.5 TB/s for
// a copy) when every warp keeps 8 KB of plain 16-byte loads in flight and does nothing else that
// could hold them up.  So every warp streams weight rows straight from global memory into
// registers, two steps deep (a step is 2 KB of each of the two rows of a "pair"), and hands them
// to the warp-level tensor-core instruction mma.sync.m16n8k16, which takes the place of unpacking
// and multiplying element by element (the diagonal of the 16 x 8 tile is the dot product, see
// diagonal_sum).  The vector (x, then z) sits in shared memory, read conflict-free by the same
// lane that holds the matching weights.  Where the CTA has to wait for others (for the previous
// kernel on the stream, at the meeting point) each warp has, besides its two steps in registers,
// one more on its way into shared memory by bulk copies (TMA), so that HBM stays busy meanwhile.
//
// Work split.  A pair is (gate row j, up row j) in the first half of a gated block, two
// consecutive rows of W_1_hat (no gate) or of W_2_hat otherwise.  The B * P pairs of a half are
// dealt to the CTAs as contiguous ranges (a range spans at most two sequences, whose vectors are
// both staged), and a CTA's range, counted in steps, to its 16 warps as contiguous ranges again.
// A pair that is cut between warps leaves partial sums in shared memory, which are added, in warp
// order, once the CTA's warps have met at the end of the half: the split is even to one step and
// every sum has a fixed order.
#include "decode_mma.cuh"

namespace griffin {

constexpr int ST_WARPS = 16;
constexpr int ST_THREADS = ST_WARPS * 32;
constexpr int ST_H = 4;                    // 16-byte units of each row of a pair, per lane and step
constexpr int ST_STEP_UNITS = 32 * ST_H;   // units of a row that one step covers (2 KB)
#ifndef GRIFFIN_ST_ACCS
#define GRIFFIN_ST_ACCS 2
#endif
constexpr int ST_ACCS = GRIFFIN_ST_ACCS;            // independent accumulators of a warp (2 or 4)
constexpr int ST_GATE_UP = 0, ST_DOWN = 1, ST_UP = 2;

struct StreamPartial {  // what a warp has summed of a pair that it shares with its neighbours
    int f;              // pair (index among the B * P of the half), -1: none
    float a0, a1;
    int pad;
};

struct StreamGeom {
    int rows;       // rows per sequence: k, or d
    int P;          // pairs per sequence
    int row_units;  // 16-byte units per row
    int S;          // steps per row
};
__device__ __forceinline__ StreamGeom stream_geom(const DecodeParams &p, int mode) {
    StreamGeom g;
    g.rows = mode == ST_DOWN ? p.d : p.k;
    g.P = mode == ST_GATE_UP ? g.rows : (g.rows + 1) / 2;
    g.row_units = (mode == ST_DOWN ? p.ldk : p.d) / 8;
    g.S = (g.row_units + ST_STEP_UNITS - 1) / ST_STEP_UNITS;
    return g;
}

// This warp's share of a half: `first` is the CTA-wide... the pair that holds its first step, sp0 the
// step within that pair, n the number of steps; b0 the sequence of the CTA's first pair.
struct StreamRange {
    int f0, sp0, n, b0;
};
// T: the pairs dealt out this way (all B * P of the half, or what the pool below leaves)
__device__ __forceinline__ StreamRange stream_range(const StreamGeom &g, long long T, int warp) {
    const int lo = (int)(T * blockIdx.x / gridDim.x), hi = (int)(T * (blockIdx.x + 1) / gridDim.x);
    const int n = (hi - lo) * g.S;  // the CTA's steps
    const int s0 = (int)((long long)n * warp / ST_WARPS), s1 = (int)((long long)n * (warp + 1) / ST_WARPS);
    const int pr = s0 / g.S;
    StreamRange r;
    r.f0 = lo + pr;
    r.sp0 = s0 - pr * g.S;
    r.n = s1 - s0;
    r.b0 = lo / g.P;
    return r;
}

__device__ __forceinline__ uint4 ldg_stream(const uint4 *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// What a finished pair turns into: one entry of z (gated), or two of z or of y.
template <int MODE>
__device__ __forceinline__ void finish_pair(const DecodeParams &p, const StreamGeom &g, int act, int f, float a0, float a1) {
    const int b = f / g.P, j = f - b * g.P;
    __nv_bfloat16 *zb = reinterpret_cast<__nv_bfloat16 *>(p.z) + (size_t)b * 2 * p.ldk;  // z of sequence b, bf16
    if (MODE == ST_GATE_UP) {
        if (p.seq[b].b_gate) a0 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[b].b_gate)[j]);
        if (p.seq[b].b_up) a1 += __bfloat162float(static_cast<const __nv_bfloat16 *>(p.seq[b].b_up)[j]);
        zb[j] = __float2bfloat16_rn(sigma_rt(act, a0) * a1);
    } else if (MODE == ST_UP) {
        const __nv_bfloat16 *bias = static_cast<const __nv_bfloat16 *>(p.seq[b].b_up);
        const int r = 2 * j;
        zb[r] = __float2bfloat16_rn(sigma_rt(act, a0 + (bias ? __bfloat162float(bias[r]) : 0.f)));
        if (r + 1 < g.rows) zb[r + 1] = __float2bfloat16_rn(sigma_rt(act, a1 + (bias ? __bfloat162float(bias[r + 1]) : 0.f)));
    } else {
        const __nv_bfloat16 *bias = static_cast<const __nv_bfloat16 *>(p.b_down);
        __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(p.y) + (size_t)b * p.d;
        const int r = 2 * j;
        y[r] = __float2bfloat16_rn(a0 + (bias ? __bfloat162float(bias[r]) : 0.f));
        if (r + 1 < g.rows) y[r + 1] = __float2bfloat16_rn(a1 + (bias ? __bfloat162float(bias[r + 1]) : 0.f));
    }
}

// One warp's part of one half.  The steps are loaded and multiplied in order; two register
// buffers A and B hold the next two of them and are used in turn.
//
// Every answer from the memory system reaches an SM in the order it was asked for, at the SM's share
// of the bandwidth: whatever a CTA asks for while it waits for others (for the previous kernel on the
// stream before it may read x, for the meeting point before it may read z) is not lost time as long
// as something is still on its way when the wait ends and the vector has been read.  So, weights only:
//   * the warp's first two steps of a half go into A and B as early as possible: at the start of
//     the kernel, and for the second half as soon as the warp has multiplied its last step of the first;
//   * up to `ahead` further steps go into the warp's own piece of shared memory by bulk copies
//     (TMA) counted on the warp's own barrier, asked for right AFTER the loads of the vector, so that
//     they are still arriving when the vector is there and the first multiplications free A and B
//     for new loads.  They are multiplied from shared memory after the first two.
template <int MODE>
struct StreamHalf {
    StreamGeom g;
    int b0;              // sequence of the CTA's first pair (its vector is slot 0, the next sequence's slot 1)
    int f_slot1;         // first pair of sequence b0 + 1
    int n_issue, n_comp; // steps of this warp not yet loaded / not yet multiplied
    int n_staged;        // steps of this warp staged in shared memory
    bool mid;            // the pair being summed began in another warp
    // load cursor: pair, step within it, unit 0 of the pair's rows
    int lf, lsp;
    const uint4 *r0, *r1;
    bool two;
    // compute cursor
    int cf, csp;
    int lane, warp;

    __device__ __forceinline__ void set_pair(const DecodeParams &p, int f) {
        const int b = f / g.P, j = f - b * g.P;
        if (MODE == ST_GATE_UP) {
            r0 = static_cast<const uint4 *>(p.seq[b].w_gate) + (size_t)j * g.row_units;
            r1 = static_cast<const uint4 *>(p.seq[b].w_up) + (size_t)j * g.row_units;
            two = true;
        } else {
            const void *m = MODE == ST_DOWN ? p.seq[b].w_down : p.seq[b].w_up;
            r0 = static_cast<const uint4 *>(m) + (size_t)(2 * j) * g.row_units;
            r1 = r0 + g.row_units;
            two = 2 * j + 1 < g.rows;
        }
    }
    __device__ __forceinline__ void advance_load(const DecodeParams &p) {
        --n_issue;
        if (++lsp == g.S) {
            lsp = 0;
            ++lf;
            if (n_issue > 0) set_pair(p, lf);
        }
    }

    // pool_pairs: pairs at the end of the half that are not dealt out here (see the pool in the kernel)
    __device__ __forceinline__ void init(const DecodeParams &p, int warp_, int lane_, int pool_pairs = 0) {
        warp = warp_;
        lane = lane_;
        g = stream_geom(p, MODE);
        const StreamRange r = stream_range(g, (long long)p.B * g.P - pool_pairs, warp);
        b0 = r.b0;
        f_slot1 = (b0 + 1) * g.P;
        n_issue = n_comp = r.n;
        n_staged = 0;
        cf = lf = r.f0;
        csp = lsp = r.sp0;
        mid = lsp != 0;
        r0 = r1 = nullptr;
        two = false;
        if (n_issue > 0) set_pair(p, lf);
    }

    // This warp takes the whole of pair f and nothing else; its vector is slot 0 of the `vec` given to run().
    __device__ __forceinline__ void init_single(const DecodeParams &p, int warp_, int lane_, int f) {
        warp = warp_;
        lane = lane_;
        g = stream_geom(p, MODE);
        b0 = f / g.P;
        f_slot1 = 0x7fffffff;
        n_issue = n_comp = g.S;
        n_staged = 0;
        cf = lf = f;
        csp = lsp = 0;
        mid = false;
        set_pair(p, lf);
    }

    // Loads the next step into r and moves the load cursor on.
    __device__ __forceinline__ void issue(const DecodeParams &p, uint4 (&r)[2 * ST_H]) {
        const int u0 = lsp * ST_STEP_UNITS + lane;
        if ((lsp + 1) * ST_STEP_UNITS <= g.row_units && two) {  // (warp-uniform) the common case: nothing to guard
#pragma unroll
            for (int i = 0; i < ST_H; ++i) {
                r[i] = ldg_stream(r0 + u0 + i * 32);
                r[ST_H + i] = ldg_stream(r1 + u0 + i * 32);
            }
        } else {  // the end of a row, or a pair of one row: what is not there counts as zero
            const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int i = 0; i < ST_H; ++i) {
                const bool in = u0 + i * 32 < g.row_units;
                r[i] = in ? ldg_stream(r0 + u0 + i * 32) : zero;
                r[ST_H + i] = (in && two) ? ldg_stream(r1 + u0 + i * 32) : zero;
            }
        }
        advance_load(p);
    }

    // The warp's first two steps, into the register buffers.
    __device__ __forceinline__ void prologue_regs(const DecodeParams &p, uint4 (&A)[2 * ST_H], uint4 (&Bq)[2 * ST_H]) {
        if (n_issue > 0) issue(p, A);
        if (n_issue > 0) issue(p, Bq);
    }
    // Up to `ahead` further steps, into stage (the warp's 2 * ST_STEP_UNITS * ahead units of shared memory)
    // by bulk copies counted on bar, the warp's barrier for this half.
    __device__ __forceinline__ void prologue_staged(const DecodeParams &p, uint4 *stage, uint64_t *bar, int ahead) {
        uint32_t bytes = 0;
        for (int s = 0; s < ahead && n_issue > 0; ++s, ++n_staged) {
            const int u0 = lsp * ST_STEP_UNITS;
            const uint32_t nb = (uint32_t)min(ST_STEP_UNITS, g.row_units - u0) * 16;
            if (lane == 0) bulk_g2s(stage + s * 2 * ST_STEP_UNITS, r0 + u0, nb, bar);
            if (lane == 1 && two) bulk_g2s(stage + (s * 2 + 1) * ST_STEP_UNITS, r1 + u0, nb, bar);
            bytes += two ? 2 * nb : nb;
            advance_load(p);
        }
        if (n_staged > 0 && lane == 0) mbar_arrive_expect_tx(bar, bytes);
    }

    // The sums of a pair, or of this warp's piece of it, are complete: hand them on.
    __device__ __forceinline__ void step_done(const DecodeParams &p, float (&acc)[ST_ACCS][4], StreamPartial *part, int act) {
        --n_comp;
        const bool complete = csp == g.S - 1;
        if (complete || n_comp == 0) {
            float sum[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float t = 0.f;
#pragma unroll
                for (int a = 0; a < ST_ACCS; a += 2) t += acc[a][e] + acc[a + 1][e];
                sum[e] = t;
#pragma unroll
                for (int a = 0; a < ST_ACCS; ++a) acc[a][e] = 0.f;
            }
            const float a0 = diagonal_sum(sum, lane);          // lane 0: first row, lane 4: second row
            const float a1 = __shfl_sync(0xffffffffu, a0, 4);
            if (lane == 0) {
                if (complete && !mid) {
                    finish_pair<MODE>(p, g, act, cf, a0, a1);
                } else {
                    StreamPartial *s = part + 2 * warp + (mid ? 0 : 1);
                    s->f = cf;
                    s->a0 = a0;
                    s->a1 = a1;
                }
            }
            mid = false;
        }
        if (++csp == g.S) {
            csp = 0;
            ++cf;
        }
    }

    // Multiplies the step held in r.
    __device__ __forceinline__ void compute(const DecodeParams &p, const uint4 (&r)[2 * ST_H], float (&acc)[ST_ACCS][4],
                                            const uint4 *vec, int vec_units, StreamPartial *part, int act) {
        const uint4 *v = vec + (cf >= f_slot1 ? vec_units : 0) + csp * ST_STEP_UNITS + lane;
#pragma unroll
        for (int i = 0; i < ST_H; ++i) {
            const uint4 vv = v[i * 32];
            mma_bf16(acc[(2 * i) & (ST_ACCS - 1)], r[i].x, r[ST_H + i].x, r[i].y, r[ST_H + i].y, vv.x, vv.y);
            mma_bf16(acc[(2 * i + 1) & (ST_ACCS - 1)], r[i].z, r[ST_H + i].z, r[i].w, r[ST_H + i].w, vv.z, vv.w);
        }
        step_done(p, acc, part, act);
    }

    // Multiplies staged step s (the copies have landed).  A staged step may be the cut end of a row or half a pair.
    __device__ __forceinline__ void compute_staged(const DecodeParams &p, const uint4 *stage, int s, float (&acc)[ST_ACCS][4],
                                                   const uint4 *vec, int vec_units, StreamPartial *part, int act) {
        const uint4 *v = vec + (cf >= f_slot1 ? vec_units : 0) + csp * ST_STEP_UNITS + lane;
        const uint4 *w = stage + s * 2 * ST_STEP_UNITS + lane;
        const int u0 = csp * ST_STEP_UNITS + lane;
        const bool second = MODE == ST_GATE_UP || 2 * (cf - (cf / g.P) * g.P) + 1 < g.rows;
        const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < ST_H; ++i) {
            const bool in = u0 + i * 32 < g.row_units;
            const uint4 a = in ? w[i * 32] : zero;
            const uint4 b = (in && second) ? w[ST_STEP_UNITS + i * 32] : zero;
            const uint4 vv = v[i * 32];
            mma_bf16(acc[(2 * i) & (ST_ACCS - 1)], a.x, b.x, a.y, b.y, vv.x, vv.y);
            mma_bf16(acc[(2 * i + 1) & (ST_ACCS - 1)], a.z, b.z, a.w, b.w, vv.z, vv.w);
        }
        step_done(p, acc, part, act);
    }

    // All of this warp's steps of the half; A and Bq hold steps 0 and 1, the staged steps follow them.
    // Returns false when the wait for the staged steps gave up.
    __device__ __forceinline__ bool run(const DecodeParams &p, uint4 (&A)[2 * ST_H], uint4 (&Bq)[2 * ST_H], const uint4 *stage,
                                        uint64_t *bar, const uint4 *vec, int vec_units, StreamPartial *part,
                                        volatile int *abort, int act) {
        float acc[ST_ACCS][4] = {};
        if (n_comp > 0) {
            compute(p, A, acc, vec, vec_units, part, act);
            if (n_issue > 0) issue(p, A);
        }
        if (n_comp > 0) {
            compute(p, Bq, acc, vec, vec_units, part, act);
            if (n_issue > 0) issue(p, Bq);
        }
        if (n_staged > 0) {
            if (!wait_or_abort(bar, 0, abort, p.ws, MODE == ST_DOWN ? 11 : 10)) return false;
            for (int s = 0; s < n_staged; ++s) compute_staged(p, stage, s, acc, vec, vec_units, part, act);
        }
        while (n_comp > 0) {
            compute(p, A, acc, vec, vec_units, part, act);
            if (n_issue > 0) issue(p, A);
            if (n_comp == 0) break;
            compute(p, Bq, acc, vec, vec_units, part, act);
            if (n_issue > 0) issue(p, Bq);
        }
        return true;
    }
};

// The pairs that were cut between warps, added up by the first warp: entry e = 2 * warp + (0: the
// warp's first pair, begun elsewhere; 1: its last, ended elsewhere) is in step order, so the pieces of
// one pair follow each other among the entries in use.  Lane e holds entry e; the lane of a pair's
// first piece collects the rest through shuffles, in entry order (a fixed order), and finishes the
// pair.  (A loop over shared memory instead took 1.4 us at the end of each half.)
template <int MODE>
__device__ __forceinline__ void combine_partials(const DecodeParams &p, const StreamPartial *part, int act, int lane) {
    static_assert(2 * ST_WARPS == 32, "one lane per entry");
    const StreamPartial me = part[lane];
    const bool valid = me.f >= 0;
    const unsigned int mask = __ballot_sync(0xffffffffu, valid);
    if (mask == 0) return;  // (warp-uniform) nothing was cut
    const unsigned int below = mask & ((1u << lane) - 1u);
    const int prev = below ? 31 - __clz(below) : lane;
    const int f_prev = __shfl_sync(0xffffffffu, me.f, prev);
    const bool head = valid && (below == 0 || f_prev != me.f);
    float a0 = me.a0, a1 = me.a1;
    bool open = head;  // still collecting
    for (int j = 1; j < 32; ++j) {
        const int f_j = __shfl_down_sync(0xffffffffu, me.f, j);
        const float a0_j = __shfl_down_sync(0xffffffffu, me.a0, j);
        const float a1_j = __shfl_down_sync(0xffffffffu, me.a1, j);
        if (lane + j >= 32) open = false;
        if (open && f_j >= 0) {
            if (f_j == me.f) {
                a0 += a0_j;
                a1 += a1_j;
            } else {
                open = false;
            }
        }
        if (!__any_sync(0xffffffffu, open)) break;
    }
    if (head) {
        const StreamGeom g = stream_geom(p, MODE);
        finish_pair<MODE>(p, g, act, me.f, a0, a1);
    }
}

// bf16 words of a 16-byte unit whose elements from `keep` on are cleared (keep in 1..7)
__device__ __forceinline__ uint4 keep_elems(uint4 v, int keep) {
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (2 * i >= keep) w[i] = 0;
        else if (2 * i + 1 >= keep) w[i] &= 0xffffu;
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// After a give-up: the copies this warp started may still be on their way into its shared memory,
// which must not be handed back under them.  One more bounded wait (normally over at once).
__device__ __forceinline__ void drain_staged(uint64_t *bar, int n_staged) {
    if (n_staged == 0 || mbar_try_wait(bar, 0)) return;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, 0))
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) break;
}

__device__ __forceinline__ uint4 ld_cg_now(const uint4 *p) {  // through L2; volatile: stays where it is written
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

// Stages the vectors of sequences b0 and b0 + 1 (x: row_units units each; z: the same with the entries
// from k on cleared) as two rows of vec_units units, zero-filled.  The loads of the first
// ST_VEC_EARLY units per thread are issued before `between` runs and stored after it: what `between`
// asks the memory system for arrives behind the vector.
constexpr int ST_VEC_EARLY = 4;
template <bool IS_Z, class F>
__device__ __forceinline__ void stage_vectors(const DecodeParams &p, uint4 *vec, int vec_units, int b0, int tid, F between) {
    const int row_units = (IS_Z ? p.ldk : p.d) / 8;
    const int limit = IS_Z ? p.k : p.d;  // elements that exist
    const uint4 zero = make_uint4(0, 0, 0, 0);
    auto src_of = [&](int u, bool &in) -> const uint4 * {
        const int slot = u >= vec_units ? 1 : 0, uu = u - slot * vec_units, b = b0 + slot;
        in = u < 2 * vec_units && uu < row_units && 8 * uu < limit && b < p.B;
        if (IS_Z) return reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(p.z) + (size_t)b * 2 * p.ldk) + uu;
        return static_cast<const uint4 *>(p.x) + (size_t)b * row_units + uu;
    };
    auto fix = [&](uint4 v, int u) -> uint4 {
        const int slot = u >= vec_units ? 1 : 0, uu = u - slot * vec_units;
        return (IS_Z && 8 * uu + 8 > limit) ? keep_elems(v, limit - 8 * uu) : v;
    };
    uint4 early[ST_VEC_EARLY];
#pragma unroll
    for (int i = 0; i < ST_VEC_EARLY; ++i) {
        bool in;
        const uint4 *src = src_of(tid + i * ST_THREADS, in);
        early[i] = in ? ld_cg_now(src) : zero;
    }
    between();
#pragma unroll
    for (int i = 0; i < ST_VEC_EARLY; ++i) {
        const int u = tid + i * ST_THREADS;
        if (u < 2 * vec_units) vec[u] = fix(early[i], u);
    }
    for (int u = tid + ST_VEC_EARLY * ST_THREADS; u < 2 * vec_units; u += ST_THREADS) {
        bool in;
        const uint4 *src = src_of(u, in);
        vec[u] = in ? fix(__ldcg(src), u) : zero;
    }
}

template <bool GATED>
__global__ void __launch_bounds__(ST_THREADS, 1) decode_stream_kernel(const __grid_constant__ DecodeParams p, int act,
                                                                    int vec_units, int ahead, int pool_chunks) {
    constexpr int FIRST = GATED ? ST_GATE_UP : ST_UP;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    // two vectors of vec_units units and, for the pool of the first half, x of the last sequence (x_units units)
    const int x_units = pool_chunks > 0 ? (p.d / 8 + ST_STEP_UNITS - 1) / ST_STEP_UNITS * ST_STEP_UNITS : 0;
    uint4 *vec = reinterpret_cast<uint4 *>(smem_raw);
    uint4 *vec_pool = vec + 2 * vec_units;
    StreamPartial *part = reinterpret_cast<StreamPartial *>(vec_pool + x_units);
    volatile int *abort = reinterpret_cast<volatile int *>(part + 2 * ST_WARPS);  // [0]: abort flag; [2], [3]: claims of the pool
    volatile int *claim = abort + 2;
    uint64_t *bars = reinterpret_cast<uint64_t *>(const_cast<int *>(abort) + 4);  // [2 halves][ST_WARPS]
    uint4 *stages = reinterpret_cast<uint4 *>(bars + 2 * ST_WARPS);                 // [ST_WARPS][ahead] steps
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint4 *stage = stages + (size_t)warp * ahead * 2 * ST_STEP_UNITS;
    uint64_t *bar1 = bars + warp, *bar2 = bars + ST_WARPS + warp;
    unsigned int *const meet = &static_cast<WsHeader *>(p.ws)->meet_stream;

    if (lane == 0) {
        mbar_init(bar1, 1);
        mbar_init(bar2, 1);
        mbar_fence_init();
    }
    __syncwarp();

    // Which half of its round the meeting-point counter is in.  Every CTA of the call before has passed its
    // meeting (this CTA runs on an SM that one of them has left), and fewer than gridDim.x CTAs of this call
    // can have reported in: the value read here and every arrival of this call fall into the same half.
    // (Asked for before the weights, so that the answer does not queue behind them; needed at the meeting.)
    unsigned int meet_at_start = 0;
    if (tid == 0) meet_at_start = *reinterpret_cast<volatile unsigned int *>(meet);

    // ---- first half: the first weights are on their way before anything else happens
    uint4 A[2 * ST_H], Bq[2 * ST_H];
    StreamHalf<FIRST> h1;
    h1.init(p, warp, lane, pool_chunks * ST_WARPS);
    h1.prologue_regs(p, A, Bq);
    // the first claim on the pool (asked for now, needed when this CTA's own share is done)
    unsigned int *const pool = &static_cast<WsHeader *>(p.ws)->pool_stream;
    int my_claim = 0;
    if (pool_chunks > 0 && tid == 0) my_claim = (int)atomicInc(pool, (unsigned int)pool_chunks + gridDim.x - 1);
    pdl_launch_dependents();
    if (tid == 0) *abort = 0;
    if (tid < 2 * ST_WARPS) part[tid].f = -1;
    pdl_wait_prior_grids();  // x, the z scratch and the outputs belong to earlier work on the stream
    stage_vectors<false>(p, vec, vec_units, h1.b0, tid, [&]() { h1.prologue_staged(p, stage, bar1, ahead); });
    for (int u = tid; u < x_units; u += ST_THREADS)
        vec_pool[u] = u < p.d / 8 ? __ldcg(static_cast<const uint4 *>(p.x) + (size_t)(p.B - 1) * (p.d / 8) + u) : make_uint4(0, 0, 0, 0);
    __syncthreads();
    h1.run(p, A, Bq, stage, bar1, vec, vec_units, part, abort, act);
    // ---- the pool: the last pool_chunks * 16 pairs of the half (all of the last sequence) are not dealt out
    //      beforehand but handed out at run time, 16 whole pairs (one per warp) at a time, to the CTAs that are done
    //      with their own share: at saturation some groups of SMs get 8 % less out of the memory system than the
    //      others, and the meeting point below waits for the slowest.  Whole pairs, each summed by one warp in the
    //      order of its steps: the result does not depend on who takes what.  Every CTA claims until it is told that
    //      nothing is left, exactly once: pool_chunks + gridDim.x claims per call take the counter round to where
    //      it was.
    if (pool_chunks > 0) {
        const int pool_base = p.B * h1.g.P - pool_chunks * ST_WARPS;
        for (int it = 0;; ++it) {
            if (tid == 0) claim[it & 1] = my_claim;
            __syncthreads();  // (also: every warp is done with its share, or with the chunk before)
            const int chunk = claim[it & 1];
            if (chunk >= pool_chunks || *abort) break;
            StreamHalf<FIRST> hp;
            hp.init_single(p, warp, lane, pool_base + chunk * ST_WARPS + warp);
            hp.prologue_regs(p, A, Bq);
            if (tid == 0) my_claim = (int)atomicInc(pool, (unsigned int)pool_chunks + gridDim.x - 1);  // (needed next time round)
            hp.run(p, A, Bq, stage, bar1, vec_pool, vec_units, part, abort, act);
        }
    }
    // the first weights of the second half, as soon as this warp has room for them
    StreamHalf<ST_DOWN> h2;
    h2.init(p, warp, lane);
    h2.prologue_regs(p, A, Bq);
    __syncthreads();  // the partial sums are in place, nobody reads x any more
    if (*abort) {  // the meeting still gets this CTA's arrival: the others are not held up and the counter stays in phase
        if (tid == 0) grid_arrive_only(meet, gridDim.x);
        drain_staged(bar1, h1.n_staged);
        return;
    }
    // ---- meeting point.  The first warp adds the cut pairs and reports this CTA in (thread 0's fence makes
    //      every z entry of the CTA visible device-wide: the other warps wrote theirs before the barrier
    //      above, the lanes of this warp before the __syncwarp).
    if (warp == 0) {
        combine_partials<FIRST>(p, part, act, lane);
        part[lane].f = -1;
        __syncwarp();
        if (lane == 0) {
            grid_arrive_only(meet, gridDim.x);  // (nothing waits for the answer: it would queue behind the weights)
            grid_wait(meet, gridDim.x, meet_at_start >= gridDim.x, abort, p.ws);
        }
    }
    __syncthreads();
    if (*abort) {  // the wait gave up (status raised)
        drain_staged(bar2, h2.n_staged);
        return;
    }
    // z of the two sequences, read through L2 (other CTAs wrote it); the staged step is asked for behind it
    stage_vectors<true>(p, vec, vec_units, h2.b0, tid, [&]() {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the staged steps of the first half have been read
        h2.prologue_staged(p, stage, bar2, ahead);
    });
    __syncthreads();
    h2.run(p, A, Bq, stage, bar2, vec, vec_units, part, abort, act);
    __syncthreads();
    if (*abort) {
        drain_staged(bar2, h2.n_staged);
        return;
    }
    if (warp == 0) combine_partials<ST_DOWN>(p, part, act, lane);
}

#ifndef GRIFFIN_ST_POOL_PCT
#define GRIFFIN_ST_POOL_PCT 8
#endif
#ifndef GRIFFIN_ST_POOL_MIN
#define GRIFFIN_ST_POOL_MIN 16
#endif
#ifndef GRIFFIN_ST_AHEAD
#define GRIFFIN_ST_AHEAD 1
#endif
constexpr size_t ST_SMEM_BUDGET = 144 * 1024;  // shared memory that vectors and staged steps may take together
griffin_status decode_bf16_stream(DecodeParams &p, int act, bool gated, uint32_t flags, cudaStream_t stream) {
    const int sms = device_sm_count();
    if (sms <= 0) return GRIFFIN_ERR_CUDA;
    if (p.ws == nullptr) return GRIFFIN_ERR_WORKSPACE;  // the meeting point's counter lives in the header
    const int grid = sms;
    if (p.B > grid) return GRIFFIN_ERR_UNSUPPORTED;  // a CTA's range must not span more than two sequences
    const bool overlap = (flags & GRIFFIN_DECODE_OVERLAP_WEIGHT_PREFETCH) != 0;
    const int units = max(p.d, p.ldk) / 8;
    int vec_units = (units + ST_STEP_UNITS - 1) / ST_STEP_UNITS * ST_STEP_UNITS;
    // The pool of the first half: GRIFFIN_ST_POOL_PCT per cent of its pairs, in chunks of 16, all within the last
    // sequence; only when every warp has at least GRIFFIN_ST_POOL_MIN pairs of its own and a pair has four steps or
    // more (the chunks cost a barrier each and restart the pipelines, with one pair per warp to fill them).  Measured
    // on B200, us per call without / with: Llama-2-13B shape, 8 sets (23 pairs per warp) 250.8 / 243.2 (5 per cent:
    // no gain, 12: as 8); Llama-2-7B shape, 8 sets 163.1 / 158.6; Mistral shape, 4 sets, keep 0.75 158.0 / 152.8, keep 1.0
    // 205.5 / 207.9, keep 0.5 (12 pairs per warp) 107.2 / 107.9 - 108.8; Gemma shape, 4 sets (pairs of three steps)
    // 133.8 / 136.8.
    const long long pairs1 = (long long)p.B * (gated ? p.k : (p.k + 1) / 2), per_seq1 = gated ? p.k : (p.k + 1) / 2;
    int pool_chunks = 0;
    if (GRIFFIN_ST_POOL_PCT > 0 && pairs1 / ((long long)grid * ST_WARPS) >= GRIFFIN_ST_POOL_MIN && p.d / 8 > 3 * ST_STEP_UNITS) {
        long long pool_pairs = pairs1 * GRIFFIN_ST_POOL_PCT / 100;
        if (pool_pairs > per_seq1) pool_pairs = per_seq1;
        pool_chunks = (int)(pool_pairs / ST_WARPS);
    }
    const int x_units = pool_chunks > 0 ? (p.d / 8 + ST_STEP_UNITS - 1) / ST_STEP_UNITS * ST_STEP_UNITS : 0;
    const size_t fixed = (size_t)(2 * vec_units + x_units) * 16 + 2 * ST_WARPS * sizeof(StreamPartial) + 16 +
                         2 * ST_WARPS * sizeof(uint64_t);
    if (fixed > 227 * 1024) return GRIFFIN_ERR_UNSUPPORTED;
    // Steps per warp staged in shared memory across the waits.  Shared memory is taken from the
    // same 256 KB as the L1 cache, which the loads in flight pass through: measured on B200, with
    // 221 KB of shared memory (three staged steps) the stream drops from 6.7 to 5.9 TB/s, with up
    // to 157 KB (two) it is unharmed.  One step (64 KB) covers the waits as well as two do.
    const size_t per_step = (size_t)ST_WARPS * 2 * ST_STEP_UNITS * 16;
    int ahead = fixed < ST_SMEM_BUDGET ? (int)((ST_SMEM_BUDGET - fixed) / per_step) : 0;
    if (ahead > GRIFFIN_ST_AHEAD) ahead = GRIFFIN_ST_AHEAD;
    const size_t smem = fixed + ahead * per_step;
    const void *fn = gated ? (const void *)decode_stream_kernel<true> : (const void *)decode_stream_kernel<false>;
    if (ensure_dynamic_smem(fn, smem) != cudaSuccess) return GRIFFIN_ERR_CUDA;
    // every CTA of the grid must be able to run at the same time (they meet half-way): one per SM
    if (!grid_can_meet(fn, ST_THREADS, smem, grid)) return GRIFFIN_ERR_UNSUPPORTED;
    void *args[] = {&p, &act, &vec_units, &ahead, &pool_chunks};
    if (launch_maybe_overlapped(fn, dim3(grid), dim3(ST_THREADS), smem, stream, overlap, args) != cudaSuccess)
        return GRIFFIN_ERR_CUDA;
    return GRIFFIN_OK;
}

}  // namespace griffin
