/*
 * griffin_ff.h -- C ABI of libgriffin_ff.so
 *
 * GRIFFIN (arXiv 2404.01365) for one feed-forward (FF) block of a decoder layer (gated, Eq. 3,
 * or without a gate, Eq. 2), as hand-written CUDA kernels for NVIDIA B200 (sm_100a).  Four steps:
 *
 *   griffin_ff_prefill_score   prompt phase: full FF over the S prompt tokens and the
 *                              selection statistic s                       (Eqs. 1, 3, 6)
 *   griffin_select_topk        expert set E = top-k of s                  (Section 4.2)
 *   griffin_compact_experts    slice W_g, W_1 by rows and W_2 by columns  (Section 4.2)
 *   griffin_ff_decode          generation phase: pruned FF on every new token (Eqs. 4, 5)
 *
 * Notation (Section 3 of the paper): d = D, d_ff = D_FF, w_gate = W_g [d_ff, d],
 * w_up = W_1 [d_ff, d], w_down = W_2 [d, d_ff], b_gate/b_up/b_down = b_g/b_1/b_2,
 * X [S, d] prompt hidden states, Z = FF_1(X) [S, d_ff], s [d_ff], E (k indices).
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless its comment says "host".  All matrices are
 *     dense row-major; base pointers must be 16-byte aligned; d and d_ff must be multiples
 *     of 8.  `dtype` is the storage type of X, the weights, the biases and Y; scores are
 *     always fp32 and indices int32.  Accumulation is always fp32.
 *   - The library allocates no device memory and frees none: the caller owns every
 *     buffer, including the workspace (size it with griffin_workspace_bytes and clear it
 *     once with griffin_workspace_init).
 *   - Every call validates its arguments on the host first; on a validation error nothing
 *     is enqueued.  Work is enqueued on `stream` (a cudaStream_t passed as void*, NULL =
 *     the default stream) and the call returns without synchronising.  The only call that
 *     synchronises is griffin_check_device_status.
 *   - Calls that share a workspace must be ordered on one stream (they may not overlap on
 *     the GPU).
 *   - No exceptions cross this boundary; every call returns a griffin_status.
 *   - Device-side waits are bounded (about two seconds of SM clocks).  A kernel whose wait runs
 *     out raises the workspace's status word and returns; griffin_check_device_status then says
 *     GRIFFIN_ERR_TIMEOUT, the outputs of that call are undefined, and the workspace must be
 *     cleared with griffin_workspace_init before its next use (the word stays raised until then).
 *   - What the library keeps between calls, per process: small host-side tables (SM count and
 *     granted shared-memory limits per device, guarded by a mutex) and, for the bf16 prompt
 *     phase, one non-blocking side stream and two events per host thread and device, created by
 *     that thread's first griffin_ff_prefill_score[_chunk] call on the device and never
 *     destroyed: the statistic's kernels run there beside the down projection and rejoin
 *     `stream` before the call returns.  Make that first call outside any stream capture.  Set
 *     the environment variable GRIFFIN_NO_SIDE_STREAM (to anything) before the first call to
 *     keep every kernel on the caller's stream.
 *   - Entry points may be called from several host threads at once, on different streams and
 *     workspaces.
 */
#ifndef GRIFFIN_FF_H
#define GRIFFIN_FF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GRIFFIN_FF_VERSION 1
#define GRIFFIN_MAX_BATCH 32      /* sequences per griffin_ff_decode call              */
#define GRIFFIN_MAX_D 8192        /* largest model width the decode kernels accept     */
#define GRIFFIN_MAX_COMBINE 256   /* samples per griffin_combine_scores call           */

typedef enum {
    GRIFFIN_OK = 0,
    GRIFFIN_ERR_INVALID_ARG = 1,  /* null pointer, size out of range, k not in [1,d_ff] */
    GRIFFIN_ERR_UNSUPPORTED = 2,  /* shape / dtype / activation this build cannot run   */
    GRIFFIN_ERR_ALIGNMENT = 3,    /* a pointer or leading dimension is not 16-byte aligned */
    GRIFFIN_ERR_WORKSPACE = 4,    /* workspace missing or smaller than griffin_workspace_bytes */
    GRIFFIN_ERR_CUDA = 5,         /* a CUDA runtime call or a kernel launch failed      */
    GRIFFIN_ERR_TIMEOUT = 6       /* a bounded device-side wait gave up (see griffin_check_device_status) */
} griffin_status;

/* Gate non-linearity sigma of Eq. 3 (the paper names the GLU variants in Section 1). */
typedef enum {
    GRIFFIN_ACT_SWIGLU = 0,       /* sigma(t) = t / (1 + exp(-t))                                   */
    GRIFFIN_ACT_GEGLU_TANH = 1,   /* sigma(t) = t/2 (1 + tanh(sqrt(2/pi) (t + 0.044715 t^3)))       */
    GRIFFIN_ACT_REGLU = 2,        /* sigma(t) = max(t, 0)                                           */
    GRIFFIN_ACT_GEGLU_ERF = 3,    /* sigma(t) = t/2 (1 + erf(t / sqrt(2)))                          */
    /* FF blocks WITHOUT a gate (Eq. 2, e.g. OPT): FF_1(x) = sigma(W_1 x + b_1).  There is no W_g:
     * w_gate / b_gate (and w_gate_c / b_gate_c of a compact set) must be NULL, every other
     * argument keeps its meaning, and each step moves two matrices instead of three. */
    GRIFFIN_ACT_RELU = 4,         /* sigma = max(t, 0)                                              */
    GRIFFIN_ACT_GELU_TANH = 5,    /* sigma = the tanh form of GEGLU_TANH                            */
    GRIFFIN_ACT_GELU_ERF = 6,     /* sigma = the erf form of GEGLU_ERF                              */
    GRIFFIN_ACT_SILU = 7          /* sigma = t / (1 + exp(-t))                                      */
} griffin_act;
/* Whether an activation code names a gated block (W_g present). */
#define GRIFFIN_ACT_IS_GATED(act) ((act) >= GRIFFIN_ACT_SWIGLU && (act) <= GRIFFIN_ACT_GEGLU_ERF)

typedef enum { GRIFFIN_DT_F32 = 0, GRIFFIN_DT_BF16 = 1 } griffin_dtype;

/* Shape and types of one FF block (Section 3). */
typedef struct {
    int32_t d;                    /* model width D                                      */
    int32_t d_ff;                 /* FF width D_FF                                      */
    int32_t act;                  /* griffin_act                                        */
    int32_t dtype;                /* griffin_dtype                                      */
} griffin_ff_desc;

/* Full weights of one FF block (Eqs. 1 and 3).  Biases may be NULL (= absent). */
typedef struct {
    const void *w_gate;           /* [d_ff, d]  W_g (NULL for a block without a gate)   */
    const void *w_up;             /* [d_ff, d]  W_1                                     */
    const void *w_down;           /* [d, d_ff]  W_2                                     */
    const void *b_gate;           /* [d_ff] or NULL                                     */
    const void *b_up;             /* [d_ff] or NULL                                     */
    const void *b_down;           /* [d]    or NULL                                     */
} griffin_ff_weights;

/* Compact weights of one sequence's expert set (Section 3: W_g_hat, W_1_hat in R^{k x D},
 * W_2_hat in R^{D x k}).  Rows of w_down_c are padded to ldk elements, ldk = k rounded up
 * to a multiple of 8 (griffin_compact_ldk); the padding holds zeros.  With E = all neurons
 * the full weights themselves are a valid compact set (k = ldk = d_ff), which is how the
 * unpruned FF is run through the same decode kernels. */
typedef struct {
    void *w_gate_c;               /* [k, d] (NULL for a block without a gate)           */
    void *w_up_c;                 /* [k, d]                                             */
    void *w_down_c;               /* [d, ldk]                                           */
    void *b_gate_c;               /* [k] or NULL                                        */
    void *b_up_c;                 /* [k] or NULL                                        */
    int32_t k;                    /* number of expert neurons                           */
    int32_t ldk;                  /* leading dimension of w_down_c, >= k, multiple of 8 */
} griffin_ff_compact;

/* Full weights of one FF block in neuron-major form: neuron j owns row j of all three
 * matrices, so w_down_t is the TRANSPOSE of W_2 (made once, when the model is loaded).  Used
 * by griffin_ff_decode_indexed.  Biases may be NULL (= absent). */
typedef struct {
    const void *w_gate;           /* [d_ff, d]  W_g (NULL for a block without a gate)   */
    const void *w_up;             /* [d_ff, d]  W_1                                     */
    const void *w_down_t;         /* [d_ff, d]  W_2 transposed                          */
    const void *b_gate;           /* [d_ff] or NULL                                     */
    const void *b_up;             /* [d_ff] or NULL                                     */
    const void *b_down;           /* [d]    or NULL                                     */
} griffin_ff_weights_nm;

/* Flags of griffin_ff_decode. */
#define GRIFFIN_DECODE_DEFAULT 0u
/* Launch the decode kernels with programmatic dependent launch: each kernel may begin
 * streaming its (read-only) weights into shared memory or registers while the previous kernel on the
 * stream is still finishing; it reads x and writes y / the workspace only after that
 * kernel has completed.  The caller promises that no earlier work still running on the
 * stream WRITES the compact weights this call reads (do not set it on the first decode
 * call after griffin_compact_experts). */
#define GRIFFIN_DECODE_OVERLAP_WEIGHT_PREFETCH 1u
/* bf16, gated blocks only (ignored otherwise): use the tcgen05 kernel (the weights go from shared memory straight into the
 * 5th-generation tensor cores) for shapes that it takes (d and ldk multiples of 128; with one
 * shared expert set 2..8 sequences); other shapes, and calls without the flag, run the
 * warp-level (mma.sync) kernels.  Results agree within the documented tolerance.  On the
 * measured workloads the warp-level kernels are the faster ones, which is why they are the
 * default. */
#define GRIFFIN_DECODE_TCGEN05 2u
/* bf16, sequences with their own expert sets: which of the two warp-level kernels runs.  Both make
 * one pass over the compact weights and hand them to mma.sync; they differ in how the weights
 * travel.  RING: bulk copies (TMA) by a producer warp into a ring of shared-memory stages that two
 * groups of consumer warps read.  STREAM: every one of 16 warps loads its own rows straight into
 * registers with plain 16-byte loads, two steps deep.  Without either flag the call picks by size:
 * the register stream is the faster one once every warp has enough to do (about 150 MB of weights
 * per call on a B200: 6.7 TB/s against 6.0-6.3 on the Llama-2-13B shape with 8 sets), the ring
 * when the call is so short that filling and draining 2368 separate pipelines shows (Llama-2-7B
 * shape, one sequence: 24.8 against 24.9-25.2 us).  Giving both is an error.  Results of the two agree
 * within the documented tolerance (the sums are taken in different orders). */
#define GRIFFIN_DECODE_RING 4u
#define GRIFFIN_DECODE_STREAM 8u

/* Status text for a code (static string, never NULL). */
const char *griffin_status_string(griffin_status st);

/* Library ABI version (GRIFFIN_FF_VERSION at build time). */
int32_t griffin_version(void);

/* Number of kernels the library has launched (or recorded into a stream capture) in this process
 * so far, over all devices and threads.  A diagnostic: the difference across a piece of work says
 * how many launches it took.  Replaying a captured graph does not go through the library and is not
 * counted. */
uint64_t griffin_kernel_launches(void);

/* k for a keep ratio (= 1 - the paper's "FF sparsity", Section 5): floor(keep*d_ff + 0.5)
 * clamped to [1, d_ff].  Host-only arithmetic. */
int32_t griffin_k_from_keep_ratio(int32_t d_ff, double keep);

/* ldk for k experts: k rounded up to a multiple of 8. */
int32_t griffin_compact_ldk(int32_t k);

/* Bytes of workspace that any call on this FF shape needs, for prompts of at most S_max
 * tokens and at most n_seq_max sequences per decode call.  Returns 0 if desc is NULL or
 * invalid. */
size_t griffin_workspace_bytes(const griffin_ff_desc *desc, int32_t S_max, int32_t n_seq_max);

/* Clears the workspace header (device status word, meeting counters of the one-kernel decode calls).
 * Enqueue once before first use, and again after a GRIFFIN_ERR_TIMEOUT. */
griffin_status griffin_workspace_init(void *workspace, size_t ws_bytes, void *stream);

/* Prompt phase (Section 4.2, "Prompt Phase Expert Neuron Selection").
 *   y[S, d]      = FF(X) = (sigma(X W_g^T + b_g) * (X W_1^T + b_1)) W_2^T + b_2   (Eqs. 1, 3)
 *                  -- the full block, never pruned, independent of k (without a gate, Eq. 2:
 *                  FF(X) = sigma(X W_1^T + b_1) W_2^T + b_2);
 *   score[d_ff]  = s, s_j = || column j of Zbar ||_2, Zbar_i = Z_i / ||Z_i||_2   (Eq. 6);
 *                  a token whose activation row is all zero contributes nothing.
 * x [S, d] in, y [S, d] out (dtype of desc), score fp32 out.  1 <= S.  Z is held in the
 * workspace in the storage dtype.  y may be NULL to skip the down projection. */
griffin_status griffin_ff_prefill_score(const griffin_ff_desc *desc, const griffin_ff_weights *w,
                                        const void *x, int32_t S, void *y, float *score,
                                        void *workspace, size_t ws_bytes, void *stream);

/* The prompt phase for a prompt that is fed piece by piece (long prompts: the workspace only
 * has to hold the activations of one piece).  Each call is griffin_ff_prefill_score on the S
 * tokens of one piece -- y[S, d] = FF(X) for them -- but the statistic is carried across the
 * calls: s_j^2 is a sum over the tokens of the prompt (Eq. 6: every token normalises its own
 * activation row, nothing couples two tokens), so
 *   sumsq[d_ff] (fp32, in/out) = (first ? 0 : sumsq) + sum over this piece's tokens of Zbar_ij^2,
 *   score[d_ff] (fp32, out, may be NULL) = sqrt(sumsq): after the last piece this is s of the
 *   whole prompt, equal to that of one call up to the order of the fp32 additions.
 * The pieces may have any lengths >= 1.  Calls on one prompt must be ordered on one stream. */
griffin_status griffin_ff_prefill_score_chunk(const griffin_ff_desc *desc, const griffin_ff_weights *w,
                                              const void *x, int32_t S, void *y, float *sumsq, float *score,
                                              int32_t first, void *workspace, size_t ws_bytes, void *stream);

/* Expert selection (Section 4.2): for each of n_seq score vectors, the indices of its k
 * largest entries, written in ascending index order; equal scores go to the lower index.
 * score [n_seq, d_ff] fp32 in, idx [n_seq, k] int32 out.  Scores must not be NaN. */
griffin_status griffin_select_topk(const float *score, int32_t n_seq, int32_t d_ff, int32_t k,
                                   int32_t *idx, void *stream);

/* Batch statistic s_bar = sum_i s_i / sqrt(S_i) (Eq. 7) for sharing one expert set among
 * n_seq <= GRIFFIN_MAX_COMBINE samples.  score [n_seq, d_ff] fp32 in, prompt_len: HOST
 * array of n_seq lengths (each >= 1), out [d_ff] fp32. */
griffin_status griffin_combine_scores(const float *score, const int32_t *prompt_len /*host*/,
                                      int32_t n_seq, int32_t d_ff, float *out, void *stream);

/* Expert compaction (Section 4.2): out.w_gate_c = W_g[E, :], out.w_up_c = W_1[E, :],
 * out.w_down_c[:, 0:k] = W_2[:, E] (padding columns k..ldk zeroed), and the matching bias
 * entries when both the source bias and the destination are non-NULL.  Bit copies.
 * idx [k] int32, every entry in [0, d_ff); an out-of-range entry is not dereferenced: its
 * row / column is filled with zeros and, when `workspace` is not NULL, the device status
 * word is raised.  out->k and out->ldk must be set by the caller (ldk from
 * griffin_compact_ldk).  Source and destination buffers must not overlap. */
griffin_status griffin_compact_experts(const griffin_ff_desc *desc, const griffin_ff_weights *w,
                                       const int32_t *idx, const griffin_ff_compact *out,
                                       void *workspace /*may be NULL*/, void *stream);

/* The same slicing from NEURON-MAJOR full weights (griffin_ff_weights_nm: w_down_t is the transpose of W_2,
 * [d_ff, d]).  The result in `out` is bit for bit that of griffin_compact_experts on the row-major W_2; what
 * differs is the traffic: the selected neurons' rows of W_2^T are contiguous, so only those k rows are read
 * (and turned into the [d, ldk] layout of w_down_c on the way), where the row-major W_2 has to be read whole
 * because at the usual keep ratios every 32-byte sector of it holds a selected column.  Same argument rules. */
griffin_status griffin_compact_experts_nm(const griffin_ff_desc *desc, const griffin_ff_weights_nm *w,
                                          const int32_t *idx, const griffin_ff_compact *out,
                                          void *workspace /*may be NULL*/, void *stream);

/* Generation phase (Eqs. 4, 5): for each of B sequences, with its own compact set,
 *   y[b] = W_2_hat (sigma(W_g_hat x[b] + b_g_hat) * (W_1_hat x[b] + b_1_hat)) + b_2
 * (without a gate: y[b] = W_2_hat sigma(W_1_hat x[b] + b_1_hat) + b_2).
 * sets: HOST array of B structs; every set must have the same k and ldk.  Entries may repeat
 * to share a set: when all the sequences of a bf16 call name the same buffers (one expert
 * set for the batch, Eq. 7), the weights are streamed once for every 8 sequences (fewer when
 * d or ldk is so large that 8 vectors do not fit in shared memory beside the weight stages)
 * and every weight row meets all those vectors at once; with distinct sets each sequence is
 * a pass of its own.  b_down [d] or NULL is shared by all sequences.  x [B, d] in,
 * y [B, d] out.  1 <= B <= GRIFFIN_MAX_BATCH, d <= GRIFFIN_MAX_D.  flags: GRIFFIN_DECODE_*.
 * The activations z_hat [B, ldk] pass through the workspace (4 bytes per entry).  With bf16
 * storage the call is one kernel whose CTAs (one per SM) meet half-way through a counter in
 * the workspace header: run it on a GPU whose SMs it can all occupy.  (The call asks the
 * runtime whether one CTA per SM can be resident and returns GRIFFIN_ERR_UNSUPPORTED when not;
 * SMs held by other work at the time can still make the bounded wait run out:
 * GRIFFIN_ERR_TIMEOUT from griffin_check_device_status, y undefined.) */
griffin_status griffin_ff_decode(const griffin_ff_desc *desc, int32_t B,
                                 const griffin_ff_compact *sets /*host*/, const void *b_down,
                                 const void *x, void *y, void *workspace, size_t ws_bytes,
                                 uint32_t flags, void *stream);

/* Generation phase (Eqs. 4, 5) without a compact copy: the pruned block
 *   y[b] = W_2[:, E_b] (sigma(W_g[E_b, :] x[b] + b_g[E_b]) * (W_1[E_b, :] x[b] + b_1[E_b])) + b_2
 * is evaluated by reading the rows idx[b, 0..k) of the neuron-major full weights in place, so
 * griffin_compact_experts and its k x d copies per sequence are not needed.  The result is
 * that of griffin_ff_decode on the compact set of the same indices, up to rounding (z stays
 * in fp32 here).  bf16 storage only (GRIFFIN_ERR_UNSUPPORTED otherwise), d <= GRIFFIN_MAX_D,
 * 1 <= B <= GRIFFIN_MAX_BATCH, 1 <= k <= d_ff.
 * idx [B, k] int32 on the DEVICE; the order of a sequence's indices does not matter and
 * sequences may share or differ in their lists.  An entry outside [0, d_ff) is not
 * dereferenced: that neuron contributes nothing and the device status word is raised.
 * x [B, d] in, y [B, d] out.  The workspace holds one fp32 partial y per SM and sequence
 * (griffin_workspace_bytes covers it).  flags: GRIFFIN_DECODE_DEFAULT or
 * GRIFFIN_DECODE_OVERLAP_WEIGHT_PREFETCH (the promise then covers idx as well as the
 * weights).  One kernel whose CTAs (one per SM) meet at the end through a counter in the
 * workspace header: run it on a GPU whose SMs it can all occupy. */
griffin_status griffin_ff_decode_indexed(const griffin_ff_desc *desc, int32_t B,
                                         const griffin_ff_weights_nm *w, const int32_t *idx, int32_t k,
                                         const void *x, void *y, void *workspace, size_t ws_bytes,
                                         uint32_t flags, void *stream);

/* The paper has no counterpart to this call: it is griffin_ff_decode for callers that have
 * no device memory to give as a workspace and may not allocate any.  That is the situation
 * of code that lives inside somebody else's process under a fixed memory budget (an
 * inference server that hands a plug-in its inputs and outputs and nothing else), and of
 * latency-critical loops that must stay clear of cudaMalloc / cudaFree because those calls
 * take the allocator's lock and synchronise the whole device.
 *
 * Same arguments, same kernels and same results as griffin_ff_decode, minus the workspace:
 * the activations z_hat go through an array that is part of the library image itself
 * (GRIFFIN_STATIC_SCRATCH_BYTES of device memory on every GPU that loads the library, held
 * until the process exits).  The call allocates and frees nothing.
 *   - Limit: B * ldk * 4 bytes must fit in GRIFFIN_STATIC_SCRATCH_BYTES, otherwise
 *     GRIFFIN_ERR_UNSUPPORTED is returned and nothing is enqueued (B = 8 sequences of up to
 *     32768 experts fit; use griffin_ff_decode with a workspace beyond that).
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls on a device share the one array.  It keeps whatever the previous call left
 *     there.  The scratch proper needs no clearing, because every entry the second half of a
 *     call reads has been written by its first half.  In front of it the array carries the
 *     256 bytes that a workspace starts with: a status word and the counters through which the
 *     CTAs of the one-kernel bf16 decode meet half-way.  They are zero when the library is
 *     loaded; the counters run round and stay in step from call to call as long as every call
 *     runs to its end (every CTA reports in exactly once per call, also after a give-up).
 *     Two calls that overlap on the GPU (different streams) race on the array: keep the calls
 *     on one device ordered.
 *   - Should a bounded wait inside a kernel give up, the call's output is incomplete;
 *     griffin_ff_decode_static_status reports it (and clears the header again). */
#define GRIFFIN_STATIC_SCRATCH_BYTES (1u << 20)
griffin_status griffin_ff_decode_static(const griffin_ff_desc *desc, int32_t B,
                                        const griffin_ff_compact *sets /*host*/, const void *b_down,
                                        const void *x, void *y, uint32_t flags, void *stream);

/* Companion of griffin_ff_decode_static (no counterpart in the paper either): synchronises `stream`,
 * reads the status word in front of the current device's static array and returns what
 * griffin_check_device_status would for a workspace.  When the word was raised, the header (word
 * and meeting counters) is cleared again, so that the array is fit for the next call; call it only
 * while no griffin_ff_decode_static call is running on the device.  Allocates nothing. */
griffin_status griffin_ff_decode_static_status(void *stream);

/* Synchronises `stream`, then reads the workspace's device status word.  GRIFFIN_OK,
 * GRIFFIN_ERR_TIMEOUT (a bounded wait inside a kernel gave up), GRIFFIN_ERR_INVALID_ARG
 * (a kernel met an out-of-range expert index) or GRIFFIN_ERR_CUDA. */
griffin_status griffin_check_device_status(const void *workspace, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* GRIFFIN_FF_H */
