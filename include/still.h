/*
 * still.h -- C ABI of the STILL intra-layer hybrid attention layer forward for
 * NVIDIA B200 (sm_100a).
 *
 * The layer (paper Sec. 3, "Methodology") takes the per-head queries, keys and
 * values of one attention layer and, for every query token t,
 *   1. computes the Self-Saliency Score of every token from sliding-window
 *      attention over the last C tokens (Sec. 3.1, Eqs. diag / nodiag / score),
 *   2. keeps, per chunk of C tokens, the top-k (the paper's lambda) scoring
 *      tokens for softmax attention; selection is delayed: a chunk is routed
 *      when it leaves the two-chunk local region (Sec. 3.3, Eq.
 *      delayed_selection),
 *   3. folds every other token of a routed chunk into a linear-attention state
 *      (s, z) through the Norm-Preserved Feature Map (Sec. 3.2, Eq.
 *      feature_map; Sec. 3.3, Eq. cache_routing_sum),
 *   4. outputs y_t = (N_SA + N_LA) / (D_SA + D_LA) (Sec. 3.3, merge equation and
 *      the definitions of N_SA, D_SA, N_LA, D_LA).
 * still_hybrid_attn_fwd is the chunk-wise parallel form (Algorithm 1) used for
 * prefill; still_hybrid_attn_step is the recurrent form (Sec. 3.3) used for
 * decode.  Both are defined per head; with grouped KV heads, query head h uses
 * KV head h / (H / Hkv) and scores, selection and state are per query head.
 *
 * General conventions
 *   - Every tensor pointer is DEVICE memory owned by the caller, contiguous in
 *     the stated layout, aligned to 16 bytes.  The library allocates no device
 *     memory.  What it keeps between calls is host-side and per host thread:
 *     encoded TMA descriptors of recently used buffers, the launch count and
 *     the timing events of still_profile_*, and -- only after a call of
 *     still_hybrid_attn_fwd_host -- three side streams and the events that
 *     order them, created on first use and kept until the thread exits.
 *     still_hybrid_attn_fwd_static adds one fixed array in the library's device
 *     image (see there).
 *   - The device that is current when a call is made must be the device of
 *     `cuda_stream` and of every buffer.
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL =
 *     the legacy default stream) and return without synchronising.
 *   - Return value: STILL_OK (0) or a negative still_status code.  No C++
 *     exception crosses this boundary.  There is no CPU fallback: a call either
 *     runs the CUDA kernels or fails.
 *   - Device-side waits (mbarrier waits inside the tensor-core kernels) are
 *     bounded; if one expires the kernel records a code in the status word at
 *     the start of the workspace, drains, frees its tensor memory and returns.
 *     still_device_status reads that word.
 */
#ifndef STILL_H_
#define STILL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum still_status {
    STILL_OK = 0,
    STILL_ERR_INVALID_ARG = -1,      /* null pointer, bad shape, topk > chunk, H % Hkv != 0, misaligned pointer */
    STILL_ERR_UNSUPPORTED = -2,      /* shape or dtype outside what the kernels cover (see still_params_t)     */
    STILL_ERR_WORKSPACE_TOO_SMALL = -3,
    STILL_ERR_STATE_FULL = -4,       /* decode state has no room for another token                             */
    STILL_ERR_CUDA = -5,             /* a CUDA runtime / driver call failed (launch error, no sm_100 device)    */
    STILL_ERR_DEVICE_TIMEOUT = -6,   /* a bounded device-side wait expired (reported by still_device_status)    */
    STILL_ERR_STATE_MISMATCH = -7    /* decode state was built with other parameters                            */
} still_status;

enum { STILL_DTYPE_FP32 = 0, STILL_DTYPE_BF16 = 1 };

/*
 * Problem description (Algorithm 1, "Input": q, k, v, gate g, feature maps
 * phi_q / phi_k, chunk size C, number lambda, small constant epsilon).
 *
 * Supported: d in {64, 128}; d_f in {32, 64, 128} with d_f <= d; chunk in
 * {32, 64, 128}; 0 <= topk <= chunk; dtype fp32 or bf16.  bf16 inputs with
 * chunk 64 or 128 run on the tcgen05 tensor-core kernels (the linear branch
 * too when d_f >= 64); fp32 inputs, and bf16 inputs with chunk 32, run on fp32
 * FMA kernels (TF32 would not meet the 1e-4 output tolerance of fp32).  The
 * bf16 decode step packs the query heads of a KV head into one tensor-core
 * tile and needs H / Hkv <= 16.
 */
typedef struct still_params {
    int32_t B;          /* batch                                                             */
    int32_t H;          /* query heads                                                       */
    int32_t Hkv;        /* KV heads, H % Hkv == 0                                            */
    int32_t d;          /* head dim                                                          */
    int32_t d_f;        /* width of the NP-Map linear map f; the feature dim is d' = 2 d_f   */
    int32_t chunk;      /* C: chunk size = score window w                                    */
    int32_t topk;       /* lambda: tokens kept for softmax attention per chunk               */
    int32_t dtype;      /* STILL_DTYPE_*: type of Q, K, V, G, Wq, bq, Wk, bk, Y               */
    float sm_scale;     /* multiplies q.k in the score and in the SA branch (1 = the main     */
                        /* text's exp(qk^T); d^-1/2 = App. A.1, Eq. softmax_attention)       */
    float eps;          /* epsilon of the Self-Saliency Score                                */
    int64_t max_salient;/* budget of the salient cache per query head, in tokens; 0 = unbounded */
                        /* (Eq. cache_routing_sum as written).  See below.                   */
} still_params_t;

/*
 * Salient-cache budget.  The paper's long-context experiments (Sec. 4.3) cap the number of cached salient
 * tokens, but its method section states no rule for what happens at the cap; the rule below is this
 * library's choice.  Selected tokens enter a head's salient cache in routing order, a chunk's top-k at a time;
 * when the cache would exceed max_salient tokens the oldest leave it and are folded into the linear state
 * (s, z) through phi_k, exactly as an unselected token is.  Every token outside the two-chunk local region is
 * thus counted once, in the softmax branch or in the linear branch, and the cost per token no longer grows
 * with the sequence (Eq. complexity's O(N) with a constant cache).  Selection itself is unchanged.
 * Supported: max_salient a positive multiple of topk (whole chunks' selections leave together), bf16 inputs
 * on the tensor-core kernels (chunk 64 or 128, d_f >= 64); otherwise STILL_ERR_UNSUPPORTED.
 */

/* Bytes of workspace still_hybrid_attn_fwd needs for a sequence of N tokens
 * (0 if the parameters are invalid).  Host-only arithmetic, no CUDA call. */
size_t still_workspace_bytes(const still_params_t *p, int64_t N);

/* Bytes of a decode state that can hold up to max_tokens tokens per sequence
 * (0 if the parameters are invalid).  Host-only arithmetic.  Layout: see
 * still_state_layout_t below. */
size_t still_state_bytes(const still_params_t *p, int64_t max_tokens);

/*
 * Byte offsets of the parts of a decode state, so that a caller can inspect,
 * copy or checkpoint it (the state is a plain buffer; copying it is a
 * checkpoint).  Fills *out and returns STILL_OK, or an error for bad parameters.
 *   header   : 256 bytes, int32 words {magic, version, B, H, Hkv, d, d_f, chunk,
 *              topk, dtype, capacity_lo, capacity_hi, t_lo, t_hi, status, 0...};
 *              t = tokens consumed so far.
 *   k_cache, v_cache : [B, Hkv, rows, d] in dtype -- the K/V history
 *              (local region + every earlier token; the salient pairs of Eq.
 *              cache_routing_sum are rows of it named by sel_idx).  rows = capacity,
 *              position q in row q.  With a salient-cache budget the store is a ring
 *              of rows = min(capacity, (max_salient / topk + 3) * chunk) -- the cached
 *              chunks, the two-chunk local region and the chunk being routed --
 *              with position q in row q % rows: it does not grow with the sequence.
 *   score    : [B, H, capacity] fp32 -- Self-Saliency Score of every token.
 *   sel_idx  : [B, H, capacity / chunk, topk] int32 -- salient positions of each
 *              routed chunk, ascending, -1 padded (rows of chunks not yet routed
 *              are unspecified).
 *   sel_mask : [B, H, capacity / chunk, chunk / 32] uint32 -- the same selection as
 *              bit masks: bit j of word w of chunk c is set when position
 *              c * chunk + 32 w + j is selected (what the decode kernel reads).
 *   S        : [B, H, 2 d_f, d] fp32 -- KV state s_t.
 *   z        : [B, H, 2 d_f] fp32 -- normaliser z_t.
 *   scratch  : split-KV partial results of the step kernel.
 */
typedef struct still_state_layout {
    size_t header, k_cache, v_cache, score, sel_idx, sel_mask, S, z, scratch, total;
    int64_t capacity; /* max_tokens rounded up to a multiple of chunk */
} still_state_layout_t;
int still_state_layout(const still_params_t *p, int64_t max_tokens, still_state_layout_t *out);

/*
 * Prefill: Algorithm 1 (Chunk-Wise Parallel Form) over N tokens.
 *
 *   Q        [B, H, N, d]     queries
 *   K, V     [B, Hkv, N, d]   keys, values
 *   G        [B, H, N, d]     gate values g_t (already activated) or NULL = ones;
 *                             multiplies N_LA only
 *   Wq, bq   [H, d, d_f], [H, d_f] or NULL      f of phi_q: f(x) = x Wq + bq
 *   Wk, bk   [Hkv, d, d_f], [Hkv, d_f] or NULL  f of phi_k
 *   Y        [B, H, N, d]     output, or NULL to skip the SA branch and the merge
 *                             (useful when only state_out is wanted)
 *   scores   [B, H, N] fp32   Self-Saliency Scores, or NULL
 *   sel_idx  [B, H, ceil(N/chunk), topk] int32: absolute positions of the selected
 *            tokens of every chunk, ascending, -1 padded when a ragged last chunk
 *            has fewer than topk tokens; or NULL (a workspace copy is used)
 *   state_out  decode state of still_state_bytes(p, max_tokens) bytes with
 *            capacity >= N, or NULL.  On return it describes the sequence after N
 *            tokens, ready for still_hybrid_attn_step with t_pos = N.
 *   state_max_tokens  the max_tokens the state was sized with (ignored if
 *            state_out is NULL)
 *   workspace, workspace_bytes  at least still_workspace_bytes(p, N)
 *
 * Ties in the score are broken by position (smaller first); NaN scores rank
 * lowest.  N need not be a multiple of chunk.  N = 0 launches nothing, except
 * that with state_out it initialises the state to "no tokens" (header, zero S
 * and z), which is how a decode from an empty sequence starts; the tensor
 * pointers may then be NULL.
 * Errors: STILL_ERR_INVALID_ARG, STILL_ERR_UNSUPPORTED,
 * STILL_ERR_WORKSPACE_TOO_SMALL, STILL_ERR_STATE_FULL (N > capacity),
 * STILL_ERR_CUDA.
 */
int still_hybrid_attn_fwd(const still_params_t *p, int64_t N, const void *Q, const void *K,
                          const void *V, const void *G, const void *Wq, const void *bq,
                          const void *Wk, const void *bk, void *Y, float *scores, int32_t *sel_idx,
                          void *state_out, int64_t state_max_tokens, void *workspace,
                          size_t workspace_bytes, void *cuda_stream);

/*
 * Decode: one step of the Recurrent Form (Sec. 3.3) for every sequence of the
 * batch.  t_pos is the number of tokens the state already holds (the new token
 * gets 0-based position t_pos); the caller tracks it on the host.  The first
 * kernel of the step compares the state's header with the call -- magic word,
 * the parameters and capacity the state was built with, the token count -- and
 * on a mismatch the step writes nothing (state and y unchanged) and records
 * STILL_ERR_STATE_MISMATCH in the state's status word (detail 1: token count,
 * 2: not a state, 3: other parameters); still_device_status reads it.  Once
 * the status word is set every later step on that state is a no-op, until a
 * prefill rebuilds the state.
 *
 *   q [B, H, d], k, v [B, Hkv, d], g [B, H, d] or NULL, y [B, H, d]
 *   Wq, bq, Wk, bk as for the prefill
 *
 * The step appends (k, v), scores the new token, routes the chunk that has just
 * left the two-chunk local region when the new token opens a chunk (top-k into
 * sel_idx, the rest into S and z), and writes y by the merge equation.
 * Errors: STILL_ERR_INVALID_ARG, STILL_ERR_UNSUPPORTED, STILL_ERR_STATE_FULL
 * (t_pos >= capacity), STILL_ERR_CUDA.
 */
int still_hybrid_attn_step(const still_params_t *p, void *state, int64_t state_max_tokens,
                           int64_t t_pos, const void *q, const void *k, const void *v,
                           const void *g, const void *Wq, const void *bq, const void *Wk,
                           const void *bk, void *y, void *cuda_stream);

/*
 * Prefill with HOST buffers: copies Q, K, V (and G, the NP-Map parameters) from
 * host memory (pinned memory makes the copies asynchronous) into `arena`, runs
 * still_hybrid_attn_fwd and copies Y (and scores / sel_idx when not NULL) back.
 * `arena` is device memory of at least still_host_arena_bytes(p, N) bytes; it
 * holds the staged tensors and the workspace.  The (batch, KV-head group) units
 * are independent, so the call is cut into up to sixteen parts whose host-to-device
 * copies, compute and device-to-host copies overlap; the parts compute alternately
 * on `cuda_stream` and on a second stream, so that one part's last thread blocks
 * run beside the next part's first ones (three side streams created on first use
 * per host thread, ordered after the work already enqueued on `cuda_stream`).  The
 * call returns after synchronising all of them, so the host outputs are valid on
 * return.
 */
size_t still_host_arena_bytes(const still_params_t *p, int64_t N);
int still_hybrid_attn_fwd_host(const still_params_t *p, int64_t N, const void *hQ, const void *hK,
                               const void *hV, const void *hG, const void *hWq, const void *hbq,
                               const void *hWk, const void *hbk, void *hY, float *hscores,
                               int32_t *hsel_idx, void *arena, size_t arena_bytes,
                               void *cuda_stream);

/*
 * Prefill without a caller-provided workspace.  (The paper has no counterpart: this is a
 * packaging variant of still_hybrid_attn_fwd, for callers that cannot allocate device memory --
 * code that runs inside another runtime's fixed memory plan, a serving loop whose memory was
 * budgeted at start-up, a context where cudaMalloc is not allowed or would stall the device.)
 *
 * The intermediate results that still_hybrid_attn_fwd keeps in `workspace` live instead in a
 * fixed array of STILL_STATIC_WORKSPACE_BYTES inside the library's device image.  Every GPU on
 * which the library is used holds that array until the process exits.  The call itself allocates
 * and frees nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 *
 *   - Arguments are those of still_hybrid_attn_fwd without state_out, workspace and their sizes;
 *     Q, K, V, (G, Wq, bq, Wk, bk), Y, scores, sel_idx are still the caller's device buffers.
 *   - Limit: still_workspace_bytes(p, N) must not exceed STILL_STATIC_WORKSPACE_BYTES, otherwise
 *     the call returns STILL_ERR_WORKSPACE_TOO_SMALL and launches nothing.  still_workspace_bytes
 *     tells in advance (it is host arithmetic); the workspace grows with B * H * N.
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress, with that device current); make that first call outside any stream
 *     capture.
 *   - All calls share the one array, and it keeps whatever the previous call left there.  The
 *     parts that must start at zero are cleared by every call on its own stream.  Two calls
 *     that overlap on the GPU (different streams, or different host threads without ordering
 *     between their streams) race on it: keep calls on one device ordered one after the other.
 *   - The device status word of the call is not reachable through still_device_status.
 * Errors: those of still_hybrid_attn_fwd, STILL_ERR_WORKSPACE_TOO_SMALL as above, STILL_ERR_CUDA
 * if the address look-up fails.
 */
#define STILL_STATIC_WORKSPACE_BYTES (16u << 20)
int still_hybrid_attn_fwd_static(const still_params_t *p, int64_t N, const void *Q, const void *K,
                                 const void *V, const void *G, const void *Wq, const void *bq,
                                 const void *Wk, const void *bk, void *Y, float *scores,
                                 int32_t *sel_idx, void *cuda_stream);

/*
 * Reads the device status word of a workspace (prefill) or of a decode state
 * after synchronising `cuda_stream`.  *status receives STILL_OK or
 * STILL_ERR_DEVICE_TIMEOUT / STILL_ERR_STATE_MISMATCH; *detail (optional)
 * receives a kernel-specific code saying which wait gave up.
 */
int still_device_status(const void *workspace_or_state, void *cuda_stream, int *status, int *detail);

/* Number of kernel launches the last still_hybrid_attn_fwd / _step call on this
 * host thread enqueued (for launch accounting in benchmarks). */
int still_last_launch_count(void);

/*
 * Self-test of the bounded device-side wait.  Launches one small kernel whose only act is the
 * mbarrier wait of the tensor-core kernels on a barrier that nothing ever arrives on, with a limit
 * of `limit_cycles` SM clock cycles instead of the kernels' built-in limit.  The wait runs out, the
 * kernel records STILL_ERR_DEVICE_TIMEOUT with detail 99 in `status_block` (256 bytes of device
 * memory, 16-byte aligned, cleared by this call) and ends normally; still_device_status(status_block)
 * then reports it.  The context stays usable.  Errors: STILL_ERR_INVALID_ARG, STILL_ERR_CUDA.
 */
int still_selftest_wait_timeout(void *status_block, int64_t limit_cycles, void *cuda_stream);

/*
 * Optional timing of the dominant kernel (the softmax-attention + merge kernel of the
 * prefill, the split-KV attend kernel of the decode step) for roofline reports.
 * still_profile_enable(n) creates n pairs of CUDA events owned by the library (host
 * objects, no device memory); from then on every call on this host thread records one
 * pair around that kernel on the caller's stream, until n pairs are used.
 * still_profile_collect synchronises the recorded events, writes the elapsed
 * milliseconds of each pair to ms[0..*n_records) (at most `capacity`), destroys the
 * events and disables the timing.  Not for use during stream capture.
 */
int still_profile_enable(int max_records);
int still_profile_collect(float *ms, int capacity, int *n_records);

/* Static string for a status code. */
const char *still_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* STILL_H_ */
