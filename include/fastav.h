/*
 * fastav.h -- C ABI of the B200-native FastAV prune step.
 *
 * FastAV (Section 2.2 of the paper) prunes the token sequence of an audio-visual LLM during
 * prefill: at a pruning layer it scores every token by the attention the last query token(s)
 * pay to it (Eq. 4:  s = mean_h softmax(Q_last K^T)),  removes the lowest-scoring P% and lets
 * the following layers run on the survivors only.  The same step serves the "global" stage at
 * the middle layer and the "fine" stage at every later layer.  This library is that step:
 *
 *     fastav_score    Eq. 4, generalised to R scored rows, grouped-query heads, varlen batches
 *     fastav_select   the bottom-P % rule of Section 2.2 as a top-k keep set
 *     fastav_compact  the survivor layout: gather hidden states, position ids, K and V rows
 *     fastav_prune    all three in one enqueue
 *
 * Conventions shared by every call
 *   - Plain C.  No CUDA types: `stream` is a cudaStream_t passed as void*.
 *   - Every data pointer is a DEVICE pointer unless its comment says "host".  The params struct
 *     is read on the host at call time.
 *   - The caller owns every buffer (inputs, outputs, workspace).  The library allocates nothing
 *     and keeps no state between calls.
 *   - Calls only enqueue work on `stream` and return; they never synchronise.  On a negative
 *     return value nothing was enqueued.
 *   - bf16 tensors are token-major.  Strides are in elements; the innermost dimension
 *     (head_dim, hidden) is contiguous.  Rows must start on 16-byte boundaries.
 *   - A batch is a packed ("varlen") concatenation of sequences: sequence b owns tokens
 *     [cu_seqlens[b], cu_seqlens[b+1]) and scored rows [cu_qlens[b], cu_qlens[b+1]).
 *   - Conditions only the device can see (a keep count outside [0, n_b], more protected tokens
 *     than k_b) are handled by clamping and reported by OR-ing FASTAV_DEV_* bits into
 *     *device_status (optional, may be NULL; the caller zeroes it).  Nothing traps.
 */
#ifndef FASTAV_H_
#define FASTAV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FASTAV_VERSION 100 /* major*10000 + minor*100 + patch */

/* return codes */
#define FASTAV_OK 0
#define FASTAV_ERR_INVALID_ARG (-1) /* NULL required pointer, batch < 1, Hq % Hkv != 0, stride < row, counts inconsistent, in/out overlap */
#define FASTAV_ERR_UNSUPPORTED (-2) /* head_dim not 64/128, hidden % 8 != 0, misaligned pointer or stride */
#define FASTAV_ERR_WORKSPACE (-3)   /* workspace NULL, misaligned or smaller than fastav_workspace_bytes() */
#define FASTAV_ERR_CUDA (-4)        /* a launch failed; fastav_last_cuda_error() has the runtime's text */
#define FASTAV_ERR_TIMEOUT (-5)     /* reserved: every device-side wait is bounded */

/* params.flags */
#define FASTAV_CAUSAL 1u              /* scored row r sees keys j <= q_idx[r] only (the model's own mask) */
#define FASTAV_PROTECT_QUERY_ROWS 2u  /* the scored rows' tokens always survive (and count toward k_b) */
#define FASTAV_KEEP_IDX_GLOBAL 4u     /* keep_idx holds indices into the packed batch, not sequence-local ones */
#define FASTAV_CHAIN_CALLS 0x1000u    /* The index arrays of this call (cu_seqlens, cu_qlens, q_idx, keep_counts, protect) were
                                         complete before the work that precedes the call on the stream was enqueued (e.g.
                                         uploaded once for all pruning layers: the survivor counts are known on the host).
                                         The call's first kernel may then start, and read them, while that earlier work is
                                         still running, which hides its set-up behind the previous call's last kernel.
                                         Without the flag the first kernel starts when all earlier work has completed, so
                                         the arrays may be what the previous kernel wrote (a cu_keep_out used as the next
                                         cu_seqlens).  q, k, v, hidden, pos, scores and keep lists are never read early. */
#define FASTAV_SELECT_LOWEST 0x800u   /* fastav_select keeps the k_b LOWEST-scoring tokens instead: the "prune the most attended
                                         tokens" control of the paper's ablations (Tables 2 and 3, "Top attentive") */

/* Diagnostics: force one implementation of fastav_score instead of the shape-based choice.  A forced
 * path that does not support the shapes makes the call fail with FASTAV_ERR_UNSUPPORTED. */
#define FASTAV_SCORE_PATH_GENERIC 0x100u /* CUDA-core tiles, any shape */
#define FASTAV_SCORE_PATH_NARROW 0x200u  /* matrix-vector path, max_qlen <= 4 */
#define FASTAV_SCORE_PATH_WIDE 0x300u    /* tensor-core path */
#define FASTAV_SCORE_PATH_MASK 0x300u

/* Diagnostics: make fastav_compact use its plain load/store kernel instead of the bulk-copy one. */
#define FASTAV_COMPACT_PATH_LOADSTORE 0x400u
#define FASTAV_COMPACT_PATH_MASK 0x400u

/* bits OR-ed into *device_status */
#define FASTAV_DEV_K_CLAMPED 1        /* some keep_counts[b] was outside [0, n_b] and was clamped */
#define FASTAV_DEV_PROTECT_OVERFLOW 2 /* more protected tokens than k_b: the lowest-index ones were kept */
#define FASTAV_DEV_WAIT_EXPIRED 4     /* a bounded wait inside a kernel ran out; results of that call are invalid */
#define FASTAV_DEV_BAD_INDEX 8        /* fastav_compact met a keep_idx entry outside its sequence and skipped that row */
#define FASTAV_DEV_SHAPE_MISMATCH 16  /* cu_seqlens / cu_qlens on the device disagree with the host scalars of params (a sequence
                                         longer than max_seqlen, a batch longer than total_tokens, more scored rows than max_qlen /
                                         total_q, more work than the launch was sized for): the excess was left out */
#define FASTAV_DEV_SLOW_PATH 32       /* informational: fastav_score could not describe q or k to the tensor-memory-accelerator
                                         (tensor-map encoding refused) and ran its CUDA-core tiles instead, much more slowly */

/*
 * Shapes of one prune call (host memory).  The counts that fix grid sizes and output sizes are
 * host scalars because the caller knows them without a device round trip: k_b is a function of
 * n_b (bottom P % removed -> k_b = n_b - floor(P n_b)).
 */
typedef struct fastav_params {
  int32_t batch;                    /* B >= 1 */
  int32_t total_tokens, max_seqlen; /* N = cu_seqlens[B]; max_b n_b */
  int32_t total_q, max_qlen;        /* sum_b R_b = cu_qlens[B]; max_b R_b */
  int32_t total_keep, max_keep;     /* sum_b k_b; max_b k_b (upper bounds are fine) */
  int32_t num_q_heads, num_kv_heads, head_dim; /* Hq % Hkv == 0; head_dim 64 or 128 */
  int32_t hidden;                   /* D, a multiple of 8 */
  int64_t q_stride_tok, q_stride_head;                                 /* q  [total_q, Hq, head_dim] */
  int64_t k_stride_tok, k_stride_head, v_stride_tok, v_stride_head;     /* k,v [N, Hkv, head_dim]    */
  int64_t ko_stride_tok, ko_stride_head, vo_stride_tok, vo_stride_head; /* outputs [total_keep, Hkv, head_dim] */
  float softmax_scale;              /* <= 0 selects 1/sqrt(head_dim); 1.0 is Eq. 4 as printed */
  uint32_t flags;                   /* FASTAV_CAUSAL | FASTAV_PROTECT_QUERY_ROWS | FASTAV_KEEP_IDX_GLOBAL */
} fastav_params;

/* Library version (FASTAV_VERSION of the build). */
int32_t fastav_version(void);

/* Static text for a return code. */
const char* fastav_status_string(int32_t status);

/* Text of the last CUDA runtime error seen by this thread inside the library ("" if none). */
const char* fastav_last_cuda_error(void);

/*
 * Bytes of device workspace that fastav_score / fastav_select / fastav_prune need for these
 * shapes (out_bytes: host).  The workspace must be 256-byte aligned; its contents are scratch
 * and need no initialisation.  Two calls running concurrently need two workspaces.
 */
int32_t fastav_workspace_bytes(const fastav_params* params, size_t* out_bytes);

/*
 * Importance scores, Eq. 4 (Section 2.2, "Fine pruning"), without forming the L x L map.
 * For sequence b, token j:
 *
 *   scores_out[cu_seqlens[b] + j] =
 *       1/(Hq R_b) * sum_{r < R_b} sum_{h < Hq} softmax_{j' in V(r)}( scale <q[r,h,:], k[j', h/G, :]> )[j]
 *
 * with G = Hq/Hkv, V(r) = all keys of the sequence, or {j' <= q_idx[r]} under FASTAV_CAUSAL
 * (keys outside V(r) get 0 from that row).  R_b = 1 at the last token is Eq. 4 itself.
 *
 *   q          [total_q, Hq, head_dim] bf16  query vectors of the scored rows (as the layer's
 *                                            attention uses them, i.e. after RoPE)
 *   q_idx      [total_q] int32               sequence-local token index of each scored row
 *   cu_qlens   [B+1] int32
 *   k          [N, Hkv, head_dim] bf16
 *   cu_seqlens [B+1] int32
 *   lse_opt    [total_q, Hq] fp32 or NULL.  Optional log-sum-exp of each scored row and head, as the
 *              layer's own attention kernel returns it for these rows: natural logarithm of
 *              sum_{j' in V(r)} exp(scale <q, k_j'>), same scale and mask as here (-inf for a row that sees
 *              no key).  The method does not rely on the attention map (Section 1: it stays compatible
 *              with FlashAttention-style kernels), and those kernels produce exactly this by-product;
 *              with it the scores need one sweep over K instead of two.  The result is the same
 *              quantity (a wrong lse gives wrong scores; nothing checks it).
 *   scores_out [N] fp32 (written for every token; a sequence with R_b = 0 gets zeros)
 */
int32_t fastav_score(const fastav_params* params, const void* q, const int32_t* q_idx, const int32_t* cu_qlens,
                     const void* k, const int32_t* cu_seqlens, const float* lse_opt, float* scores_out,
                     void* workspace, size_t workspace_bytes, int32_t* device_status, void* stream);

/*
 * The first sweep alone: log sum exp of every scored row's logits, per head -- what an attention kernel
 * reports for these rows, in its convention (Section 1: the method needs no attention map, only what a
 * FlashAttention-style kernel already has):
 *
 *   lse_out [total_q, Hq] fp32   natural logarithm of sum_j exp(scale * <q[r,h,:], k[j,h/G,:]>) over the keys
 *                                row r may see; -inf for a row that sees none
 *
 * Handing it back to fastav_score as lse_opt gives the same scores as the self-contained call (to rounding).
 * Arguments, workspace and errors as for fastav_score.
 */
int32_t fastav_lse(const fastav_params* params, const void* q, const int32_t* q_idx, const int32_t* cu_qlens, const void* k,
                   const int32_t* cu_seqlens, float* lse_out, void* workspace, size_t workspace_bytes, int32_t* device_status,
                   void* stream);

/*
 * The bottom-P % rule of Section 2.2 ("Fine pruning"), stated on the survivors: per sequence keep the
 * keep_counts[b] highest-scoring tokens; equal scores go to the lower index; protected tokens
 * (protect_opt[j] != 0, and the scored rows' tokens under FASTAV_PROTECT_QUERY_ROWS) rank above
 * every score.  Survivors are written in ascending index order.
 *
 *   scores       [N] fp32 (finite)
 *   keep_counts  [B] int32          k_b; values outside [0, n_b] are clamped (FASTAV_DEV_K_CLAMPED)
 *   protect_opt  [N] uint8 or NULL
 *   q_idx, cu_qlens                 read only under FASTAV_PROTECT_QUERY_ROWS (else may be NULL)
 *   keep_idx_out [total_keep] int32 sequence-local indices (packed-batch indices under
 *                                   FASTAV_KEEP_IDX_GLOBAL), ascending within each sequence
 *   cu_keep_out  [B+1] int32        prefix sums of the clamped k_b
 */
int32_t fastav_select(const fastav_params* params, const float* scores, const int32_t* cu_seqlens,
                      const int32_t* keep_counts, const uint8_t* protect_opt, const int32_t* q_idx,
                      const int32_t* cu_qlens, int32_t* keep_idx_out, int32_t* cu_keep_out, void* workspace,
                      size_t workspace_bytes, int32_t* device_status, void* stream);

/*
 * Keep set given by rule instead of by score.  The paper's deployed GLOBAL stage (Section 2.2, "Global
 * pruning"; Section 3.1, implementation details) is positional: the rollout analysis fixes once which
 * positions matter (e.g. the first 10 audio tokens, the first 4 frames) and at the middle layer every
 * other audio/video token is dropped without looking at scores.  The caller states such a rule as a mask;
 * this call turns it into the keep list that fastav_compact consumes:
 *
 *   keep_mask    [N] uint8            token j of the packed batch survives iff keep_mask[j] != 0
 *   keep_idx_out [total_keep] int32   survivors, ascending per sequence (same convention as fastav_select)
 *   cu_keep_out  [B+1] int32          prefix sums of the per-sequence survivor counts
 *
 * params.total_keep is the capacity of keep_idx_out: survivors beyond it are not written, cu_keep_out is
 * clamped to it and FASTAV_DEV_K_CLAMPED is set.  Of params only batch, total_tokens, total_keep and flags
 * are read.  Workspace: 256-byte aligned, at least 4 * batch bytes (rounded up to 256).
 */
int32_t fastav_select_mask(const fastav_params* params, const uint8_t* keep_mask, const int32_t* cu_seqlens,
                           int32_t* keep_idx_out, int32_t* cu_keep_out, void* workspace, size_t workspace_bytes,
                           int32_t* device_status, void* stream);

/*
 * Survivor layout (what the layer-by-layer shrinking of the token set in Section 2.2 leaves for the next
 * layer): output row cu_keep[b] + i is input row cu_seqlens[b] + keep_idx[cu_keep[b] + i] of
 *
 *   hidden  [N, hidden] bf16   -> hidden_out [total_keep, hidden]
 *   pos     [N] int32          -> pos_out    [total_keep]      (position ids are carried, never renumbered)
 *   k, v    [N, Hkv, head_dim] -> k_out, v_out [total_keep, Hkv, head_dim] (strides from params)
 *
 * Bit-exact copies.  Any in/out pair may be NULL (both NULL) and is skipped.  Outputs must not
 * overlap inputs.  Needs no workspace.
 */
int32_t fastav_compact(const fastav_params* params, const int32_t* keep_idx, const int32_t* cu_keep,
                       const int32_t* cu_seqlens, const void* hidden_in, void* hidden_out, const int32_t* pos_in,
                       int32_t* pos_out, const void* k_in, void* k_out, const void* v_in, void* v_out,
                       int32_t* device_status, void* stream);

/*
 * The whole prune step of one pruning layer (Fig. 3; Section 2.2): fastav_score, fastav_select
 * and fastav_compact enqueued back to back.  scores_out, keep_idx_out and cu_keep_out are still
 * written, so the caller can inspect or reuse them.  The argument list is the union of the three
 * calls above, each argument with the meaning it has there -- lse_opt included: a caller whose
 * attention kernel already returned the log-sum-exp of the scored rows for this layer (Section 1:
 * the method works beside FlashAttention-style kernels) passes it and the scores take one sweep
 * over K; NULL makes the call self-contained.
 */
int32_t fastav_prune(const fastav_params* params, const void* q, const int32_t* q_idx, const int32_t* cu_qlens,
                     const void* k, const void* v, const int32_t* cu_seqlens, const float* lse_opt, const int32_t* keep_counts,
                     const uint8_t* protect_opt, const void* hidden_in, const int32_t* pos_in, float* scores_out,
                     int32_t* keep_idx_out, int32_t* cu_keep_out, void* hidden_out, int32_t* pos_out, void* k_out,
                     void* v_out, void* workspace, size_t workspace_bytes, int32_t* device_status, void* stream);

/*
 * The same prune step for tensors that live in HOST memory (offloaded activations or KV cache):
 * every data pointer of this call is a host pointer (pinned memory makes the copies asynchronous).
 * The call enqueues host-to-device copies of the inputs, fastav_prune, and device-to-host copies
 * of scores, keep_idx, cu_keep, the compacted tensors and the device status word (status_out,
 * optional) on `stream`, staged through `device_arena`, a DEVICE buffer of at least
 * fastav_host_arena_bytes() bytes, 256-byte aligned, owned by the caller.  Host outputs are valid
 * once the stream has been synchronised.  Only packed layouts are accepted (token stride =
 * heads * head_dim, head stride = head_dim; otherwise FASTAV_ERR_UNSUPPORTED).  Every check of
 * fastav_prune is made before the first copy, so a negative return value leaves nothing enqueued.
 * FASTAV_CHAIN_CALLS is ignored: the index arrays are uploaded by this very call.  The paper has no
 * counterpart for this entry point; it computes exactly what fastav_prune computes.
 */
int32_t fastav_host_arena_bytes(const fastav_params* params, size_t* out_bytes);
int32_t fastav_prune_host(const fastav_params* params, const void* q, const int32_t* q_idx, const int32_t* cu_qlens,
                          const void* k, const void* v, const int32_t* cu_seqlens, const float* lse_opt, const int32_t* keep_counts,
                          const uint8_t* protect_opt, const void* hidden_in, const int32_t* pos_in, float* scores_out,
                          int32_t* keep_idx_out, int32_t* cu_keep_out, void* hidden_out, int32_t* pos_out, void* k_out,
                          void* v_out, int32_t* status_out, void* device_arena, size_t arena_bytes, void* stream);

/*
 * fastav_select without any caller-provided scratch.  The paper has no counterpart for this
 * entry point: it exists for callers that cannot allocate device memory at the point where they
 * prune -- a plug-in running inside a host application that hands it input and output tensors
 * only, a real-time loop in which cudaMalloc's implicit synchronisation is not acceptable, a
 * process whose memory pool is fixed and fully assigned at start-up.  fastav_select needs a
 * workspace (one 32-bit key per token) whenever a sequence is too long for shared memory; here
 * the keys always go to an array built into the library, so the call takes no workspace and
 * never calls cudaMalloc, cudaFree or any routine that allocates.
 *
 * Limits and rules
 *   - total_tokens <= FASTAV_NOALLOC_MAX_TOKENS, else FASTAV_ERR_UNSUPPORTED (nothing enqueued).
 *     The array costs 4 * FASTAV_NOALLOC_MAX_TOKENS bytes (4 MiB) of device memory on every GPU
 *     on which the library is loaded, until the process exits.
 *   - The first call on each device looks up the array's device address (a runtime query, made
 *     with that device current, cached afterwards).  Make that first call during set-up, before
 *     any stream capture.
 *   - All calls on a device share the one array.  Two calls whose kernels can overlap on the GPU
 *     (different streams, no dependency between them) race on it and both results are undefined;
 *     calls on one stream, or otherwise ordered, are fine.  Nothing has to be cleared between
 *     calls: each call overwrites every key before reading it.
 *   - Of params only batch, total_tokens, max_seqlen, total_q, total_keep and flags are read.
 * Arguments, outputs, tie rule and device status bits are exactly those of fastav_select, and
 * the two produce identical keep_idx_out / cu_keep_out.
 */
#define FASTAV_NOALLOC_MAX_TOKENS (1 << 20)
int32_t fastav_select_noalloc(const fastav_params* params, const float* scores, const int32_t* cu_seqlens,
                              const int32_t* keep_counts, const uint8_t* protect_opt, const int32_t* q_idx,
                              const int32_t* cu_qlens, int32_t* keep_idx_out, int32_t* cu_keep_out,
                              int32_t* device_status, void* stream);

/*
 * Diagnostic (the paper has no counterpart): enqueues a one-block kernel that waits, with the same bounded
 * wait the scoring and compaction kernels use, on a barrier nothing ever completes.  After limit_ms
 * (1..1000) milliseconds the wait gives up, the kernel sets FASTAV_DEV_WAIT_EXPIRED in *device_status and
 * exits normally; the CUDA context stays usable.  It shows what a stuck copy or MMA would turn into: an error
 * bit, not a hang.
 */
int32_t fastav_selftest_bounded_wait(int32_t limit_ms, int32_t* device_status, void* stream);

/*
 * ---- Attention rollout (Section 2.1, "Analysis of audio-visual token importance via attention rollout") ----
 *
 * The analysis that tells where the global stage may cut.  For ONE sequence of n tokens and layers 1..L:
 *
 *   A^l   [n, n]  head-mean of layer l's attention weights: row i is token i's softmax over the keys it may
 *                 see (j <= i under FASTAV_CAUSAL), averaged over the Hq query heads (head h reads KV head
 *                 h / G; softmax scale as in fastav_score)
 *   Eq. 2         A~^l = alpha A^l + (1 - alpha) I
 *   Eq. 3         R^l  = A~^l A~^(l-1) ... A~^1
 *
 * The running product lives in a caller-owned, opaque STATE buffer (256-byte aligned,
 * fastav_rollout_state_bytes(n) bytes; the library keeps R transposed, as a pair of bf16 planes whose sum
 * carries about 16 mantissa bits, twice: one copy is read while the other is written).  Calls, all
 * asynchronous on `stream`, none allocates:
 *
 *   fastav_rollout_begin   R <- I
 *   fastav_rollout_layer   forms A^l from this layer's q [n, Hq, d] and k [n, Hkv, d] (bf16, strides from
 *                          params, post-RoPE as the layer's attention uses them), applies Eq. 2 and multiplies
 *                          it onto R from the left (Eq. 3).  `layer_index` counts the layers applied so far
 *                          (0 for the first call after begin); it selects which copy of the state is read.
 *                          lse_opt: NULL, or [n, Hq] fp32 natural-log row sums exp as an attention kernel
 *                          returns them for this layer (then the statistics pass is skipped).
 *                          map_out_opt: NULL, or [n, n] fp32 row-major, receives A^l itself (the "raw
 *                          attention weights" the paper compares the rollout with).
 *                          Of params: batch (must be 1), total_tokens = total_q = max_seqlen = max_qlen = n,
 *                          head counts, head_dim (64 or 128), q/k strides, softmax_scale, FASTAV_CAUSAL.
 *                          Workspace: 256-byte aligned, fastav_rollout_workspace_bytes(params) bytes.
 *   fastav_rollout_read    importance_out [n] fp32: mean over rows of column j of R (Section 2.1 after Eq. 3:
 *                          the influence of input token j on all tokens); rollout_out_opt: NULL or
 *                          [n, n] fp32 row-major R.  `layers_applied` = number of fastav_rollout_layer calls.
 *   fastav_rollout_threshold  keep_mask_out [n] uint8 = importance[j] >= threshold, or protect_opt[j] != 0;
 *                          *cut_out (device int32) = one past the last unprotected token that reaches the
 *                          threshold (0 if none): the positional rule "drop everything from there on".  The
 *                          mask feeds fastav_select_mask.
 *
 * n <= FASTAV_ROLLOUT_MAX_TOKENS, else FASTAV_ERR_UNSUPPORTED.  Errors as for the other calls; a wait that runs
 * out inside a kernel sets FASTAV_DEV_WAIT_EXPIRED.  alpha outside [0, 1] is FASTAV_ERR_INVALID_ARG.
 */
#define FASTAV_ROLLOUT_MAX_TOKENS 32768
int32_t fastav_rollout_state_bytes(int32_t n, size_t* out_bytes);
int32_t fastav_rollout_workspace_bytes(const fastav_params* params, size_t* out_bytes);
int32_t fastav_rollout_begin(int32_t n, void* state, size_t state_bytes, void* stream);
int32_t fastav_rollout_layer(const fastav_params* params, const void* q, const void* k, const float* lse_opt, float alpha,
                             int32_t layer_index, void* state, size_t state_bytes, float* map_out_opt, void* workspace,
                             size_t workspace_bytes, int32_t* device_status, void* stream);
int32_t fastav_rollout_read(int32_t n, int32_t layers_applied, const void* state, size_t state_bytes, float* importance_out,
                            float* rollout_out_opt, void* stream);
int32_t fastav_rollout_threshold(int32_t n, const float* importance, float threshold, const uint8_t* protect_opt,
                                 uint8_t* keep_mask_out, int32_t* cut_out, void* stream);

/*
 * Number of kernels this library has launched in this process so far (a diagnostic counter; the
 * only process-wide state the library has).  Benchmarks read it before and after a timed region.
 */
int64_t fastav_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* FASTAV_H_ */
