/*
 * ulorl.h -- C ABI of the fused UloRL token-loss library (CUDA, sm_100a).
 *
 * One call pair computes, for T packed response tokens, the per-token part of the UloRL
 * policy update: LM-head logits z = kappa * hidden W^T, log-softmax and entropy per
 * token (the policy of Eq. 6 and the vocabulary sum of Eq. 10's H-bar), the segment-aware
 * or pseudo-on-policy importance ratio (Eq. 8, Section 3.1.2), the well-mastered-positive-
 * token mask (Eq. 9) under the entropy gate of Eq. 10, the clipped token-normalised
 * surrogate (Eq. 10 with the bounds of Eq. 7), and its gradients to hidden and W.
 * The T x V logits are never written to global memory.
 *
 * Conventions
 *  - Every pointer except `params` is DEVICE memory owned by the caller, row-major and
 *    contiguous.  The library allocates and frees no device memory; results depend only on
 *    the arguments of the call.
 *  - State kept by the library (process lifetime, created on first use under one internal
 *    mutex, so first calls from several host threads are safe): per device, the shared-memory
 *    opt-in of each kernel, the multiprocessor count, the device address of the built-in
 *    scratch of ulorl_token_loss_decide_static, and the two copy streams with their events of
 *    ulorl_token_loss_step_host; per process, the driver entry point that encodes tensor
 *    maps, the launch counter and the events of ulorl_kernel_timing_*.  No environment
 *    variable is read.
 *  - Every path is deterministic: no floating-point atomics; reductions over tokens run in a
 *    fixed order (d_W: one reduce-add per element and panel, panels in order), so equal
 *    inputs give bit-identical outputs on equal hardware.
 *  - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*) and never
 *    synchronise.  `loss` and `stats` stay on the device.
 *  - The return value is the host-side validation / launch status.  Device-side problems
 *    (a target outside [0, V), a bounded wait that ran out) are recorded in a status word
 *    inside the workspace and read back by ulorl_check_status(); offending rows are
 *    clamped, never read out of bounds.
 *  - Tokens are response tokens only; there is no ignore-index.
 *  - hidden, W and d_hidden have the element type `dtype`.  H must be a multiple of 8, and
 *    T ln(V + 1) < 2^29 (the range of the exact per-sequence entropy sums).
 */
#ifndef ULORL_H_
#define ULORL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ULORL_OK = 0,
  ULORL_ERR_INVALID_ARG = -1,   /* NULL pointer, negative size, inconsistent offsets    */
  ULORL_ERR_UNSUPPORTED = -2,   /* shape / dtype / alignment the kernels do not cover   */
  ULORL_ERR_WORKSPACE = -3,     /* workspace smaller than ulorl_workspace_bytes()       */
  ULORL_ERR_CUDA = -4,          /* a CUDA runtime or driver call failed                 */
  ULORL_ERR_DEVICE_TIMEOUT = -5,/* a bounded device-side wait ran out                   */
  ULORL_ERR_BAD_TARGET = -6,    /* some target id was outside [0, V) (row was clamped)  */
  ULORL_ERR_STATIC_LIMIT = -7   /* batch exceeds the built-in scratch of ulorl_token_loss_decide_static */
} ulorl_status_t;

typedef enum { ULORL_F32 = 0, ULORL_BF16 = 1 } ulorl_dtype_t;
typedef enum { ULORL_IS_SAIS = 0, ULORL_IS_POIS = 1 } ulorl_is_mode_t;            /* Eq. 8 | Section 3.1.2 */
typedef enum { ULORL_MPT_OFF = 0, ULORL_MPT_ALWAYS = 1, ULORL_MPT_DYNAMIC = 2 } ulorl_mpt_mode_t; /* Section 3.2 */
typedef enum { ULORL_ENT_PER_SEQ = 0, ULORL_ENT_BATCH = 1, ULORL_ENT_SUPPLIED = 2 } ulorl_ent_scope_t;
/* AUTO = TENSOR for bf16, SIMT for f32.  TENSOR: tcgen05 kernels on CTA pairs (one 256 x 256 MMA tile per
 * pair).  TENSOR_1CTA: the same kernels with one CTA per 128 x 256 tile, kept as a cross-check. */
typedef enum { ULORL_PATH_AUTO = 0, ULORL_PATH_SIMT = 1, ULORL_PATH_TENSOR = 2,
               ULORL_PATH_TENSOR_1CTA = 3 } ulorl_kernel_path_t;

/* bits of flags[t] */
#define ULORL_FLAG_MASKED    1u  /* MPT and gate open: excluded from the objective (Eq. 10)   */
#define ULORL_FLAG_CLIP_HIGH 2u  /* A > 0 and ratio > 1 + eps_high: gradient clipped           */
#define ULORL_FLAG_CLIP_LOW  4u  /* A < 0 and ratio < 1 - eps_low : gradient clipped           */
#define ULORL_FLAG_MPT       8u  /* well-mastered positive token (Eq. 9), whatever the gate    */

#define ULORL_N_STALENESS 16

/* Normalisation of the loss.  TOKENS: every response token weighs 1/N, N = all response tokens
 * (Eq. 7 and Eq. 10, the paper's method).  SEQUENCE: a token of sequence i weighs 1/(G |o_i|), the
 * per-sample mean of Eq. 5 (GRPO); |o_i| is taken from seq_offsets, so sequences must be whole. */
typedef enum { ULORL_NORM_TOKENS = 0, ULORL_NORM_SEQUENCE = 1 } ulorl_loss_norm_t;

typedef struct {
  int32_t T, H, V, num_seqs;   /* packed tokens, hidden size, vocabulary, sequences (seq_offsets[num_seqs] == T) */
  int32_t dtype;               /* ulorl_dtype_t of hidden, W, d_hidden                                           */
  int32_t is_mode;             /* ulorl_is_mode_t                                                                */
  int32_t mpt_mode;            /* ulorl_mpt_mode_t                                                               */
  int32_t ent_scope;           /* ulorl_ent_scope_t: which entropy the gate H-bar < sigma is taken on            */
  int32_t adv_per_token;       /* 0: advantages[num_seqs]; 1: advantages[T]                                      */
  float clip_eps_low;          /* Eq. 7 bounds; the paper gives no value, workloads use 0.2 / 0.2                */
  float clip_eps_high;
  float mpt_tau;               /* probability threshold of Eq. 9 (0.99 in Section 4.1)                           */
  float entropy_target;        /* sigma of Eq. 10 (0.2 in Section 4.1)                                           */
  float inv_temperature;       /* kappa multiplying the logits; 1 unless the caller trains at a temperature      */
  int64_t norm_tokens;         /* N of Eq. 10; 0 means T (a micro-batch passes the global token count)           */
  int32_t current_version;     /* id of the latest policy; staleness = current_version - segment_version[t]      */
  int32_t dw_accumulate;       /* bwd: 0 overwrite d_W, 1 add into it (micro-batching)                           */
  int32_t kernel_path;         /* ulorl_kernel_path_t; AUTO = tensor-core path for bf16, SIMT path for f32       */
  int32_t bwd_panel_tokens;    /* bwd: tokens per staging panel; 0 = library default                             */
  int32_t compact_rows;        /* bwd, tensor path: 1 = run the three contractions only on tokens whose          */
                               /* grad_coef is non-zero (a masked token, and without a KL term a clipped or      */
                               /* zero-advantage one, adds nothing to either gradient, Eq. 10); results are the  */
                               /* same, the workspace grows by two                                               */
                               /* [T, H] copies.  0 = all rows.  Part of the workspace size: pass the same value */
                               /* to ulorl_workspace_bytes and to both calls.                                    */
  int32_t loss_norm;           /* ulorl_loss_norm_t: weight of a token's term in the loss                        */
  int32_t norm_seqs;           /* G of Eq. 5 for ULORL_NORM_SEQUENCE; 0 means num_seqs                           */
  int32_t dw_dtype;            /* ulorl_dtype_t of d_W: F32 (default), or BF16 -- the sum over tokens is then    */
                               /* still taken in float32 (in the workspace, which grows by 4 V H bytes) and      */
                               /* rounded once when a row of d_W is final.  Part of the workspace size.          */
  float kl_beta;               /* beta of the KL-to-reference term of Eq. 5; 0 (the paper's method, Section 2.3:  */
                               /* the term is removed) leaves ref_logp unread.  With beta > 0 the token term is   */
                               /* s_t - beta k_t, k_t = e^u - u - 1, u = ref_logp[t] - logp[t], inside the mask.  */
} ulorl_params_t;

typedef struct {
  float loss;                  /* -(1/N) sum_t (1 - msk_t) (s_t - kl_beta k_t)                                    */
  float mean_entropy;          /* token mean of the per-token entropy over the call                               */
  int32_t n_tokens, n_active, n_mpt, n_masked, n_clip_high, n_clip_low;
  int32_t stale_tokens[ULORL_N_STALENESS];     /* tokens per staleness bucket (last bucket = that or more)        */
  int32_t stale_clipped[ULORL_N_STALENESS];    /* of which clipped                                                */
  float stale_mean_abs_logratio[ULORL_N_STALENESS];
  int32_t device_status;       /* copy of the workspace status word at the end of the forward call                */
  float mean_kl;               /* token mean of the KL estimate k_t over the call (0 when kl_beta = 0)            */
  int32_t reserved[2];
} ulorl_stats_t;

/* Bytes of workspace both calls need for these params (pure host function; 0 on invalid params). */
size_t ulorl_workspace_bytes(const ulorl_params_t* params);

/*
 * Forward (Eq. 6, 8, 9, 10).  Inputs:
 *   hidden [T,H], W [V,H]  element type params->dtype
 *   targets [T] int32      generated token ids y_t
 *   old_logp [T] f32       log-prob recorded at rollout by the policy that generated the token's
 *                          segment (Eq. 8); may be NULL in POIS mode
 *   ref_logp [T] f32       log-prob of the token under the reference policy of Eq. 5's KL term; read only
 *                          when kl_beta > 0, else may be NULL
 *   segment_version [T]    id of the policy that generated the token's segment (the map f of Eq. 8; statistics
 *                          only); may be NULL
 *   advantages             f32, [num_seqs] or [T] (adv_per_token)
 *   seq_offsets [S+1]      int32, non-decreasing, seq_offsets[0] = 0, seq_offsets[S] = T
 *   entropy_supplied [S]   f32 gate values, read only when ent_scope = SUPPLIED
 * Outputs (all f32 unless noted; any of logp/entropy/lse/grad_coef/flags/seq_entropy must be non-NULL):
 *   logp[T], entropy[T], lse[T], grad_coef[T] (= d loss / d logp_t, saved for bwd),
 *   flags[T] uint8, seq_entropy[S] (H-bar_i), loss[1], stats (ulorl_stats_t, may be NULL).
 */
int ulorl_token_loss_fwd(const ulorl_params_t* params,
                         const void* hidden, const void* W, const int32_t* targets,
                         const float* old_logp, const float* ref_logp, const int32_t* segment_version,
                         const float* advantages, const int32_t* seq_offsets,
                         const float* entropy_supplied,
                         float* logp, float* entropy, float* lse, float* grad_coef,
                         uint8_t* flags, float* seq_entropy, float* loss, void* stats,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The elementwise stage alone (Eq. 8, 9, 10 given per-token log-prob and entropy): per-sequence
 * mean entropy, ratio, mask, clipped surrogate, loss, d loss / d logp.  Same arguments as the
 * forward call with logp[T] and entropy[T] as INPUTS.
 */
int ulorl_token_loss_decide(const ulorl_params_t* params,
                            const float* logp, const float* entropy,
                            const float* old_logp, const float* ref_logp, const int32_t* segment_version,
                            const float* advantages, const int32_t* seq_offsets,
                            const float* entropy_supplied,
                            float* grad_coef, uint8_t* flags, float* seq_entropy, float* loss,
                            void* stats, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same elementwise stage as ulorl_token_loss_decide for callers that cannot hand over a
 * workspace because they cannot allocate device memory at the point of the call: code running
 * inside another framework's step where the allocator is frozen (a memory plan fixed ahead of
 * time, a pool that is full by design), plugins that only receive the tensors of the op they
 * implement, or a process whose memory budget was handed out entirely at start-up.  (The paper
 * has no counterpart to this function; it is a packaging variant, not a step of the method.)
 *
 * The scratch that ulorl_token_loss_decide takes from the caller's workspace (status word,
 * per-sequence 64-bit entropy sums, one partial record per 1024 tokens) lives instead in a fixed
 * array inside the library's device image: about 0.8 MB on every GPU that loads the library,
 * held until the process exits.  Limits: T <= ULORL_STATIC_MAX_TOKENS and num_seqs <=
 * ULORL_STATIC_MAX_SEQS; larger batches are rejected with ULORL_ERR_STATIC_LIMIT (and a message
 * on stderr) before anything is launched.  Inputs and outputs are the caller's device buffers,
 * exactly as for ulorl_token_loss_decide; results are identical.
 *
 * The function calls no allocating routine.  Its first call on a device looks up the device
 * address of the array (one runtime query with that device current) and keeps it; make that
 * first call outside any stream capture.  All calls on a device share the one array, which keeps
 * the previous call's contents (the call clears the status word itself): two calls whose kernels
 * can overlap on the GPU -- different streams without an ordering between them -- race on it and
 * give wrong results.  Calls on one stream are ordered and safe.  Device-side findings (sequence
 * offsets out of order, clamped) land in the array's own status word: read it with
 * ulorl_check_status(NULL, stream), or from stats->device_status.
 */
#define ULORL_STATIC_MAX_TOKENS (1 << 20)
#define ULORL_STATIC_MAX_SEQS   (1 << 16)
int ulorl_token_loss_decide_static(const ulorl_params_t* params,
                                   const float* logp, const float* entropy,
                                   const float* old_logp, const float* ref_logp, const int32_t* segment_version,
                                   const float* advantages, const int32_t* seq_offsets,
                                   const float* entropy_supplied,
                                   float* grad_coef, uint8_t* flags, float* seq_entropy, float* loss,
                                   void* stats, void* cuda_stream);

/*
 * The mean entropy H-bar_i of Eq. 10 when a sequence is cut over several calls or ranks (token-range
 * sharding of an ultra-long response).  The library keeps every per-sequence entropy sum as an exact
 * 64-bit integer in units of 2^-34 nats, so pieces add up to the unsplit sum bit for bit:
 *
 *   ulorl_sequence_entropy_partials  from entropy[T] (the forward's output) and the call's seq_offsets,
 *       fills table[total_seqs][2] = (entropy sum, token count) for the call's pieces -- piece k is global
 *       sequence seq_ids[k] (NULL: k) -- and zeros elsewhere.  Tables of all calls / ranks are then added
 *       element by element (an int64 SUM all-reduce).
 *   ulorl_sequence_entropy_combine   from the summed table, writes seq_entropy[k] = mean of sequence
 *       seq_ids[k], k < num_seqs, in float32 with the arithmetic of the forward call (the value an unsplit
 *       call returns), and optionally batch_entropy[0] = token mean over all sequences.  These go to
 *       ulorl_token_loss_decide as entropy_supplied (ent_scope = SUPPLIED).
 *
 * All pointers are device memory.  workspace may be NULL; if given, its status word reports offsets or
 * ids out of range (they are skipped).
 */
int ulorl_sequence_entropy_partials(const ulorl_params_t* params, const float* entropy,
                                    const int32_t* seq_offsets, const int32_t* seq_ids, int32_t total_seqs,
                                    int64_t* table, void* workspace, void* cuda_stream);
int ulorl_sequence_entropy_combine(const int64_t* table, int32_t total_seqs, const int32_t* seq_ids,
                                   int32_t num_seqs, float* seq_entropy, float* batch_entropy, void* cuda_stream);

/*
 * Group-normalised advantages (Eq. 4) for responses stored group after group (`group_size` responses
 * per prompt, the last group may be shorter): advantages[i] = (R_i - mean) / std over the group,
 * population standard deviation, 0 for a group without spread.  keep[i] (optional) is 1 when the
 * group satisfies the dynamic-sampling constraint of Eq. 7, 0 < #(R == 1) < G.  rewards,
 * advantages [num_responses] f32 and keep [num_responses] uint8 are device pointers; the result
 * is what ulorl_token_loss_fwd takes as per-sequence advantages.
 */
int ulorl_group_advantages(const float* rewards, int32_t num_responses, int32_t group_size,
                           float* advantages, uint8_t* keep, void* cuda_stream);

/*
 * Backward (chain rule through Eq. 6): with dz[t,v] = kappa * grad_loss * grad_coef[t] *
 * (1[v = y_t] - exp(z[t,v] - lse[t])), writes d_hidden[T,H] (params->dtype) and d_W[V,H]
 * (params->dw_dtype, f32 by default; added into when params->dw_accumulate).  grad_loss is a
 * device scalar or NULL (= 1).  Logits are recomputed tile by tile; nothing of size T x V is kept
 * beyond one token panel of dz in the workspace.
 */
int ulorl_token_loss_bwd(const ulorl_params_t* params,
                         const void* hidden, const void* W, const int32_t* targets,
                         const float* lse, const float* grad_coef, const float* grad_loss,
                         void* d_hidden, void* d_W,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same backward for a caller that wants to start moving d_W before the pass is over -- the sum of
 * d_W over data-parallel ranks (the one exchange of the update of Algorithm 1 when whole sequences are
 * sharded), or a copy to the host.  d_W is a sum over all tokens, so its rows are final only while the
 * LAST token panel is processed; there the library computes d_W before d_hidden and in slabs of
 * vocabulary rows (whole waves of tiles, about eight slabs), and calls
 *     on_slab(user, first_row, rows)
 * on the calling host thread right after the launches that make rows [first_row, first_row + rows)
 * of d_W final have been put on cuda_stream.  Nothing has run yet at that point: the callback orders
 * its own work behind those launches (record an event on cuda_stream and make another stream wait for
 * it, or start a collective that orders itself after cuda_stream) and returns; the d_hidden launches of
 * the panel follow on cuda_stream and overlap with it.  The slabs come in ascending row order and cover
 * [0, V) once.  A non-zero return value stops the pass and is returned.  on_slab = NULL gives
 * ulorl_token_loss_bwd.  Results are those of ulorl_token_loss_bwd bit for bit.
 */
typedef int (*ulorl_dw_slab_fn)(void* user, int32_t first_row, int32_t rows);
int ulorl_token_loss_bwd_slabs(const ulorl_params_t* params,
                               const void* hidden, const void* W, const int32_t* targets,
                               const float* lse, const float* grad_coef, const float* grad_loss,
                               void* d_hidden, void* d_W, ulorl_dw_slab_fn on_slab, void* user,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The float32 thresholds the decision stage compares against for these params (pure host function):
 * out[0] = ln tau (Eq. 9 read as logp >= ln tau), out[1] = ln(1 + clip_eps_high), out[2] = ln(1 - clip_eps_low)
 * (the clip bounds of Eq. 7 / Eq. 10 on the log-ratio; -inf when clip_eps_low = 1).  Each is the float64
 * logarithm of the float32 parameter rounded to float32, so that no transcendental sits in a comparison.
 */
int ulorl_decision_thresholds(const ulorl_params_t* params, float* out);

/* Synchronises the stream, reads the workspace status word (workspace = NULL: the status word of the built-in
 * scratch of ulorl_token_loss_decide_static on the current device) and returns it: ULORL_OK, or
 * ULORL_ERR_DEVICE_TIMEOUT, ULORL_ERR_INVALID_ARG (seq_offsets on the device were not
 * 0 = o[0] <= ... <= o[S] = T; the offending ranges were clamped), ULORL_ERR_BAD_TARGET, ULORL_ERR_CUDA. */
int ulorl_check_status(void* workspace, void* cuda_stream);

const char* ulorl_status_string(int status);

/*
 * Self-test of the failure path: launches one small block that waits, with the bounded wait the tensor-core
 * kernels use, on a barrier nobody signals; after limit_cycles SM clocks (1e3 .. 1e8) the wait gives up, the
 * block sets the timeout bit in the workspace status word and returns normally.  ulorl_check_status then
 * reports ULORL_ERR_DEVICE_TIMEOUT; the next forward call clears the word.  Nothing else runs in the block:
 * no copy, no tensor memory, so the context stays usable.
 */
int ulorl_selftest_bounded_wait(void* workspace, int64_t limit_cycles, void* cuda_stream);

/* Number of kernel launches issued by this library since it was loaded (host counter). */
int64_t ulorl_launch_count(void);

/*
 * Per-kernel timing of the four tensor-core kernels (0 online-softmax statistics, 1 dz recompute,
 * 2 d_hidden, 3 d_W).  Between begin and end every such launch is bracketed by a CUDA event pair
 * on its stream; end waits for those events and returns, per kernel, the summed duration in
 * milliseconds (total_ms[4], host) and the number of launches (launches[4], host).  The events are
 * created on first use and kept; this is a measurement aid, not part of the update path.
 */
int ulorl_kernel_timing_begin(void);
int ulorl_kernel_timing_end(float* total_ms, int64_t* launches);

/*
 * One whole step (forward then backward of Eq. 10's objective) for a caller whose buffers live in
 * HOST memory (pinned memory makes the copies asynchronous).  Inputs h_* are copied to the device
 * arena, both passes run there, and every non-NULL output is copied back: h_logp[T], h_entropy[T],
 * h_flags[T], h_seq_entropy[S], h_loss[1], h_stats (ulorl_stats_t), h_d_hidden[T,H] (params->dtype),
 * h_d_W[V,H] (params->dw_dtype).  d_arena is DEVICE memory of at least ulorl_host_step_arena_bytes(params)
 * bytes, owned by the caller and reusable across calls; it holds the device copies, the outputs
 * and the workspace.  Asynchronous on cuda_stream: synchronise the stream before reading outputs
 * or reusing the host buffers.  Copies are overlapped with the passes: a first chunk of hidden states
 * arrives, then W in slabs of vocabulary rows while the statistics kernel already sweeps that chunk
 * against the slabs that have landed, then the other chunks while it runs on those before them; the
 * d_hidden rows of each backward panel leave on an outbound copy stream while the next panel is
 * computed, and on the last panel d_W is computed first and leaves slab by slab under the rest.  The two copy streams and their events are created on
 * the first call and kept for the life of the process; cuda_stream waits for both before the call's
 * work on it is complete.
 */
size_t ulorl_host_step_arena_bytes(const ulorl_params_t* params);
int ulorl_token_loss_step_host(const ulorl_params_t* params,
                               const void* h_hidden, const void* h_W, const int32_t* h_targets,
                               const float* h_old_logp, const float* h_ref_logp, const int32_t* h_segment_version,
                               const float* h_advantages, const int32_t* h_seq_offsets,
                               const float* h_entropy_supplied,
                               float* h_logp, float* h_entropy, uint8_t* h_flags, float* h_seq_entropy,
                               float* h_loss, void* h_stats, void* h_d_hidden, void* h_d_W,
                               void* d_arena, size_t arena_bytes, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ULORL_H_ */
