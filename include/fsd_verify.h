/*
 * fsd_verify.h -- C ABI of the batched verification step of Fuzzy Speculative
 * Decoding (FSD) and of strict speculative sampling (SD) on one NVIDIA B200.
 *
 * What a call computes, for every batch row b and candidate position i:
 *   1. P_T[i] = softmax(target_logits[b, i, :]), P_D[i] = softmax(draft_logits[b, i, :])
 *      (Section 4, the two distributions compared by Eq. 4).
 *   2. The divergence D[b, i] = Div(P_T[i], P_D[i]) in nats: Jensen-Shannon
 *      (Appendix C.2, the paper's default), KL(P_T || P_D) (Appendix C.1) or total
 *      variation (Appendix C.3).
 *   3. The acceptance bit: FSD accepts iff D < T (Section 4, Eq. 4; "<=" selectable);
 *      SD accepts iff u_accept < min(1, P_T(x_i)/P_D(x_i)) (Section 3, Eq. 1-2);
 *      rFSD accepts iff either holds (Section 4.3, Eq. 6).
 *   4. accept_len[b] = index of the first rejected position, or gamma (Section 3: the
 *      candidates before the earliest failing test are kept).
 *   5. next_token[b]: FSD draws it from P_T at the rejected position (Section 4);
 *      SD and rFSD from max(0, P_T - P_D) renormalised (Section 3, Eq. 3); when every
 *      candidate was accepted it is drawn from P_T of the extra row gamma.  The draw
 *      is the inverse CDF in vocabulary order at u_sample[b] (smallest k whose
 *      cumulative weight exceeds u * total), or the argmax when FSD_SAMPLE_GREEDY
 *      (Section 6.3).
 * fsd_verify_tree applies the same per-node test to a draft tree (Section 6.4) and
 * returns the deepest root-to-node path whose nodes all pass.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless a parameter says
 *     "host".  The library allocates no device memory: scratch space is the caller's
 *     `workspace`, sized by fsd_workspace_bytes().
 *   - Logit tensors are row-major and contiguous, both of the dtype named in the
 *     options.  Rows whose byte length is a multiple of 16 with 16-byte aligned bases
 *     take the vectorised kernels; any other shape takes a slower scalar kernel.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream).  Outputs are valid once the stream has been synchronised.
 *   - The return value is a host-side status: FSD_OK (0) or a negative FSD_ERR_*.
 *     On error no kernel of the call has run (a launch the runtime refuses, FSD_ERR_CUDA, can
 *     leave a 256-byte memset of the workspace's flag block on the stream; everything that
 *     can fail before that is checked first).  Nothing aborts, throws or traps.
 *   - Conditions found on the device are reported per batch row in row_status.
 *   - -inf logits are legal (probability zero).  A row holding NaN, +inf or no finite
 *     value makes its position's divergence NaN, rejects the position and sets
 *     FSD_ROW_NONFINITE.
 */
#ifndef FSD_VERIFY_H
#define FSD_VERIFY_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* divergence (Appendix C) */
#define FSD_DIV_JS 0
#define FSD_DIV_KL 1   /* KL(P_T || P_D) */
#define FSD_DIV_TV 2
/* acceptance rule */
#define FSD_MODE_FSD  0 /* Section 4, Eq. 4 */
#define FSD_MODE_SD   1 /* Section 3, Eq. 1-3 */
#define FSD_MODE_RFSD 2 /* Section 4.3, Eq. 6 */
/* threshold comparison */
#define FSD_CMP_LT 0    /* accept iff D <  T (as printed in Eq. 4) */
#define FSD_CMP_LE 1    /* accept iff D <= T */
/* replacement-token choice */
#define FSD_SAMPLE_INVCDF 0
#define FSD_SAMPLE_GREEDY 1 /* Section 6.3 */
/* logit storage */
#define FSD_F32  0
#define FSD_BF16 1

/* host status codes */
#define FSD_OK               0
#define FSD_ERR_NULL        -1  /* a required pointer is NULL */
#define FSD_ERR_SHAPE       -2  /* B < 1, gamma/N < 1, V < 1, max_depth < 1, or a size overflows */
#define FSD_ERR_ALIGN       -3  /* a pointer is not aligned to its element size (workspace: 256 bytes) */
#define FSD_ERR_ENUM        -4  /* an option value is out of range, or struct_size is wrong */
#define FSD_ERR_WORKSPACE   -5  /* workspace_bytes is smaller than fsd_workspace_bytes() reports */
#define FSD_ERR_UNSUPPORTED -6  /* combination not defined (SD / rFSD on a tree) */
#define FSD_ERR_CUDA        -7  /* the CUDA runtime refused a launch or a copy */
#define FSD_ERR_TOO_LARGE   -8  /* B * gamma exceeds what the built-in scratch of fsd_verify_chain_static holds */

/* row_status bit flags (device-side conditions) */
#define FSD_ROW_NONFINITE 1  /* some logit row read for this batch row was not a valid distribution */
#define FSD_ROW_TIMEOUT   2  /* a bounded device-side wait ran out; outputs of the row are not valid */
#define FSD_ROW_BADTREE   4  /* parent[] violated -1 <= parent[j] < j */

typedef struct fsd_opts {
    uint32_t struct_size;  /* sizeof(fsd_opts), for versioning */
    int32_t  divergence;   /* FSD_DIV_*    */
    int32_t  mode;         /* FSD_MODE_*   */
    int32_t  compare;      /* FSD_CMP_*    */
    int32_t  sample;       /* FSD_SAMPLE_* */
    int32_t  logit_dtype;  /* FSD_F32 | FSD_BF16 (both tensors) */
    float    threshold;    /* T of Eq. 4, in nats */
} fsd_opts;

/* Fills `opts` with the defaults: JS divergence, FSD rule, "<", inverse-CDF sampling,
 * bf16 logits, T = 0.  Host pointer. */
void fsd_default_opts(fsd_opts *opts);

/* Bytes of device scratch the verify calls need for B batch rows of `positions`
 * candidates each (gamma for a chain, N for a tree).  `bytes_out` is a host pointer.
 * Returns FSD_OK or FSD_ERR_NULL / FSD_ERR_SHAPE / FSD_ERR_ENUM. */
int fsd_workspace_bytes(int B, int positions, int V, const fsd_opts *opts, size_t *bytes_out);

/* Chain verification (Sections 3 and 4).
 *   target_logits [B, gamma+1, V]  row i scores candidate i; row gamma supplies the bonus token
 *   draft_logits  [B, gamma,   V]
 *   draft_tokens  [B, gamma] int32 candidate ids x_i; may be NULL when mode == FSD_MODE_FSD.
 *                 An id outside [0, V) is rejected by the ratio test.
 *   u_accept      [B, gamma] float uniforms in [0,1) for the ratio test; may be NULL in FSD mode
 *   u_sample      [B]        float uniforms in [0,1) for the one token drawn per row
 *   opts          host pointer
 *   accept_len    [B] out    n in [0, gamma]
 *   next_token    [B] out    token id, or -1 if the row it is drawn from is not a valid distribution
 *   divergence    [B, gamma] out, float, computed for every position in every mode
 *   row_status    [B] out    FSD_ROW_* flags
 *   workspace     device scratch, 256-byte aligned, at least fsd_workspace_bytes() bytes;
 *                 contents need not be initialised and are not preserved
 * Calls that share a workspace must be ordered on the stream(s) that use it.
 * The call enqueues a memset and two kernels (the first a cooperative launch of at most one
 * thread block per SM) and nothing else, so it can be captured in a CUDA graph and replayed --
 * after one ordinary call with the same options on that device, which sets the kernels'
 * attributes (that cannot be done under capture). */
int fsd_verify_chain(const void *target_logits, const void *draft_logits,
                     const int32_t *draft_tokens, const float *u_accept, const float *u_sample,
                     int B, int gamma, int V, const fsd_opts *opts,
                     int32_t *accept_len, int32_t *next_token, float *divergence, int32_t *row_status,
                     void *workspace, size_t workspace_bytes, void *stream);

/* Tree verification (Section 6.4; the paper states no rule, this is the reading used).
 *   target_logits [B, N+1, V]  row 0 = distribution after the root context, row j+1 = after node j
 *   draft_logits  [B, N,   V]  row j = distribution node j's token was proposed from
 *   parent        [B, N] int32  parent[j] in [-1, j); -1 = child of the root
 *   u_sample      [B]
 *   max_depth     width of `path`; nodes deeper than max_depth are not eligible
 *   accept_len    [B] out     depth of the chosen node (0 = nothing accepted)
 *   path          [B, max_depth] out  node ids from the root's child down to the chosen node, -1 padded
 *   next_token    [B] out     drawn from the target row after the chosen node (row 0 if none)
 *   divergence    [B, N] out  Div(P_T[row parent(j)+1], P_D[row j])
 * Node j passes iff its divergence passes the threshold test; it is on an accepted path iff it
 * and all its ancestors pass; the chosen node is the deepest such node, ties to the lowest index.
 * Only FSD_MODE_FSD is defined for trees (others: FSD_ERR_UNSUPPORTED).  A row whose parent
 * array is invalid gets FSD_ROW_BADTREE, accept_len 0, next_token -1 and a path of -1. */
int fsd_verify_tree(const void *target_logits, const void *draft_logits,
                    const int32_t *parent, const float *u_sample,
                    int B, int N, int V, int max_depth, const fsd_opts *opts,
                    int32_t *accept_len, int32_t *path, int32_t *next_token, float *divergence,
                    int32_t *row_status, void *workspace, size_t workspace_bytes, void *stream);

/* Chain verification with HOST buffers (same computation as fsd_verify_chain).
 * Every h_* pointer is a HOST pointer (pinned memory makes the copies faster; pageable works).
 * The call copies the inputs into `staging` (device scratch, 256-byte aligned, at least
 * fsd_host_staging_bytes() bytes, owned by the caller), runs fsd_verify_chain on them on
 * `stream`, copies the four outputs back and synchronises the stream before it returns, so the
 * host outputs are valid on return.  h_draft_tokens / h_u_accept may be NULL in FSD mode.
 * Errors as fsd_verify_chain; a failed copy gives FSD_ERR_CUDA. */
int fsd_host_staging_bytes(int B, int gamma, int V, const fsd_opts *opts, size_t *bytes_out);
int fsd_verify_chain_host(const void *h_target_logits, const void *h_draft_logits,
                          const int32_t *h_draft_tokens, const float *h_u_accept, const float *h_u_sample,
                          int B, int gamma, int V, const fsd_opts *opts,
                          int32_t *h_accept_len, int32_t *h_next_token, float *h_divergence,
                          int32_t *h_row_status, void *staging, size_t staging_bytes, void *stream);

/* Chain verification for callers that cannot provide scratch memory.
 * (The paper has no counterpart to this entry point; it exists for integration only.)
 *
 * Some hosts of this library are not allowed to allocate device memory at the point where they
 * verify: a decoding loop whose memory pool was sized and frozen at start-up, a plugin that runs
 * inside another framework's allocator and must not go around it, a serving process whose whole
 * device budget is already handed out.  Such a caller has no buffer to pass as `workspace` and
 * cannot call cudaMalloc to get one.  This variant computes exactly what fsd_verify_chain
 * computes, with the same kernels, but keeps the per-position scratch (accept bits, status words
 * and the 592-byte record of each position) in a fixed array that is part of the library's device image, so the caller passes only inputs and
 * outputs.  It calls no cudaMalloc, cudaFree or any other allocating routine.
 *
 * Limits and rules
 *   - B * gamma must not exceed FSD_STATIC_MAX_POSITIONS; larger calls are refused with
 *     FSD_ERR_TOO_LARGE and nothing is launched.  The array (FSD_STATIC_SCRATCH_BYTES, 768 KiB)
 *     is resident on every GPU that loads the library until the process exits.
 *   - The first call on each device looks up the array's device address (once per device, with
 *     that device current).  Make that first call outside any stream capture.
 *     The address is remembered for the life of the process: do not reset the device
 *     (cudaDeviceReset) between calls; after a reset the remembered address is stale.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left.
 *     Nothing in it has to start at zero: every word a call reads was written earlier by the
 *     same call.  Two calls that overlap on the GPU (different streams, no ordering between
 *     them) race on it and give wrong results; order them, or use fsd_verify_chain with
 *     separate workspaces.
 * Arguments, outputs and the other error codes are those of fsd_verify_chain. */
#define FSD_STATIC_SCRATCH_BYTES 786432
#define FSD_STATIC_MAX_POSITIONS 1024
int fsd_verify_chain_static(const void *target_logits, const void *draft_logits,
                            const int32_t *draft_tokens, const float *u_accept, const float *u_sample,
                            int B, int gamma, int V, const fsd_opts *opts,
                            int32_t *accept_len, int32_t *next_token, float *divergence,
                            int32_t *row_status, void *stream);

/* Human-readable name of a host status code (static storage, never NULL). */
const char *fsd_status_string(int status);

/* Library version: major * 10000 + minor * 100 + patch. */
int fsd_version(void);

/* Measurement aid (no counterpart in the paper).  While an event is set, every verify call
 * records it (cudaEventRecord) on the call's stream between its pair kernel and its finish
 * kernel, so a caller that brackets the call with two events of its own can time the two
 * kernels separately.  `event` is a cudaEvent_t passed as void*, owned by the caller; NULL
 * clears the hook.  Process-wide and not synchronised with calls in flight on other host
 * threads: set it, make the calls to be measured, clear it.  The record between the two
 * kernels also keeps the finish kernel from being set up early, so timings taken with the hook
 * are for attribution, not throughput.  Returns FSD_OK. */
int fsd_set_stage_event(void *event);

/* Test aid (no counterpart in the paper).  Every wait inside the streaming kernel is bounded; a
 * wait that runs out raises a flag in the workspace, the thread blocks that see it take no
 * further work, the call still returns, and every row's row_status carries FSD_ROW_TIMEOUT (its
 * other outputs are then not valid).  mode 1: verify calls raise that flag themselves (a 4-byte
 * memset between the two kernels), which exercises the reporting path alone.  mode 2: in the
 * streaming kernel one thread block keeps its first statistics message to itself and the limit
 * of the exchange wait is lowered to about a tenth of a second, so its partners' wait really
 * runs out and the kernel's own give-up path runs (every wait stays bounded; nothing faults).
 * mode 0: off (the default).  Process-wide, read when a call is made.  Returns FSD_OK, or
 * FSD_ERR_ENUM for another mode. */
int fsd_set_timeout_injection(int mode);

/* Test and tuning aid (no counterpart in the paper).  The streaming kernel splits every
 * (row, position) pair along the vocabulary over a group of 1..16 thread blocks; the library
 * picks the group size from the row length and the number of pairs.  A nonzero `group_size`
 * replaces that choice in later verify calls wherever it is possible (at least the smallest
 * size whose slice fits on chip, at most 16; otherwise the library's own choice stands); 0
 * restores the library's choice.  Results do not depend on the group size beyond the order of
 * floating-point additions.  Process-wide, read when a call is made.  Returns FSD_OK, or
 * FSD_ERR_SHAPE for a size outside 0..16. */
int fsd_set_group_size(int group_size);

/* Debug build (no counterpart in the paper).  A library compiled with -DFSD_DEBUG_CHECKS
 * (python -m paper_2502_20704_b200.build --debug) checks, inside its kernels, the indices and
 * ranges behind its memory accesses -- pair ids, slice and stage bounds of the copies, tensor-
 * memory columns, record and row indices, vocabulary chunks, token ids, tree paths -- and ORs a
 * bit per kind of violation into one int of the workspace; the release build compiles the checks
 * out.  Returns 1 if this library has the checks, else 0; if `word_offset` is not NULL (host
 * pointer) and B, positions >= 1, stores the byte offset of that int inside a workspace for that
 * shape.  The word is zero after a call in which no check failed. */
int fsd_debug_checks(int B, int positions, size_t *word_offset);

/* ---- Threshold tuning (Section "Selecting T"; Discussion, "Potential further developments") ----
 * The paper tunes T on a small development set by running FSD at candidate thresholds and
 * looking at the speed each gives, and notes that FSD's decisions are a deterministic function
 * of the two distributions.  Everything such a sweep needs is in the divergences a verify call
 * returns, so these three helpers work on `divergence` ([B, positions] float, device, row-major,
 * as written by fsd_verify_chain; values >= 0, +inf, or NaN for non-finite inputs) and never touch
 * logits.  The accepted length of a row at threshold T is the index of its first position that
 * fails `D compare T` (NaN never passes); the speed proxy is its mean over the rows.  All pointers
 * are device pointers owned by the caller; the calls are asynchronous on `stream`, allocate
 * nothing and need no workspace.  Errors: FSD_ERR_NULL, FSD_ERR_SHAPE (B < 1, positions < 1,
 * n_thresholds < 1, target negative or NaN), FSD_ERR_ENUM (compare), FSD_ERR_CUDA. */

/* For each of `n_thresholds` candidate thresholds (device array): the mean accepted length over
 * the B rows and the accepted fraction of all B * positions positions. */
int fsd_threshold_sweep(const float *divergence, int B, int positions,
                        const float *thresholds, int n_thresholds, int compare,
                        float *mean_accept_len,   /* [n_thresholds] out */
                        float *accept_fraction,   /* [n_thresholds] out */
                        void *stream);

/* The smallest float T >= 0 whose mean accepted length is at least `target_mean_accept_len`
 * (ceil(target * B) positions accepted, at most B * positions), and the mean it achieves.  +inf if
 * no finite threshold gets there (rows cut short by NaN, or by +inf under FSD_CMP_LT). */
int fsd_calibrate_threshold(const float *divergence, int B, int positions,
                            float target_mean_accept_len, int compare,
                            float *threshold_out,  /* [1] out */
                            float *achieved_out,   /* [1] out: mean accepted length at threshold_out */
                            void *stream);

/* labels[b, i] = 1 if position (b, i) alone passes `D compare threshold`, else 0 (NaN: 0): the
 * token-level accept / reject labels the paper's Discussion proposes to learn from; the prefix
 * rule is not applied. */
int fsd_accept_labels(const float *divergence, int B, int positions, float threshold, int compare,
                      uint8_t *labels,             /* [B, positions] out */
                      void *stream);

#ifdef __cplusplus
}
#endif
#endif /* FSD_VERIFY_H */
