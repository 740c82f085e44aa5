/*
 * libatts - the verification hot path of asynchronous test-time scaling (ATTS) on one B200.
 *
 * The target model scores many parallel draft samples, the scores are ranked against an online
 * calibration set to give conformal p-values, the p-values are thresholded at the rejection rate
 * alpha, and the calibration set grows by the new scores.
 *
 * Conventions for every entry point
 *   - Pointers marked "dev" are device pointers of the current CUDA device, "host" are host
 *     pointers.  The caller owns every buffer, workspaces included; the library allocates no
 *     device memory and keeps no state between calls except a per-process cache of the device's
 *     properties, one device-side status word and the fixed scratch of atts_calib_update_static.
 *   - Every call only enqueues work on `cuda_stream` (a cudaStream_t passed as void*, NULL = the
 *     legacy default stream) and returns; results are valid in stream order, and a sequence of
 *     calls can be captured in a CUDA graph once each entry point has been called once on the
 *     device (the first call probes the device).  The only calls that synchronise are
 *     atts_last_device_status and atts_profile_end.
 *   - The return value is an atts_status.  Argument errors are found before anything is launched
 *     and leave every output untouched.  There is no CPU or non-sm_100 fallback: on another device
 *     the calls return ATTS_ERR_ARCH, without a device ATTS_ERR_CUDA.
 *   - Outputs must not alias inputs.  Sizes of 0 (M, Nc, k) are valid no-ops.
 *   - Results of the conformal calls are bit-reproducible; atts_score_logprob is bit-reproducible
 *     for a given shape on a given device (its reduction order is fixed by a static schedule).
 */
#ifndef ATTS_H_
#define ATTS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ATTS_OK = 0,
  ATTS_ERR_NULL = 1,      /* a required pointer is NULL                                  */
  ATTS_ERR_SHAPE = 2,     /* a size is negative, too large, or not a supported multiple  */
  ATTS_ERR_ALIGN = 3,     /* a pointer is not aligned as documented                      */
  ATTS_ERR_WORKSPACE = 4, /* workspace_bytes is smaller than the matching *_workspace_bytes */
  ATTS_ERR_CAPACITY = 5,  /* n + k exceeds the calibration buffer's capacity             */
  ATTS_ERR_ARG = 6,       /* a scalar argument is out of range (alpha, score_mode)       */
  ATTS_ERR_ARCH = 7,      /* the current device is not sm_100                            */
  ATTS_ERR_CUDA = 8,      /* a CUDA runtime or driver call failed                        */
  ATTS_ERR_TIMEOUT = 9,   /* reported by atts_last_device_status: a bounded device wait expired */
  ATTS_ERR_SCRATCH_LIMIT = 10, /* atts_calib_update_static: the sizes exceed its built-in scratch */
  ATTS_ERR_INDEX = 11     /* reported by atts_last_device_status: a calibration index did not match its buffer */
} atts_status;

/* Bits of the device status word returned by atts_last_device_status. */
#define ATTS_DEV_TOKEN_ID_RANGE 1u /* a token id was outside [0, V): that row's log-prob is NaN */
#define ATTS_DEV_WAIT_EXPIRED 2u   /* a pipeline wait in the scoring kernel ran out; outputs invalid */
#define ATTS_DEV_GROUP_ID_RANGE 4u /* a group id was outside [0, G): that candidate has numer 0 */
#define ATTS_DEV_INDEX_STALE 8u    /* an indexed call was given an index that does not describe fill n; nothing written */

/* Stage labels written by atts_classify (the three stages of the rejection-sampling pipeline,
 * Sec. 3.3): the highest stage a sample reaches in this turn. */
#define ATTS_STAGE_DRAFT 1    /* nothing was verified (the sample has no score)          */
#define ATTS_STAGE_ACCEPTED 2 /* verified and p > alpha: the draft continuation is kept  */
#define ATTS_STAGE_TARGET 3   /* verified and p <= alpha: the target model takes over    */

/* Static string for a status code; never NULL. */
const char* atts_strerror(int status);
/* Library version, major * 10000 + minor * 100 + patch. */
int atts_version(void);

/*
 * Bytes of workspace atts_score_logprob needs for M rows, hidden size d, vocabulary V and S
 * samples on the current device.  host out: *bytes.  The figure depends on the device's SM count.
 */
int atts_score_workspace_bytes(int64_t M, int64_t d, int64_t V, int64_t S, size_t* bytes);

/*
 * Target-model scoring of draft tokens (Sec. 3.3 "Verification"; the score of Sec. 3.2, the equation before
 * Eq. p-value).  Reading adopted: the score handed to the conformal layer is the sample's mean negative
 * log-likelihood under the target model (larger = the target finds the draft less likely), so that p <= alpha
 * rejects the unlikely samples; score modes 2 and 3 give the opposite sign.
 *
 * For every row i (one scored draft token): logits z_i = W h_i over the whole vocabulary,
 * token_logprob[i] = z_i[token_ids[i]] - log sum_v exp(z_i[v]).  The logits are produced tile by
 * tile on the tensor cores and reduced on the fly; the M x V logit matrix is never written to
 * memory.  For every sample k (rows seg_offsets[k] .. seg_offsets[k+1]-1):
 *   score_mode 0: sample_score[k] = -mean(token_logprob)   (mean NLL, the default reading)
 *              1: -sum     2: +mean     3: +sum;            an empty sample scores NaN.
 *
 *   hidden_bf16   dev  [M, d] bf16, row-major, leading dimension d, 16-byte aligned
 *   lm_head_bf16  dev  [V, d] bf16, row-major (one row per vocabulary entry), 16-byte aligned
 *   token_ids     dev  [M] int32, each in [0, V); an id outside sets ATTS_DEV_TOKEN_ID_RANGE and
 *                      yields NaN for that row
 *   seg_offsets   dev  [S + 1] int32, 0 = o_0 <= o_1 <= ... <= o_S = M (not checked on the device
 *                      beyond clamping to [0, M])
 *   M, d, V, S         0 <= M <= 2^30, d a multiple of 64 with 64 <= d <= 16384 (the fp32 accumulation error of
 *                      a logit grows with d; 2e-3 on the log-probs was verified up to this size), 1 <= V < 2^31,
 *                      0 <= S
 *   token_logprob dev  [M] fp32 out, may be NULL
 *   sample_score  dev  [S] fp32 out, may be NULL when S == 0
 *   workspace     dev  256-byte aligned scratch of at least atts_score_workspace_bytes(...);
 *                      contents are undefined afterwards
 * Arithmetic: bf16 x bf16 products accumulated in fp32 (tcgen05), fp32 exponentials and sums,
 * fp64 accumulation of the per-sample sum.
 */
int atts_score_logprob(const void* hidden_bf16, const void* lm_head_bf16, const int32_t* token_ids,
                       const int32_t* seg_offsets, int64_t M, int64_t d, int64_t V, int64_t S,
                       int32_t score_mode, float* token_logprob, float* sample_score,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Scoring with a per-row factor on the logits: z_i = row_scale[i] * (W h_i).  This is the LM head applied to
 * an RMS-normalised hidden state (the step just before the path, Sec. 3.3 "Verification": the target's final
 * norm) without materialising the normalised copy: row_scale[i] = 1 / sqrt(mean(h_i^2) + eps) from
 * atts_rms_inv, and the norm's gain vector folded into the columns of lm_head by the caller.  The factor is
 * folded into the exponent's scale in the epilogue, so the cost is that of atts_score_logprob.
 *   row_scale     dev  [M] fp32, each finite and > 0 (a row with another value has an undefined result)
 * Everything else as atts_score_logprob.
 */
int atts_score_logprob_scaled(const void* hidden_bf16, const void* lm_head_bf16, const int32_t* token_ids,
                              const float* row_scale, const int32_t* seg_offsets, int64_t M, int64_t d,
                              int64_t V, int64_t S, int32_t score_mode, float* token_logprob,
                              float* sample_score, void* workspace, size_t workspace_bytes,
                              void* cuda_stream);

/*
 * Scoring with the vocabulary sharded over GPUs (W split by rows, as a tensor-parallel LM head is).  Each
 * rank runs atts_score_slice on its rows of W and gets, per scored token, the triple
 *   slice_stats[i] = { max_v z_iv,  sum_v exp(z_iv - max),  z_i[token_ids[i]] or -inf if that id is not in
 *                      [vocab_offset, vocab_offset + V_slice) }
 * over its slice (same fused kernel, logits never stored).  The ranks exchange their [M, 3] blocks (an
 * all-gather of 12 bytes per token; this library does not communicate), and atts_score_combine merges G
 * blocks laid out [G][M][3] into token log-probs and sample scores exactly as atts_score_logprob merges
 * its own vocabulary chunks: LSE = Mx + log sum_g l_g exp(m_g - Mx).  A token id that no slice holds sets
 * ATTS_DEV_TOKEN_ID_RANGE and yields NaN.
 *   workspace of atts_score_slice: atts_score_workspace_bytes(M, d, V_slice, 0);
 *   workspace of atts_score_combine: at least 4 * M + 512 bytes, 256-byte aligned.
 * Other arguments as atts_score_logprob.
 */
int atts_score_slice(const void* hidden_bf16, const void* lm_head_slice_bf16, const int32_t* token_ids,
                     int64_t M, int64_t d, int64_t V_slice, int64_t vocab_offset, float* slice_stats,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);
int atts_score_combine(const float* slice_stats, int64_t G, const int32_t* seg_offsets, int64_t M, int64_t S,
                       int32_t score_mode, float* token_logprob, float* sample_score, void* workspace,
                       size_t workspace_bytes, void* cuda_stream);

/*
 * row_scale[i] = 1 / sqrt(mean_k hidden[i, k]^2 + eps), fp32 accumulation.
 *   hidden_bf16   dev  [M, d] bf16 row-major, 16-byte aligned, d a multiple of 8;  eps >= 0
 *   row_scale     dev  [M] fp32 out
 */
int atts_rms_inv(const void* hidden_bf16, int64_t M, int64_t d, float eps, float* row_scale,
                 void* cuda_stream);

/*
 * Marginal conformal p-value by rank (Eq. p-value, Proposition 1):
 *   numer[j]  = 1 + #{ i < n : calib_sorted[i] >= scores[j] },  pvalue[j] = numer[j] / (n + 1).
 * Ties count.  A NaN calibration score (sorted last) counts for every candidate; a NaN candidate
 * has no score: numer = 0, pvalue = NaN.
 *
 *   scores        dev  [Nc] fp32, 16-byte aligned
 *   calib_sorted  dev  [n] fp32 ascending, NaNs last (as atts_calib_update leaves it); may be NULL
 *                      when n == 0
 *   Nc, n              0 <= Nc < 2^31, 0 <= n < 2^24 - 1 (so that n + 1 is exact in fp32)
 *   numer         dev  [Nc] uint32 out, 16-byte aligned
 *   pvalue        dev  [Nc] fp32 out (one correctly rounded fp32 division), 16-byte aligned, may be NULL
 * A pointer that is not aligned as stated is refused with ATTS_ERR_ALIGN before anything is launched.
 */
int atts_conformal_rank(const float* scores, int64_t Nc, const float* calib_sorted, int64_t n,
                        uint32_t* numer, float* pvalue, void* cuda_stream);

/*
 * Threshold at the rejection rate alpha and ordinal stage label (acceptance rule after
 * Eq. p-value, Eq. prediction_set, the three stages of Sec. 3.3).  With
 * k_alpha = floor(alpha * (n + 1)) evaluated in IEEE double on the host:
 *   numer == 0             -> ATTS_STAGE_DRAFT
 *   1 <= numer <= k_alpha  -> ATTS_STAGE_TARGET    (p <= alpha)
 *   otherwise              -> ATTS_STAGE_ACCEPTED  (p >  alpha)
 *
 *   numer         dev  [Nc] uint32, as written by atts_conformal_rank for the same n, 16-byte aligned
 *   alpha              0 < alpha < 1, else ATTS_ERR_ARG
 *   stage         dev  [Nc] uint8 out, 16-byte aligned (ATTS_ERR_ALIGN otherwise)
 *   stage_counts  dev  [3] uint32 out (numbers of samples in stages 1, 2, 3; the third is the
 *                      budget B of "Budget Prediction"), overwritten; may be NULL
 */
int atts_classify(const uint32_t* numer, int64_t Nc, int64_t n, double alpha, uint8_t* stage,
                  uint32_t* stage_counts, void* cuda_stream);

/*
 * atts_conformal_rank and atts_classify for up to four rejection rates in one launch (the
 * conformal-only workload thresholds the same p-values at several alpha).  Outputs are byte for
 * byte those of one atts_conformal_rank call followed by n_alpha atts_classify calls.
 *
 *   alphas        host [n_alpha] double, each in (0, 1); 1 <= n_alpha <= 4
 *   numer, pvalue      as atts_conformal_rank
 *   stage         dev  [n_alpha][Nc] uint8 out (row a holds the stages at alphas[a]), 16-byte
 *                      aligned; with n_alpha > 1, Nc must be a multiple of 16 so that every row is
 *   stage_counts  dev  [n_alpha][3] uint32 out, overwritten; may be NULL
 */
int atts_rank_classify(const float* scores, int64_t Nc, const float* calib_sorted, int64_t n,
                       const double* alphas, int32_t n_alpha, uint32_t* numer, float* pvalue,
                       uint8_t* stage, uint32_t* stage_counts, void* cuda_stream);

/*
 * Budget report ("Budget Prediction", Sec. 3.2: B is the number of candidates that are rejected; "Target
 * Sampling", Sec. 3.3: the target model continues exactly those): the positions of the samples whose stage is
 * ATTS_STAGE_TARGET, ascending, and their number B.
 *
 *   stage         dev  [Nc] uint8, as written by atts_classify (a row of atts_rank_classify's output); only the value
 *                      ATTS_STAGE_TARGET counts, any other byte value is skipped.  Any alignment: the kernel reads the
 *                      aligned 16-byte pieces that hold the array, so up to 15 bytes before stage[0], inside the
 *                      piece that holds it, are read and ignored
 *   ids           dev  [ids_cap] int32 out: the first min(B, ids_cap) positions; may be NULL when ids_cap == 0
 *   count         dev  [1] uint32 out: B (also when B > ids_cap); may be NULL
 *   workspace     dev  256-byte aligned, at least atts_takeover_ids_workspace_bytes(Nc) bytes
 */
int atts_takeover_ids_workspace_bytes(int64_t Nc, size_t* bytes);
int atts_takeover_ids(const uint8_t* stage, int64_t Nc, int32_t* ids, int64_t ids_cap, uint32_t* count,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Threshold form of the acceptance rule (the quantile-threshold construction of the classic set-up,
 * Eqs. quantile / pred_set, read for the rejection side): with tau = the k_alpha-th largest calibration
 * score, k_alpha = floor(alpha * (n + 1)), a sample is rejected iff s > tau - exactly the samples with
 * numer <= k_alpha, ties included.  k_alpha = 0 gives tau = +inf (nobody can be rejected).
 *   tau           dev  [1] fp32 out
 */
int atts_threshold(const float* calib_sorted, int64_t n, double alpha, float* tau, void* cuda_stream);

/*
 * Stages from one comparison per sample against *tau (no rank, no p-value): ATTS_STAGE_TARGET if s > tau,
 * ATTS_STAGE_DRAFT if s is NaN, else ATTS_STAGE_ACCEPTED.  Same bytes as atts_conformal_rank followed by
 * atts_classify for the alpha that produced tau.
 *   scores dev [Nc] fp32 (16-byte aligned); tau dev [1]; stage dev [Nc] uint8 out (16-byte aligned);
 *   stage_counts dev [3] uint32 out, overwritten, may be NULL (the third is the budget B)
 */
int atts_classify_threshold(const float* scores, int64_t Nc, const float* tau, uint8_t* stage,
                            uint32_t* stage_counts, void* cuda_stream);

/*
 * Conditional conformal p-value (Proposition 2; Sec. 3.2: "adjusting the comparison with the ... calibration
 * set from the current input sample"): candidate j is ranked only against the calibration scores of its own
 * input group_ids[j].  Reading adopted: the same count as the marginal form over the group's scores,
 *   numer[j] = 1 + #{ i in group : calib[i] >= scores[j] },  denom[j] = |group| + 1,  p = numer / denom.
 *   scores        dev  [Nc] fp32;  group_ids dev [Nc] int32 in [0, G) (outside: ATTS_DEV_GROUP_ID_RANGE, numer 0)
 *   calib_segments dev [calib_total] fp32: the groups' scores one after the other, each group ascending (NaNs last)
 *   calib_total   number of entries of calib_segments, < 2^31
 *   seg_offsets   dev  [G + 1] int32, group g is calib_segments[seg_offsets[g] .. seg_offsets[g+1]); a group whose
 *                      offsets are not 0 <= seg_offsets[g] <= seg_offsets[g+1] <= calib_total is never read: its
 *                      candidates get numer 0 and ATTS_DEV_GROUP_ID_RANGE is recorded
 *   numer, denom  dev  [Nc] uint32 out;  pvalue dev [Nc] fp32 out, may be NULL
 * Every array 4-byte aligned; 16-byte aligned scores, group_ids and outputs take 128-bit loads and stores, a 32-byte
 * aligned calib_segments 256-bit loads.
 */
int atts_conformal_rank_conditional(const float* scores, const int32_t* group_ids, int64_t Nc,
                                    const float* calib_segments, int64_t calib_total, const int32_t* seg_offsets,
                                    int64_t G, uint32_t* numer, uint32_t* denom, float* pvalue, void* cuda_stream);

/*
 * atts_classify with every candidate's own denominator: reject iff 1 <= numer <= floor(alpha * denom)
 * (IEEE double).  stage / stage_counts as atts_classify.
 */
int atts_classify_conditional(const uint32_t* numer, const uint32_t* denom, int64_t Nc, double alpha,
                              uint8_t* stage, uint32_t* stage_counts, void* cuda_stream);

/* Bytes of workspace atts_calib_update needs to insert k scores into a buffer holding n. */
int atts_calib_workspace_bytes(int64_t n, int64_t k, size_t* bytes);

/*
 * Online calibration (Sec. 3.2 "Online Calibration"): the calibration set grows by k new scores.
 * The set is kept as an ascending fp32 array; after the call (in stream order) calib[0 .. n+k) is
 * the sorted union, as a multiset, of the old n entries and the k new ones.  -0.0 is stored as
 * +0.0 and every NaN as 0x7FC00000, sorted last, so the result is a unique bit pattern.  Nothing
 * is evicted.
 *
 *   calib         dev  fp32 buffer of `cap` elements, the first n ascending (NaNs last); updated
 *                      in place
 *   n, cap, k          0 <= n, 0 <= k, n + k <= cap (else ATTS_ERR_CAPACITY), cap < 2^24 - 1
 *   new_scores    dev  [k] fp32, any order; may be NULL when k == 0
 *   n_out         host out, may be NULL: n + k
 *   workspace     dev  256-byte aligned scratch of at least atts_calib_workspace_bytes(n, k)
 */
int atts_calib_update(float* calib, int64_t n, int64_t cap, const float* new_scores, int64_t k,
                      int64_t* n_out, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Calibration index (a convenience of this library for speed; the paper has no counterpart; results are
 * those of Eq. p-value, byte for byte what atts_rank_classify writes).
 *
 * Ranking many candidates against a buffer too large for shared memory is bound by the divergent loads
 * of each candidate's search.  An index kept beside the buffer - a copy of the buffer, the last entry of every
 * aligned group of 8, 64, ... entries, and the coarsest of those levels laid out as a search tree - lets a
 * candidate finish with one to four 32-byte loads (one up to n = 262,143, two up to 2,097,151, three up to
 * 16,776,703).  The index
 * holds all of this twice: an update reads the half that describes the present fill and writes the other half
 * and the caller's buffer in one pass, so it needs no copy back, and it touches nothing that a rank of the fill
 * it started from reads.  The calibration state of a caller that uses these calls is the buffer AND its index:
 * both describe the same fill n.
 *
 *   atts_calib_index_bytes   host out *bytes: size of an index for buffers of up to `cap` entries,
 *                            0 <= cap < 2^24 - 1 (about 9.2 bytes per entry plus 256 KB)
 *   index         dev  256-byte aligned; index_bytes: the size of that allocation, the same value in every call
 *                      (the layout is derived from it); too small for n (+ k): ATTS_ERR_WORKSPACE
 *   atts_calib_index_build   makes `index` describe calib_sorted[0, n) (a buffer filled some other way, or the
 *                            start of a sequence)
 *   atts_calib_update_indexed   arguments and result as atts_calib_update; `index` must describe calib[0, n)
 *                            when the call runs and describes calib[0, n + k) afterwards, and it still holds
 *                            the description of fill n until the next update.  If it does not describe fill n,
 *                            nothing is changed and ATTS_DEV_INDEX_STALE is recorded.  (Small updates -
 *                            n <= 28,672, k <= 4096, 8 k <= n + 64 - and k == 0 rebuild the index from the
 *                            buffer instead and need no valid index.)
 *   atts_rank_classify_indexed  arguments and outputs as atts_rank_classify, but n_alpha may be 0 (rank and
 *                            p-values only; stage and stage_counts are then ignored).  With n > 8191 and
 *                            Nc >= 16384 the candidates are ranked against the index's own copy of the buffer
 *                            (calib_sorted is not read).  If `index` does not describe fill n nothing is written
 *                            and ATTS_DEV_INDEX_STALE is recorded (atts_last_device_status then returns
 *                            ATTS_ERR_INDEX).
 *                            With stage_counts the call gathers the counts in a few words of the index header
 *                            (which is why `index` is not const): two such calls on one index must not overlap.
 * Overlap: atts_rank_classify_indexed for fill n and the atts_calib_update_indexed that starts from fill n may run
 * at the same time (different streams).  The update after that one overwrites what that rank reads: order it
 * behind the rank.
 * Both kernels are launched with programmatic stream serialisation: they may be set up on the SMs while the kernel
 * before them in the stream drains, and wait for its completion before they read anything.
 */
int atts_calib_index_bytes(int64_t cap, size_t* bytes);
int atts_calib_index_build(const float* calib_sorted, int64_t n, void* index, size_t index_bytes, void* cuda_stream);
int atts_calib_update_indexed(float* calib, int64_t n, int64_t cap, const float* new_scores, int64_t k, int64_t* n_out,
                              void* index, size_t index_bytes, void* workspace, size_t workspace_bytes,
                              void* cuda_stream);
int atts_rank_classify_indexed(const float* scores, int64_t Nc, const float* calib_sorted, int64_t n,
                               void* index, const double* alphas, int32_t n_alpha, uint32_t* numer,
                               float* pvalue, uint8_t* stage, uint32_t* stage_counts, void* cuda_stream);

/*
 * Allocation-free variant of atts_calib_update (a convenience of this library; the paper has no
 * counterpart).  Same result, bit for bit, but the caller passes no workspace: the scratch is a
 * fixed array inside the library's device image.
 *
 * Who this is for: code that runs where device memory can no longer be obtained - a plug-in of a
 * serving engine that has claimed nearly all of HBM for its KV cache at start-up, a control loop
 * that must not call cudaMalloc because that call synchronises the whole device and would stall the
 * asynchronous pipeline this method exists to keep busy, or a component that is simply handed a
 * stream and a few pointers and owns no allocator.  This entry point never calls cudaMalloc,
 * cudaFree or any other allocating routine.
 *
 * Limits: n + k <= ATTS_STATIC_MAX_TOTAL and k <= ATTS_STATIC_MAX_NEW, else
 * ATTS_ERR_SCRATCH_LIMIT and nothing is launched (use atts_calib_update with a workspace then).
 * Cost: every device that loads the library holds the array (ATTS_STATIC_SCRATCH_BYTES) until the
 * process exits, whether or not this entry point is ever called.
 *
 * Set-up: the first call on each device looks up the array's device address (with that device
 * current).  Make that first call during start-up, before any stream capture is begun.
 * Sharing: all calls on a device use the same array, and it keeps whatever the last call left in
 * it.  Nothing in it needs to start at zero (each call overwrites every element it later reads),
 * but two calls whose work overlaps on the GPU - different streams, or different host threads
 * without ordering between them - race on it and corrupt each other's result.  Issue them on one
 * stream, or order them with events.
 *
 * Arguments as for atts_calib_update, minus the workspace.
 */
#define ATTS_STATIC_MAX_TOTAL 65536
#define ATTS_STATIC_MAX_NEW 16384
#define ATTS_STATIC_SCRATCH_BYTES (4 * ATTS_STATIC_MAX_TOTAL)
int atts_calib_update_static(float* calib, int64_t n, int64_t cap, const float* new_scores, int64_t k,
                             int64_t* n_out, void* cuda_stream);

/*
 * Waits for `cuda_stream`, then returns in *bits (host out) the OR of the ATTS_DEV_* conditions
 * device code has recorded on the current device since the last call, and clears them.  Returns
 * ATTS_ERR_TIMEOUT if ATTS_DEV_WAIT_EXPIRED is among them, else ATTS_ERR_INDEX if ATTS_DEV_INDEX_STALE is,
 * else ATTS_OK.
 */
int atts_last_device_status(void* cuda_stream, uint32_t* bits);

/*
 * Schedule inspection (diagnostic; the paper has no counterpart; needs no device).  The static schedule the
 * fused kernel would use for M x d x V with `workers` concurrent workers of `ctas` (1 or 2) CTAs each:
 *   atts_debug_score_plan: out[0..8) = {row blocks, vocabulary tiles, k blocks, chunks per row block,
 *                          row blocks per panel, units, padded rows, ctas}
 *   atts_debug_score_unit: out[0..4) = {row block, chunk, first tile, one past the last tile} of unit u
 * Both return ATTS_ERR_SHAPE / ATTS_ERR_ARG for sizes atts_score_logprob would reject.
 */
int atts_debug_score_plan(int64_t M, int64_t d, int64_t V, int32_t workers, int32_t ctas, int32_t* out);
int atts_debug_score_unit(int64_t M, int64_t d, int64_t V, int32_t workers, int32_t ctas, int32_t u,
                          int32_t* out);

/*
 * Bounded waits of the scoring kernel (diagnostic; the paper has no counterpart).  Every wait inside
 * atts_score_logprob's fused kernel (for a shared-memory stage to fill or drain, for an accumulator to complete or be
 * read) gives up after a number of SM cycles; the kernel then stops, lets copies in flight land, frees its tensor
 * memory and returns, ATTS_DEV_WAIT_EXPIRED is recorded and atts_last_device_status returns ATTS_ERR_TIMEOUT.  The
 * outputs of such a call are invalid; the context stays usable.
 *   atts_debug_set_wait   limit_cycles > 0: the bound for later calls in this process (default 4e9, about two seconds;
 *                         the environment variable ATTS_WAIT_LIMIT presets it); limit_cycles <= 0: the default.
 *                         withhold_loads = 1: the kernel's producer issues no loads at all, so the first wait for data
 *                         can never be satisfied and must run out - the way to exercise the expiry path without a
 *                         fault (nothing is in flight when the kernel gives up); 0: normal operation.
 *   atts_debug_score_form host out *ctas: 1 if atts_score_logprob would run M x d x V on single CTAs on the current
 *                         device, 2 if on CTA pairs.
 */
int atts_debug_set_wait(int64_t limit_cycles, int32_t withhold_loads);
int atts_debug_score_form(int64_t M, int64_t d, int64_t V, int32_t* ctas);

/*
 * Timing hooks (measurement aid; the paper has no counterpart).  Between atts_profile_begin and
 * atts_profile_end every atts_score_logprob call records a pair of CUDA events on its stream
 * directly around the fused LM-head kernel, for at most `max_records` calls (<= 4096).
 * atts_profile_end waits for the recorded events, writes the kernel durations in milliseconds to
 * ms[0 .. min(*count, cap)) (host), sets *count (host) to the number of recorded launches and
 * releases the events.  Not thread-safe; one profiling session per process at a time.
 */
int atts_profile_begin(int max_records);
int atts_profile_end(float* ms, int cap, int* count);

#ifdef __cplusplus
}
#endif
#endif /* ATTS_H_ */
