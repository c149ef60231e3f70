/*
 * libssd -- decision kernels of CTC-draft self-speculative decoding for LLM-based ASR.
 *
 * The library computes, on one CUDA device, what wraps the LLM forward pass in the method:
 *   stage 1 (ssd_ctc_draft, ssd_entropy_gate): from the CTC head's logits, per-frame
 *     log-sum-exp, entropy and greedy argmax; the collapsed draft hypothesis; the
 *     utterance-level entropy gate;
 *   stage 2 (ssd_verify): from the LLM's logits at the draft positions, each draft token's
 *     log-likelihood, the relaxed acceptance rule and the accepted prefix length.
 *
 * Conventions for every call
 *   - All array pointers are DEVICE pointers owned by the caller unless a comment says
 *     "host".  The library allocates nothing, frees nothing and never synchronises: work is
 *     enqueued on `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *   - A batch is ragged: utterance b owns rows [off[b], off[b+1]) of a row-major matrix with
 *     `ld` elements between consecutive rows (ld >= V).  off is int64, off[0] = 0,
 *     off[B] = number of rows.  The row count is also passed as a host scalar so that no
 *     device-to-host read is needed.  B = 0, empty utterances and zero rows are legal.
 *   - Logits are SSD_F32 (IEEE binary32) or SSD_BF16 (bfloat16).  The matrix base must be
 *     aligned to the element size.  All accumulation is fp32.  -inf is a legal (masked)
 *     logit; NaN, +inf or a row of only -inf set SSD_UTT_NONFINITE for the utterance and
 *     leave that row's float outputs unspecified.
 *   - Return value: SSD_OK or an error found on the host before anything was enqueued
 *     (nothing is written in that case).  Problems only visible in the data are reported
 *     per utterance in `utt_status` (bit set, no trap, nothing out of bounds is touched).
 *   - Ties of the argmax go to the lowest index.  Entropy is in nats.
 *   - CUDA graphs: every call only enqueues kernels on `stream` and may be captured into a
 *     graph and replayed with new contents in the same buffers.  Make one call of each kind,
 *     with the same sizes, before capturing (the first use of a kernel sets a function
 *     attribute and looks up device properties).  What a replay cannot renew is the call
 *     number that marks a workspace's error word: after a replay that reported
 *     SSD_UTT_INTERNAL, later replays of the same graph report it too; capture again.
 *     ssd_verify with opts->finish == 2 is refused (SSD_ERR_ARG) while its stream is capturing.
 */
#ifndef SSD_H_
#define SSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { SSD_F32 = 0, SSD_BF16 = 1 } ssd_dtype;

/* return codes */
enum {
    SSD_OK = 0,
    SSD_ERR_NULL = 1,      /* a required pointer is NULL */
    SSD_ERR_ARG = 2,       /* negative size, ld < V, blank_id outside [0,V), bad option ... */
    SSD_ERR_DTYPE = 3,     /* dtype is neither SSD_F32 nor SSD_BF16 */
    SSD_ERR_WORKSPACE = 4, /* workspace NULL or smaller than the *_workspace_bytes() answer */
    SSD_ERR_CUDA = 5,      /* a CUDA runtime call failed; see ssd_last_cuda_error() */
    SSD_ERR_ALIGN = 6,     /* logits base not aligned to the element size */
    SSD_ERR_TOO_LARGE = 7  /* ssd_verify_static: the sizes need more scratch than its fixed array */
};

/* bits of utt_status[b] */
enum {
    SSD_UTT_NONFINITE = 1u,     /* a row of the utterance held NaN / +inf or only -inf */
    SSD_UTT_BAD_DRAFT_ID = 2u,  /* a draft id outside [0,V): treated as rejected, never read */
    SSD_UTT_BAD_OFFSETS = 4u,   /* off[b] < 0, off[b+1] < off[b] or off[b+1] > rows: utterance
                                   treated as empty and never accepted */
    SSD_UTT_INTERNAL = 0x80000000u /* a bounded wait inside a kernel ran out while this utterance
                                      was processed: discard every output of the call */
};

/*
 * Optional launch controls, for tuning and measurement.  Pass NULL for the defaults.  Zero in
 * a field means "choose automatically".  The struct is read on the host during the call only.
 */
typedef struct ssd_launch_opts {
    int32_t kernel;       /* 0 auto; 1 plain-load kernels; 2 bulk-copy (TMA) pipelined kernels */
    int32_t ctas;         /* grid size of the streaming kernel */
    int32_t warps;        /* compute warps per CTA of the streaming kernel */
    int32_t stages;       /* verify: shared-memory pipeline depth */
    int32_t stage_bytes;  /* bytes per pipeline stage (verify) / passes per tile (ctc_draft) */
    int32_t split;        /* verify: column spans per logits row; ctc_draft: lanes per row
                             (2, 4, 8, 16 or 32; refused with SSD_ERR_ARG when a lane would walk
                             more than 160 16-byte chunks of a row) */
    void *ev_begin;       /* cudaEvent_t recorded just before the streaming kernel, or NULL */
    void *ev_end;         /* cudaEvent_t recorded just after the streaming kernel, or NULL */
    int32_t fma_exp;      /* bf16: pairs of exponentials per 16-byte chunk evaluated by a
                             polynomial on the FMA pipe instead of the special-function unit:
                             0 auto; 1..3 that many of the 4 pairs (ctc_draft: at most 2);
                             -1 none */
    int32_t finish;       /* ssd_verify: where a row's log-likelihood and the utterance decisions
                             are finished: 0 auto (the closing kernel); 1 in a closing kernel of
                             their own; 2 inside the streaming kernel, one launch instead of two
                             (refused with SSD_ERR_ARG where that is not possible: column spans,
                             the plain-load kernel, B > 2047, a stream that is capturing) */
} ssd_launch_opts;

/* Human-readable name of a return code (static storage). */
const char *ssd_status_string(int32_t status);

/* cudaError_t of the last failing CUDA call seen by this thread (0 if none). */
int32_t ssd_last_cuda_error(void);

/* Library version, major*10000 + minor*100 + patch. */
int32_t ssd_version(void);

/* Kernels this host thread has launched through the library so far (for launch accounting in
 * benchmarks; the paper has no counterpart). */
uint64_t ssd_launch_count(void);

/* Bytes of device scratch the calls below need for these sizes and options (may be 0). */
size_t ssd_ctc_draft_workspace_bytes(int32_t B, int64_t N, int32_t V, ssd_dtype dtype,
                                     const ssd_launch_opts *opts);
size_t ssd_verify_workspace_bytes(int32_t B, int64_t M, int32_t V, ssd_dtype dtype,
                                  const ssd_launch_opts *opts);

/*
 * Stage 1: CTC draft.  Section 2.1 of the paper.
 *
 * For every frame t (row of `logits`, V = size of the augmented vocabulary incl. blank):
 *   frame_lse[t]     = log sum_a exp(x_ta)          (so log p(a|h_t) = x_ta - frame_lse[t])
 *   frame_entropy[t] = sum_a -p(a|h_t) log p(a|h_t)                     (Eq. 3, left side)
 *   frame_argmax[t]  = argmax_a p(a|h_t)                                (Eq. 2)
 * and for every utterance b the draft hypothesis B(argmax path): consecutive duplicates
 * merged, then blanks removed (in this order, the mapping B of Section 2.1):
 *   draft_tokens[frame_off[b] + k], k < draft_len[b]   the first draft_len[b] tokens
 *   draft_frames[frame_off[b] + k]                     frame index (within the utterance) that
 *                                                      emitted token k            (nullable)
 *   draft_full_len[b] = U, the uncapped length; draft_len[b] = min(U, max_draft_len)
 *   utt_max_entropy[b] = max_t frame_entropy[t] over the utterance (0 if it has no frames)
 *
 * logits         [N, ld] dtype, read once.                          frame_off [B+1] int64
 * frame_entropy  [N] f32   frame_argmax [N] i32   frame_lse [N] f32 (nullable)
 * frame_logprob  [N, ld] f32 dense log-softmax x - lse (nullable; for inspection and tests:
 *                it writes 4*N*V bytes and is not part of the timed path)
 * draft_tokens   [N] i32 (U <= T guarantees the capacity; entries past draft_len[b] inside an
 *                utterance's range are left untouched)
 * draft_len, draft_full_len [B] i32   utt_max_entropy [B] f32   utt_status [B] u32 (overwritten)
 * workspace      NULL, or at least ssd_ctc_draft_workspace_bytes(...) bytes (2,048), 256-byte
 *                aligned: counters from which the streaming kernel's warps claim their tiles
 *                of frames, so that SMs that run ahead take more.  It needs no clearing, before
 *                the first call or between calls (the words carry a per-call tag), but two
 *                calls whose kernels may run at the same time must not share it.  Without it
 *                the tiles are dealt out in a fixed order; the results are the same.
 * Errors: SSD_ERR_NULL, SSD_ERR_ARG (B,N < 0; V < 1; ld < V; blank_id outside [0,V);
 * max_draft_len < 0), SSD_ERR_DTYPE, SSD_ERR_ALIGN, SSD_ERR_WORKSPACE, SSD_ERR_CUDA.
 */
int32_t ssd_ctc_draft(const void *logits, ssd_dtype dtype, int32_t V, int64_t ld,
                      const int64_t *frame_off, int32_t B, int64_t N,
                      int32_t blank_id, int32_t max_draft_len,
                      float *frame_entropy, int32_t *frame_argmax, float *frame_lse,
                      float *frame_logprob,
                      int32_t *draft_tokens, int32_t *draft_frames,
                      int32_t *draft_len, int32_t *draft_full_len,
                      float *utt_max_entropy, uint32_t *utt_status,
                      void *workspace, size_t workspace_bytes, void *stream,
                      const ssd_launch_opts *opts);

/*
 * Stage 1 decision: the entropy gate.  Eq. 3 of the paper: the draft of utterance b is
 * accepted as final iff frame_entropy[t] < tau_ctc for ALL of its frames (strict).
 *   gate_accept[b]  = 1 / 0          (an utterance without frames passes iff 0 < tau_ctc;
 *                                     a NaN entropy or malformed offsets never pass)
 *   max_entropy[b]  = max over the utterance's frames (0 if none)
 *   argmax_frame[b] = first frame attaining it, -1 if none                     (nullable)
 * Two forms:
 *   from frame entropies   utt_max_entropy == NULL (or argmax_frame wanted): frame_entropy [N]
 *                          f32, from ssd_ctc_draft or anywhere else, is read once;
 *   from utterance maxima  utt_max_entropy [B] f32 and utt_status [B] u32 as ssd_ctc_draft left
 *                          them, argmax_frame == NULL: "all frames below tau" is "the maximum is
 *                          below tau", so B values are read instead of N (frame_entropy and
 *                          frame_off are not looked at and may be NULL); an utterance whose
 *                          status has SSD_UTT_NONFINITE, SSD_UTT_BAD_OFFSETS or SSD_UTT_INTERNAL
 *                          set does not pass, exactly as in the first form.
 * Errors: SSD_ERR_NULL, SSD_ERR_ARG, SSD_ERR_CUDA.
 */
int32_t ssd_entropy_gate(const float *frame_entropy, const int64_t *frame_off,
                         int32_t B, int64_t N, float tau_ctc,
                         uint8_t *gate_accept, float *max_entropy, int32_t *argmax_frame,
                         const float *utt_max_entropy, const uint32_t *utt_status,
                         void *stream);

/*
 * Stage 2: LLM verification of the draft.  Eq. 5 and Section 2.3 of the paper.
 *
 * Row i of `logits` (V = LLM vocabulary) is the LLM's output distribution that predicts
 * draft token i of its utterance (the caller has already aligned positions, and passes only
 * the rows at draft positions).  For every row:
 *   row_lse[i]    = log sum_v exp(x_iv)                                        (nullable)
 *   token_logp[i] = x[i, draft_ids[i]] - row_lse[i]   = log p(y_i | y_<i, g)   (Eq. 5)
 * Position i is rejected iff p <= tau_slm, evaluated as token_logp[i] <= log(tau_slm)
 * (accepted iff p > tau_slm, Eq. 5).  For every utterance b with K_b rows:
 *   accepted_len[b] = index (0-based, within the utterance) of the first rejected position,
 *                     K_b if none: the verified prefix has accepted_len[b] tokens and AR
 *                     decoding would resume at that position (the paper's j is this + 1)
 *   all_accepted[b] = (accepted_len[b] == K_b): Eq. 5 holds (vacuously for K_b = 0)
 * tau_slm <= 0 rejects nothing; tau_slm >= 1 rejects everything.  A NaN likelihood or a
 * draft id outside [0,V) is a rejected position.
 * skip [B] u8 (nullable): nonzero = the utterance was already accepted by the gate; its rows
 * are not read, accepted_len = K_b, all_accepted = 1, its token_logp / row_lse untouched.
 *
 * logits [M, ld] dtype, read once    tok_off [B+1] int64    draft_ids [M] i32
 * token_logp [M] f32   accepted_len [B] i32   all_accepted [B] u8   utt_status [B] u32
 * workspace: at least ssd_verify_workspace_bytes(...) bytes, 256-byte aligned.
 * Errors: SSD_ERR_NULL, SSD_ERR_ARG, SSD_ERR_DTYPE, SSD_ERR_ALIGN, SSD_ERR_WORKSPACE,
 * SSD_ERR_CUDA.
 */
int32_t ssd_verify(const void *logits, ssd_dtype dtype, int32_t V, int64_t ld,
                   const int64_t *tok_off, const int32_t *draft_ids, int32_t B, int64_t M,
                   float tau_slm, const uint8_t *skip,
                   float *token_logp, float *row_lse,
                   int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                   void *workspace, size_t workspace_bytes, void *stream,
                   const ssd_launch_opts *opts);

/*
 * ssd_verify that stops reading an utterance once its first rejected position is known.
 * Section 2.3 of the paper needs only j, the FIRST position whose likelihood is <= tau_SLM:
 * the rows after it cannot change the decision.  Rows are visited position by position across
 * all utterances; a row is skipped when a smaller rejected position of its utterance has
 * already been found.  accepted_len and all_accepted are exactly those of ssd_verify;
 * utt_status has those of ssd_verify's bits that the rows read give rise to (a NaN or a bad
 * draft id in a row after the first reject goes unseen).  token_logp / row_lse are
 * written for every row that was read -- always including positions 0 .. accepted_len[b] --
 * and left untouched for the others; which later rows still get read depends on timing.
 *   rows_read[b] (nullable, [B] i32): rows of utterance b that were read; -1 for every
 *   utterance when the call fell back to the full kernel (fewer than four rows per CTA, or
 *   column spans in use), which reads all rows of every verified utterance.
 * Use ssd_verify when the complete token_logp is wanted (e.g. for ssd_threshold_sweep).
 * workspace: at least ssd_verify_early_exit_workspace_bytes(...) bytes, 256-byte aligned.
 * Errors: as ssd_verify.
 */
size_t ssd_verify_early_exit_workspace_bytes(int32_t B, int64_t M, int32_t V, ssd_dtype dtype,
                                             const ssd_launch_opts *opts);
int32_t ssd_verify_early_exit(const void *logits, ssd_dtype dtype, int32_t V, int64_t ld,
                              const int64_t *tok_off, const int32_t *draft_ids, int32_t B,
                              int64_t M, float tau_slm, const uint8_t *skip,
                              float *token_logp, float *row_lse,
                              int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                              int32_t *rows_read,
                              void *workspace, size_t workspace_bytes, void *stream,
                              const ssd_launch_opts *opts);

/*
 * Operating points from one pass.  Section 3.2 of the paper studies tau_CTC in [0.7, 3.0] and
 * tau_SLM in {0.1, 0.2} (Table 1 gives two of the points); both decisions depend on the logits
 * only through the per-utterance maximum entropy (Eq. 3) and the per-token log-likelihoods
 * (Eq. 5), which ssd_ctc_draft / ssd_entropy_gate and ssd_verify leave behind.  For every pair
 * p < P and utterance b:
 *   gate_accept[p*B + b]  = (utt_max_entropy[b] < tau_ctc[p])            (Eq. 3; NaN never passes)
 *   accepted_len[p*B + b] = first i with token_logp[i] <= log(tau_slm[p]), else K_b   (Section 2.3)
 *   all_accepted[p*B + b] = (accepted_len == K_b)                                     (Eq. 5)
 *   counts[3*p + 0..2]    = utterances final by the gate / final by verification only / left
 *                           to the auto-regressive pass                                (nullable)
 * tau_slm[p] <= 0 rejects nothing; a NaN or -inf log-likelihood is a reject otherwise.  The
 * verification outcome is computed for every utterance, gate-accepted or not (token_logp of
 * utterances ssd_verify skipped is whatever the caller left there).  Malformed offsets give
 * accepted_len 0, all_accepted 0.
 * utt_max_entropy [B] f32, token_logp [M] f32, tok_off [B+1] int64: device.
 * tau_ctc, tau_slm [P] f32: HOST arrays, read during the call.
 * gate_accept, all_accepted [P*B] u8, accepted_len [P*B] i32, counts [P*3] i32: device.
 * Errors: SSD_ERR_NULL, SSD_ERR_ARG, SSD_ERR_CUDA.
 */
int32_t ssd_threshold_sweep(const float *utt_max_entropy, const float *token_logp,
                            const int64_t *tok_off, int32_t B, int64_t M,
                            const float *tau_ctc, const float *tau_slm, int32_t P,
                            uint8_t *gate_accept, int32_t *accepted_len, uint8_t *all_accepted,
                            int32_t *counts, void *stream);

/*
 * The final hypothesis, Eq. 7 of the paper, and the hand-over to the auto-regressive pass
 * (Section 2.3; Section 3.2 batches that pass separately).  tokens[tok_off[b] .. tok_off[b+1])
 * is the draft of utterance b in the token space it was verified in.  If Eq. 3 or Eq. 5 holds
 * (gate_accept[b] or all_accepted[b] nonzero) the draft is final; otherwise the hypothesis
 * starts with the verified prefix of accepted_len[b] tokens and the utterance is listed for
 * the auto-regressive pass:
 *   final_tokens  same layout as tokens; the first final_len[b] entries of an utterance are
 *                 written, the rest left untouched
 *   final_len[b]  K_b if final, else accepted_len[b] clamped to [0, K_b]
 *   is_final[b]   1 / 0
 *   ar_count[0]   number of utterances that are not final
 *   ar_utt[k], ar_resume[k], k < ar_count: their ids in ascending order and the length of
 *                 their verified prefix (the position the auto-regressive pass generates first)
 * All pointers device.  tokens, final_tokens [M] i32; final_len, ar_utt, ar_resume [B] i32;
 * is_final [B] u8; ar_count [1] i32.
 * Errors: SSD_ERR_NULL, SSD_ERR_ARG, SSD_ERR_CUDA.
 */
int32_t ssd_assemble(const int32_t *tokens, const int64_t *tok_off, int32_t B, int64_t M,
                     const uint8_t *gate_accept, const int32_t *accepted_len,
                     const uint8_t *all_accepted,
                     int32_t *final_tokens, int32_t *final_len, uint8_t *is_final,
                     int32_t *ar_count, int32_t *ar_utt, int32_t *ar_resume, void *stream);

/*
 * One step of the greedy auto-regressive fallback, Eq. 6 of the paper: for each of R rows of
 * LLM logits (one row per utterance still decoding),
 *   next_token[r] = argmax_v p(v | ...)   (lowest index on ties)
 *   next_logp[r]  = log p(next_token[r] | ...) = x[r, next_token[r]] - row_lse[r]   (nullable)
 *   row_lse[r]    = log sum_v exp(x[r, v])                                           (nullable)
 *   row_status[r] = SSD_UTT_NONFINITE for a row holding NaN / +inf or only -inf      (nullable)
 * logits [R, ld] dtype, read once by the same streaming kernel as ssd_verify, which here also
 * tracks the running maximum and its first position.
 * workspace: at least ssd_greedy_step_workspace_bytes(...) bytes, 256-byte aligned.
 * Errors: SSD_ERR_NULL, SSD_ERR_ARG (also opts->kernel == 1: the plain-load kernel has no
 * arg-max variant), SSD_ERR_DTYPE, SSD_ERR_ALIGN, SSD_ERR_WORKSPACE, SSD_ERR_CUDA.
 */
size_t ssd_greedy_step_workspace_bytes(int64_t R, int32_t V, ssd_dtype dtype,
                                       const ssd_launch_opts *opts);
int32_t ssd_greedy_step(const void *logits, ssd_dtype dtype, int32_t V, int64_t ld, int64_t R,
                        int32_t *next_token, float *next_logp, float *row_lse,
                        uint32_t *row_status, void *workspace, size_t workspace_bytes,
                        void *stream, const ssd_launch_opts *opts);

/*
 * ssd_verify without a workspace argument, for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of ssd_verify, same arithmetic.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a region the host
 * framework forbids allocation in (a real-time audio callback, a plugin sandbox that hands out
 * only the buffers it owns, an embedding runtime whose memory is carved up before start-up), or
 * simply a caller that has no allocator of its own and does not want to size a workspace.
 * ssd_verify asks such a caller for scratch it has no means to provide; this call brings its own.
 *
 * The scratch is a fixed array of SSD_VERIFY_STATIC_SCRATCH_BYTES inside the library's device
 * image.  Every device that loads the library holds that much memory until the process exits,
 * whether or not this function is ever called.  The call itself allocates and frees nothing
 * (no cudaMalloc, no cudaFree, no allocating library routine); inputs and outputs are still
 * the caller's buffers, exactly as for ssd_verify, and the results are the same.
 *
 * Limit: sizes for which ssd_verify_workspace_bytes(B, M, V, dtype, opts) exceeds
 * SSD_VERIFY_STATIC_SCRATCH_BYTES are refused with SSD_ERR_TOO_LARGE before anything is
 * enqueued (with the default options the scratch is 96 or 128 bytes per logits row plus a header,
 * so at least 65,000 rows fit; few rows of a wide vocabulary use more per row and still fit).
 *
 * First call on a device: the function looks up the device address of the array (once per
 * device, under a lock, with the caller's current device).  Make that first call outside any
 * stream capture.  Later calls only read the cached address.  `stream` must belong to the
 * device that is current during the call: the array the kernels get is the current device's.
 *
 * Sharing: all calls on a device use the same array and it keeps whatever the last call left
 * in it.  Nothing in it needs clearing between calls.  Two calls whose kernels can run at the
 * same time on one device (different streams, or different host threads on different streams)
 * overwrite each other's partial sums: keep calls to this function on a device in one stream,
 * or otherwise ordered.
 *
 * Errors: those of ssd_verify except SSD_ERR_WORKSPACE, plus SSD_ERR_TOO_LARGE.
 */
#define SSD_VERIFY_STATIC_SCRATCH_BYTES (8u << 20)
int32_t ssd_verify_static(const void *logits, ssd_dtype dtype, int32_t V, int64_t ld,
                          const int64_t *tok_off, const int32_t *draft_ids, int32_t B, int64_t M,
                          float tau_slm, const uint8_t *skip,
                          float *token_logp, float *row_lse,
                          int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                          void *stream, const ssd_launch_opts *opts);

/*
 * Stage 2 over a vocabulary-parallel LLM head.  Eq. 5 of the paper needs, per draft position,
 * the softmax over the whole LLM vocabulary; when the head's columns are split over R ranks
 * (tensor parallelism), each rank holds logits[:, col0 : col0 + V_local] and the log-sum-exp
 * needs one exchange.  (The paper runs on one GPU and has no such step; the arithmetic is Eq. 5's.)
 *
 * ssd_verify_shard, on every rank: for each row i of a verified utterance
 *   shard_stats[3*i + 0] = max over the local columns of x_iv
 *   shard_stats[3*i + 1] = sum over the local columns of exp(x_iv - that maximum)
 *   shard_stats[3*i + 2] = x[i, draft_ids[i] - col0] if col0 <= draft_ids[i] < col0 + V_local,
 *                          else -inf            (draft_ids are ids in the whole vocabulary)
 * Rows of skipped (or malformed) utterances are not read and their triples are left untouched.
 * logits [M, ld] dtype (this rank's columns), shard_stats [M, 3] f32, workspace as for
 * ssd_verify with V = V_local (ssd_verify_workspace_bytes(B, M, V_local, dtype, opts)).
 *
 * The exchange is the caller's: an all-gather of the R ranks' shard_stats (12 bytes per row)
 * into stats_all [R, M, 3], rank-major, with whatever collective library it uses.
 *
 * ssd_verify_combine, on any rank that wants the decisions: per row
 *   row_lse[i]    = log sum_r shard sums re-based to the global maximum          (nullable)
 *   token_logp[i] = (the draft token's logit, from the rank that owns it) - row_lse[i]
 * then acceptance, accepted_len, all_accepted and utt_status exactly as ssd_verify (a draft id
 * outside [0, V_total) is a rejected position and sets SSD_UTT_BAD_DRAFT_ID).
 * R = 1 with col0 = 0 reproduces ssd_verify.
 * Errors: as ssd_verify; SSD_ERR_ARG also for col0 < 0, R < 1 or V_total < 1.
 */
int32_t ssd_verify_shard(const void *logits, ssd_dtype dtype, int32_t V_local, int64_t ld,
                         int64_t col0, const int64_t *tok_off, const int32_t *draft_ids,
                         int32_t B, int64_t M, const uint8_t *skip, float *shard_stats,
                         void *workspace, size_t workspace_bytes, void *stream,
                         const ssd_launch_opts *opts);
int32_t ssd_verify_combine(const float *stats_all, int32_t R, int64_t V_total,
                           const int64_t *tok_off, const int32_t *draft_ids, int32_t B, int64_t M,
                           float tau_slm, const uint8_t *skip,
                           float *token_logp, float *row_lse,
                           int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                           void *stream);

/*
 * Read-span hooks.  The paper has no counterpart: these are test hooks of this library, host
 * only (no GPU, no stream; base_addr is an integer that is never dereferenced).
 *
 * The bulk-copy kernels fetch 16-byte-aligned ranges, while rows of logits may start anywhere a
 * whole element can (odd vocabulary sizes, column slices).  These functions replay on the host
 * the very address arithmetic those kernels use (one shared header) for a matrix that would
 * start at base_addr, over all of its tiles (ssd_ctc_draft) or rows, column spans and stage
 * parts (ssd_verify, whose streaming kernel ssd_greedy_step shares), and report
 *   lo, hi   the lowest address that would be read and one past the highest
 *   faults   how many tiles / rows break a rule: a read outside the matrix (outside the row,
 *            for ssd_verify), a bulk copy off a 16-byte boundary or larger than its stage, or
 *            reads that do not cover the tile's / row's bytes exactly once
 *   kernel   2: the bulk-copy kernel would run; 1: the plain-load kernel, which indexes
 *            elements one by one (lo, hi are then the matrix's own extent)
 * so a caller -- the tests do -- can assert faults == 0, lo >= base_addr and
 * hi <= base_addr + ((rows - 1) * ld + V) * element size for any shape and misalignment.
 * Errors: SSD_ERR_NULL, SSD_ERR_ARG, SSD_ERR_DTYPE, SSD_ERR_ALIGN (base_addr not a multiple of
 * the element size).
 */
typedef struct ssd_read_span {
    uint64_t lo, hi;
    int64_t faults;
    int32_t kernel;
    int32_t reserved;
} ssd_read_span;
int32_t ssd_ctc_draft_read_span(uint64_t base_addr, ssd_dtype dtype, int32_t V, int64_t ld,
                                int64_t N, const ssd_launch_opts *opts, ssd_read_span *out);
int32_t ssd_verify_read_span(uint64_t base_addr, ssd_dtype dtype, int32_t V, int64_t ld,
                             int64_t M, int32_t B, const ssd_launch_opts *opts,
                             ssd_read_span *out);

#ifdef __cplusplus
}
#endif
#endif /* SSD_H_ */
