/*
 * ssd_oracle.c -- CPU oracle for the draft-and-verify decision path of
 * "Self-Speculative Decoding for LLM-based ASR with CTC Encoder Drafts".
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, sequential,
 * fp64 restatement of the paper's definitions, written so that it can be checked
 * against the paper by eye.  It shares no code with the CUDA library.  Only the
 * test-suite, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * What each function follows:
 *   row statistics   -- Eq. 2 (greedy alignment: per-frame argmax of the CTC
 *                       posterior) and Eq. 3 (frame entropy, natural log), with
 *                       the posterior a softmax over the augmented vocabulary
 *                       (Section 2.1, the text under Eq. 1);
 *   collapse         -- the mapping B of Section 2.1: remove consecutive duplicates,
 *                       then blanks, in this order;
 *   entropy gate     -- Eq. 3: accept iff every frame entropy is < tau_CTC;
 *   verify           -- Eq. 5: token likelihood under the LLM's softmax, accepted iff
 *                       > tau_SLM; Section 2.3: j = first position whose likelihood
 *                       is <= tau_SLM, the verified prefix has j-1 tokens.
 *
 * Arithmetic: every logit is widened exactly to double (a bf16 value is the top 16
 * bits of an IEEE binary32); softmax is the two-pass definition (max, then sum of
 * exponentials); no blocking, fusion or reordering.
 *
 *   threshold sweep  -- the operating-point study of Section 3.2 / Table 1: the gate of
 *                       Eq. 3 and the first reject of Section 2.3 re-evaluated for a list
 *                       of (tau_CTC, tau_SLM) pairs from stored per-utterance maxima and
 *                       per-token log-likelihoods;
 *   assemble         -- Eq. 7: the final hypothesis is the draft if Eq. 3 or Eq. 5 holds,
 *                       else the verified prefix, to be continued by the AR pass;
 *   greedy step      -- one step of Eq. 6's greedy decoding: the most likely next token
 *                       under the LLM's softmax and its log-likelihood.
 *
 * Parity pins (tests/test_oracle_pins.py): closed-form entropies (uniform, one-hot,
 * k-of-V, binary), planted probability vectors, shift invariance, brute-force
 * enumeration of alignments and of collapses on tiny vocabularies, planted reject
 * positions, strictness at exact thresholds, and agreement with scipy's
 * logsumexp / log_softmax / entropy on special cases.  No function here is
 * "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define SSD_REF_F32 0
#define SSD_REF_BF16 1

/* per-utterance status bits (same meaning as the library's, values restated here) */
#define SSD_REF_UTT_NONFINITE 1u
#define SSD_REF_UTT_BAD_DRAFT_ID 2u
#define SSD_REF_UTT_BAD_OFFSETS 4u
#define SSD_REF_UTT_LOGP_P_DISAGREE 0x100u /* oracle only: p<=tau and logp<=ln(tau) differ */

static double ref_load(const void *base, int dtype, int64_t idx) {
    if (dtype == SSD_REF_F32) {
        return (double)((const float *)base)[idx];
    } else {
        uint16_t h = ((const uint16_t *)base)[idx];
        uint32_t w = ((uint32_t)h) << 16;
        float f;
        memcpy(&f, &w, sizeof f);
        return (double)f;
    }
}

/*
 * One softmax row of V logits starting at element index `start` of `base`.
 *   *lse      = log sum_a exp(x_a)
 *   *entropy  = sum_a -p_a log p_a, p_a = exp(x_a - lse)      (Eq. 3; 0 log 0 = 0)
 *   *argmax   = smallest a attaining max_a x_a                 (Eq. 2)
 *   logprob   = x_a - lse for each a (nullable)
 * Returns 1 when lse is finite, 0 otherwise (NaN / +inf entries, or all -inf).
 */
int ssd_ref_row_stats(const void *base, int dtype, int64_t start, int32_t V,
                      double *lse, double *entropy, int32_t *argmax, double *logprob) {
    double m = -INFINITY;
    int32_t arg = 0;
    int bad = 0;
    for (int32_t a = 0; a < V; ++a) {
        double x = ref_load(base, dtype, start + a);
        if (isnan(x) || x == INFINITY) bad = 1;
        if (x > m) { m = x; arg = a; }
    }
    double Z = 0.0;
    for (int32_t a = 0; a < V; ++a) {
        double x = ref_load(base, dtype, start + a);
        Z += exp(x - m);
    }
    double l = m + log(Z);
    double H = 0.0;
    for (int32_t a = 0; a < V; ++a) {
        double x = ref_load(base, dtype, start + a);
        double lp = x - l;
        double p = exp(lp);
        if (p > 0.0) H += -p * lp;
        if (logprob) logprob[a] = lp;
    }
    if (lse) *lse = l;
    if (entropy) *entropy = H;
    if (argmax) *argmax = arg;
    return (!bad && isfinite(l)) ? 1 : 0;
}

/*
 * The mapping B (Section 2.1) on one alignment a[0..T): first merge runs of equal
 * symbols, then drop blanks.  Written as one left-to-right walk: a frame emits its
 * symbol iff the symbol differs from the previous frame's symbol (run start) and is
 * not blank.  out / out_frames (nullable) receive the first min(U, cap) tokens and the
 * frame index of each; returns U, the uncapped length.
 */
int32_t ssd_ref_collapse(const int32_t *a, int64_t T, int32_t blank_id, int32_t cap,
                         int32_t *out, int32_t *out_frames) {
    int32_t U = 0;
    for (int64_t t = 0; t < T; ++t) {
        int run_start = (t == 0) || (a[t] != a[t - 1]);
        if (run_start && a[t] != blank_id) {
            if (U < cap) {
                if (out) out[U] = a[t];
                if (out_frames) out_frames[U] = (int32_t)t;
            }
            ++U;
        }
    }
    return U;
}

static int offsets_ok(const int64_t *off, int32_t b, int64_t total) {
    return off[b] >= 0 && off[b + 1] >= off[b] && off[b + 1] <= total;
}

/*
 * Stage 1 on a ragged batch: rows [frame_off[b], frame_off[b+1]) of the [N, ld]
 * logits belong to utterance b.  Outputs as in the library call of the same name
 * (without the ssd_ref_ prefix), in double where the library has float.
 * draft_tokens / draft_frames are [N]; utterance b writes from frame_off[b] on.
 */
int32_t ssd_ref_ctc_draft(const void *logits, int32_t dtype, int32_t V, int64_t ld,
                          const int64_t *frame_off, int32_t B, int64_t N,
                          int32_t blank_id, int32_t max_draft_len,
                          double *frame_entropy, int32_t *frame_argmax, double *frame_lse,
                          double *frame_logprob /* nullable [N, V] dense */,
                          int32_t *draft_tokens, int32_t *draft_frames /* nullable */,
                          int32_t *draft_len, int32_t *draft_full_len,
                          double *utt_max_entropy, uint32_t *utt_status /* nullable */) {
    if (!logits && N > 0) return 1;
    if (V < 1 || ld < V || B < 0 || N < 0 || blank_id < 0 || blank_id >= V || max_draft_len < 0)
        return 2;
    if (dtype != SSD_REF_F32 && dtype != SSD_REF_BF16) return 3;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b) {
        uint32_t st = 0;
        if (!offsets_ok(frame_off, b, N)) {
            draft_len[b] = 0;
            draft_full_len[b] = 0;
            utt_max_entropy[b] = 0.0;
            if (utt_status) utt_status[b] = SSD_REF_UTT_BAD_OFFSETS;
            continue;
        }
        int64_t t0 = frame_off[b], T = frame_off[b + 1] - t0;
        double hmax = 0.0; /* entropies are >= 0; an empty utterance has max 0 */
        for (int64_t t = 0; t < T; ++t) {
            int64_t r = t0 + t;
            double l, H;
            int32_t arg;
            int ok = ssd_ref_row_stats(logits, dtype, r * ld, V, &l, &H, &arg,
                                       frame_logprob ? frame_logprob + r * (int64_t)V : NULL);
            if (!ok) st |= SSD_REF_UTT_NONFINITE;
            frame_entropy[r] = H;
            frame_argmax[r] = arg;
            if (frame_lse) frame_lse[r] = l;
            if (H > hmax) hmax = H;
        }
        int32_t U = ssd_ref_collapse(frame_argmax + t0, T, blank_id, max_draft_len,
                                     draft_tokens + t0, draft_frames ? draft_frames + t0 : NULL);
        draft_full_len[b] = U;
        draft_len[b] = U < max_draft_len ? U : max_draft_len;
        utt_max_entropy[b] = hmax;
        if (utt_status) utt_status[b] = st;
    }
    return 0;
}

/*
 * Eq. 3 as a decision: gate_accept[b] = 1 iff H_t < tau for every frame t of the
 * utterance, i.e. iff max_t H_t < tau.  max_entropy[b] is that maximum (0 for an empty
 * utterance), argmax_frame[b] (nullable) the first frame attaining it (-1 if empty).
 */
int32_t ssd_ref_entropy_gate(const double *frame_entropy, const int64_t *frame_off,
                             int32_t B, int64_t N, double tau_ctc,
                             uint8_t *gate_accept, double *max_entropy, int32_t *argmax_frame) {
    if (B < 0 || N < 0) return 2;
    for (int32_t b = 0; b < B; ++b) {
        double hmax = 0.0;
        int32_t where = -1;
        int all_below = 1;
        if (offsets_ok(frame_off, b, N)) {
            for (int64_t r = frame_off[b]; r < frame_off[b + 1]; ++r) {
                double H = frame_entropy[r];
                if (!(H < tau_ctc)) all_below = 0;
                if (where < 0 || H > hmax) { hmax = H; where = (int32_t)(r - frame_off[b]); }
            }
            /* an empty utterance has max entropy 0, so it passes iff 0 < tau */
            if (where < 0) all_below = (0.0 < tau_ctc);
        } else {
            all_below = 0; /* malformed offsets: never accepted */
        }
        gate_accept[b] = (uint8_t)all_below;
        max_entropy[b] = hmax;
        if (argmax_frame) argmax_frame[b] = where;
    }
    return 0;
}

/*
 * Stage 2 on a ragged batch: rows [tok_off[b], tok_off[b+1]) of the [M, ld] LLM logits
 * are the distributions that predict draft tokens 0..K_b-1 of utterance b.
 *   token_logp[i] = x[i, draft_ids[i]] - lse_i                         (Eq. 5, in log)
 *   reject_i      = not (p_i > tau_slm), i.e. p_i <= tau_slm, or p_i is NaN  (Eq. 5; 2.3)
 *   accepted_len  = first rejected position (0-based), K_b if none
 *   all_accepted  = (accepted_len == K_b)                              (Eq. 5 holds)
 * The decision is also evaluated as token_logp <= log(tau); a disagreement sets
 * SSD_REF_UTT_LOGP_P_DISAGREE.  tau <= 0 rejects nothing; an out-of-range draft id is a
 * rejected position and is never dereferenced.  skip[b] != 0 (nullable): the utterance
 * is not read, accepted_len = K_b, all_accepted = 1, token_logp untouched.
 */
int32_t ssd_ref_verify(const void *logits, int32_t dtype, int32_t V, int64_t ld,
                       const int64_t *tok_off, const int32_t *draft_ids, int32_t B, int64_t M,
                       double tau_slm, const uint8_t *skip,
                       double *token_logp, double *row_lse /* nullable */,
                       int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status) {
    if (!logits && M > 0) return 1;
    if (V < 1 || ld < V || B < 0 || M < 0) return 2;
    if (dtype != SSD_REF_F32 && dtype != SSD_REF_BF16) return 3;
    double log_tau = tau_slm > 0.0 ? log(tau_slm) : -INFINITY;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b) {
        uint32_t st = 0;
        if (!offsets_ok(tok_off, b, M)) {
            accepted_len[b] = 0;
            all_accepted[b] = 0;
            if (utt_status) utt_status[b] = SSD_REF_UTT_BAD_OFFSETS;
            continue;
        }
        int64_t i0 = tok_off[b];
        int32_t K = (int32_t)(tok_off[b + 1] - i0);
        if (skip && skip[b]) {
            accepted_len[b] = K;
            all_accepted[b] = 1;
            if (utt_status) utt_status[b] = 0;
            continue;
        }
        int32_t first_reject = K;
        for (int32_t i = 0; i < K; ++i) {
            int64_t r = i0 + i;
            double l;
            int ok = ssd_ref_row_stats(logits, dtype, r * ld, V, &l, NULL, NULL, NULL);
            if (!ok) st |= SSD_REF_UTT_NONFINITE;
            if (row_lse) row_lse[r] = l;
            int32_t id = draft_ids[r];
            int reject;
            if (id < 0 || id >= V) {
                st |= SSD_REF_UTT_BAD_DRAFT_ID;
                token_logp[r] = -INFINITY;
                reject = 1;
            } else {
                double lp = ref_load(logits, dtype, r * ld + id) - l;
                double p = exp(lp);
                token_logp[r] = lp;
                /* Eq. 5 accepts iff p > tau; "not accepted" also covers a NaN likelihood,
                 * for which p <= tau (Section 2.3) would be false as well */
                reject = !(p > tau_slm);
                int reject_log = !(lp > log_tau);
                if (tau_slm <= 0.0) { reject = 0; reject_log = 0; }
                if (reject != reject_log) st |= SSD_REF_UTT_LOGP_P_DISAGREE;
            }
            if (reject && i < first_reject) first_reject = i;
        }
        accepted_len[b] = first_reject;
        all_accepted[b] = (uint8_t)(first_reject == K);
        if (utt_status) utt_status[b] = st;
    }
    return 0;
}

/*
 * Operating points from one pass (Section 3.2 sweeps tau_CTC in [0.7, 3.0] with
 * tau_SLM in {0.1, 0.2}).  For pair p and utterance b:
 *   gate_accept[p*B+b]  = (utt_max_entropy[b] < tau_ctc[p])            (Eq. 3: max over frames)
 *   accepted_len[p*B+b] = first i with exp(token_logp[i]) <= tau_slm[p], else K_b  (Section 2.3)
 *   all_accepted[p*B+b] = (accepted_len == K_b)                                     (Eq. 5)
 * counts (nullable) [P,3]: utterances final by the gate / final by verification only /
 * left to the AR pass.  A NaN maximum never passes; a NaN likelihood is a reject;
 * tau_slm <= 0 rejects nothing.  Malformed offsets: accepted_len 0, all_accepted 0.
 */
int32_t ssd_ref_threshold_sweep(const double *utt_max_entropy, const double *token_logp,
                                const int64_t *tok_off, int32_t B, int64_t M,
                                const double *tau_ctc, const double *tau_slm, int32_t P,
                                uint8_t *gate_accept, int32_t *accepted_len,
                                uint8_t *all_accepted, int32_t *counts) {
    if (B < 0 || M < 0 || P < 0) return 2;
    for (int32_t p = 0; p < P; ++p) {
        int32_t n_gate = 0, n_verify = 0, n_ar = 0;
        for (int32_t b = 0; b < B; ++b) {
            int64_t o = (int64_t)p * B + b;
            int g = utt_max_entropy[b] < tau_ctc[p];
            int32_t K = 0, first = 0;
            int all = 0;
            if (offsets_ok(tok_off, b, M)) {
                K = (int32_t)(tok_off[b + 1] - tok_off[b]);
                first = K;
                for (int32_t i = 0; i < K; ++i) {
                    double prob = exp(token_logp[tok_off[b] + i]);
                    int reject = !(prob > tau_slm[p]);
                    if (tau_slm[p] <= 0.0) reject = 0;
                    if (reject) { first = i; break; }
                }
                all = (first == K);
            }
            gate_accept[o] = (uint8_t)g;
            accepted_len[o] = first;
            all_accepted[o] = (uint8_t)all;
            if (g) ++n_gate; else if (all) ++n_verify; else ++n_ar;
        }
        if (counts) { counts[3 * p] = n_gate; counts[3 * p + 1] = n_verify; counts[3 * p + 2] = n_ar; }
    }
    return 0;
}

/*
 * Eq. 7.  tokens[tok_off[b] .. tok_off[b+1]) is the draft of utterance b in the token space it
 * was verified in.  If the gate accepted it (Eq. 3) or every token passed (Eq. 5) the draft is
 * final: final_len = K_b, is_final = 1.  Otherwise the final hypothesis starts with the
 * verified prefix (accepted_len tokens, Section 2.3) and the utterance joins the list for the
 * AR pass: ar_utt (ascending utterance ids), ar_resume (length of the prefix = position the AR
 * pass generates first), *ar_count.  final_tokens has the layout of tokens; only the first
 * final_len[b] entries of an utterance are written.
 */
int32_t ssd_ref_assemble(const int32_t *tokens, const int64_t *tok_off, int32_t B, int64_t M,
                         const uint8_t *gate_accept, const int32_t *accepted_len,
                         const uint8_t *all_accepted,
                         int32_t *final_tokens, int32_t *final_len, uint8_t *is_final,
                         int32_t *ar_count, int32_t *ar_utt, int32_t *ar_resume) {
    if (B < 0 || M < 0) return 2;
    int32_t n = 0;
    for (int32_t b = 0; b < B; ++b) {
        int32_t K = 0;
        if (offsets_ok(tok_off, b, M)) K = (int32_t)(tok_off[b + 1] - tok_off[b]);
        int fin = (gate_accept[b] != 0) || (all_accepted[b] != 0);
        int32_t len = K;
        if (!fin) {
            len = accepted_len[b];
            if (len < 0) len = 0;
            if (len > K) len = K;
        }
        for (int32_t i = 0; i < len; ++i) final_tokens[tok_off[b] + i] = tokens[tok_off[b] + i];
        final_len[b] = len;
        is_final[b] = (uint8_t)fin;
        if (!fin) { ar_utt[n] = b; ar_resume[n] = len; ++n; }
    }
    *ar_count = n;
    return 0;
}

/*
 * One greedy step of Eq. 6 for R independent rows of LLM logits [R, ld]:
 *   next_token[r] = argmax_v p(v | ...) = smallest v attaining the largest logit
 *   next_logp[r]  = log p(next_token[r] | ...) = x_max - lse            (nullable)
 *   row_lse[r]                                                          (nullable)
 * Returns the number of rows whose lse is not finite in *bad_rows (nullable).
 */
int32_t ssd_ref_greedy_step(const void *logits, int32_t dtype, int32_t V, int64_t ld, int64_t R,
                            int32_t *next_token, double *next_logp, double *row_lse,
                            uint8_t *row_bad) {
    if (!logits && R > 0) return 1;
    if (V < 1 || ld < V || R < 0) return 2;
    if (dtype != SSD_REF_F32 && dtype != SSD_REF_BF16) return 3;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t r = 0; r < R; ++r) {
        double l;
        int32_t arg;
        int ok = ssd_ref_row_stats(logits, dtype, r * ld, V, &l, NULL, &arg, NULL);
        next_token[r] = arg;
        if (next_logp) next_logp[r] = ref_load(logits, dtype, r * ld + arg) - l;
        if (row_lse) row_lse[r] = l;
        if (row_bad) row_bad[r] = (uint8_t)!ok;
    }
    return 0;
}

/* Utterances are independent, so the two batch loops above may run one utterance per
 * thread; this sets how many threads they use and returns the count in effect
 * (1 when built without OpenMP).  The arithmetic per utterance is unchanged. */
int32_t ssd_ref_set_threads(int32_t n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
    return (int32_t)omp_get_max_threads();
#else
    (void)n;
    return 1;
#endif
}
