// The C ABI of libssd: argument validation and dispatch.  Every step of the path runs in the
// kernels of ssd_ctc.cu and ssd_verify.cu; nothing here computes.
#include <map>
#include <mutex>
#include <utility>

#include "ssd_common.cuh"

namespace ssd {
namespace {
constexpr int kMaxDevices = 64;
std::mutex g_mutex;
int g_sm_count[kMaxDevices];                                   // 0: not asked yet
std::map<std::pair<const void *, int>, size_t> g_smem_set;     // (kernel, device) -> bytes set
thread_local int t_replay = 0;
}  // namespace

PlanReplay::PlanReplay() { ++t_replay; }
PlanReplay::~PlanReplay() { --t_replay; }

int device_sm_count() {
    if (t_replay > 0) return 148;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_sm_count[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            return 0;
        g_sm_count[dev] = n;
    }
    return g_sm_count[dev];
}

cudaError_t ensure_dynamic_smem(const void *kernel, size_t bytes) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(g_mutex);
    size_t &have = g_smem_set[std::make_pair(kernel, dev)];
    if (bytes <= have) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) have = bytes;
    return e;
}

static thread_local int32_t t_last_cuda_error = 0;
void record_cuda_error(cudaError_t e) { t_last_cuda_error = (int32_t)e; }
static thread_local uint64_t t_launches = 0;
void count_launch() { ++t_launches; }
}  // namespace ssd

using namespace ssd;

// The plan behind a call or a workspace query.  The shape of a launch depends on the device's
// SM count; where no device can be asked (a host-only build step, an argument check without a
// GPU) the plan is the one for the 148-SM part the kernels are tuned for, and a launch that
// follows fails with SSD_ERR_CUDA.
static int plan_for_query(int B, int64_t M, int V, ssd_dtype dtype, const ssd_launch_opts *opts,
                          VerifyPlan *plan) {
    if (device_sm_count() > 0) return plan_verify(B, M, V, dtype, opts, plan);
    PlanReplay replay;
    return plan_verify(B, M, V, dtype, opts, plan);
}

extern "C" {

const char *ssd_status_string(int32_t status) {
    switch (status) {
        case SSD_OK: return "SSD_OK";
        case SSD_ERR_NULL: return "SSD_ERR_NULL: a required pointer is NULL";
        case SSD_ERR_ARG: return "SSD_ERR_ARG: invalid size, leading dimension, id or option";
        case SSD_ERR_DTYPE: return "SSD_ERR_DTYPE: dtype must be SSD_F32 or SSD_BF16";
        case SSD_ERR_WORKSPACE: return "SSD_ERR_WORKSPACE: workspace missing, misaligned or too small";
        case SSD_ERR_CUDA: return "SSD_ERR_CUDA: a CUDA runtime call failed";
        case SSD_ERR_ALIGN: return "SSD_ERR_ALIGN: logits not aligned to the element size";
        case SSD_ERR_TOO_LARGE:
            return "SSD_ERR_TOO_LARGE: the sizes need more scratch than ssd_verify_static's fixed array";
        default: return "unknown status";
    }
}

int32_t ssd_last_cuda_error(void) { return t_last_cuda_error; }

int32_t ssd_version(void) { return 200; }

uint64_t ssd_launch_count(void) { return t_launches; }

size_t ssd_ctc_draft_workspace_bytes(int32_t B, int64_t N, int32_t V, ssd_dtype dtype,
                                     const ssd_launch_opts *opts) {
    if (B < 0 || N < 0 || V < 1 || (dtype != SSD_F32 && dtype != SSD_BF16)) return 0;
    CtcPlan plan;
    if (plan_ctc(dtype, V, V, N, B, opts, &plan) != SSD_OK) return 0;
    return plan.workspace_bytes;
}

size_t ssd_verify_workspace_bytes(int32_t B, int64_t M, int32_t V, ssd_dtype dtype,
                                  const ssd_launch_opts *opts) {
    if (B < 0 || M < 0 || V < 1 || (dtype != SSD_F32 && dtype != SSD_BF16)) return 0;
    VerifyPlan plan;
    if (plan_for_query(B, M, V, dtype, opts, &plan) != SSD_OK) return 0;
    return plan.workspace_bytes;
}

int32_t ssd_ctc_draft(const void *logits, ssd_dtype dtype, int32_t V, int64_t ld,
                      const int64_t *frame_off, int32_t B, int64_t N,
                      int32_t blank_id, int32_t max_draft_len,
                      float *frame_entropy, int32_t *frame_argmax, float *frame_lse,
                      float *frame_logprob,
                      int32_t *draft_tokens, int32_t *draft_frames,
                      int32_t *draft_len, int32_t *draft_full_len,
                      float *utt_max_entropy, uint32_t *utt_status,
                      void *workspace, size_t workspace_bytes, void *stream,
                      const ssd_launch_opts *opts) {
    if (dtype != SSD_F32 && dtype != SSD_BF16) return SSD_ERR_DTYPE;
    if (B < 0 || N < 0 || V < 1 || ld < V || blank_id < 0 || blank_id >= V || max_draft_len < 0)
        return SSD_ERR_ARG;
    if (!frame_off) return SSD_ERR_NULL;
    if (N > 0 && (!logits || !frame_entropy || !frame_argmax || !draft_tokens)) return SSD_ERR_NULL;
    if (B > 0 && (!draft_len || !draft_full_len || !utt_max_entropy || !utt_status))
        return SSD_ERR_NULL;
    const int es = dtype == SSD_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(logits) % es) return SSD_ERR_ALIGN;
    CtcPlan plan;
    int rc = plan_ctc(dtype, V, ld, N, B, opts, &plan);
    if (rc != SSD_OK) return rc;
    if (workspace && (workspace_bytes < plan.workspace_bytes ||
                      reinterpret_cast<uintptr_t>(workspace) % 256))
        return SSD_ERR_WORKSPACE;
    Launch L{static_cast<cudaStream_t>(stream), opts};
    rc = launch_ctc_rows(logits, dtype, V, ld, N, frame_entropy, frame_argmax, frame_lse,
                         frame_logprob, workspace, plan, L);
    if (rc != SSD_OK) return rc;
    return launch_collapse(frame_argmax, frame_entropy, frame_off, B, N, blank_id, max_draft_len,
                           draft_tokens, draft_frames, draft_len, draft_full_len,
                           utt_max_entropy, utt_status, workspace, L.stream);
}

int32_t ssd_entropy_gate(const float *frame_entropy, const int64_t *frame_off,
                         int32_t B, int64_t N, float tau_ctc,
                         uint8_t *gate_accept, float *max_entropy, int32_t *argmax_frame,
                         const float *utt_max_entropy, const uint32_t *utt_status,
                         void *stream) {
    if (B < 0 || N < 0) return SSD_ERR_ARG;
    if (B > 0 && (!gate_accept || !max_entropy)) return SSD_ERR_NULL;
    if (utt_max_entropy && !argmax_frame) {
        // the maxima are already there: B values to look at instead of N
        if (B > 0 && !utt_status) return SSD_ERR_NULL;
        return launch_gate_from_maxima(utt_max_entropy, utt_status, B, tau_ctc, gate_accept,
                                       max_entropy, static_cast<cudaStream_t>(stream));
    }
    if (!frame_off) return SSD_ERR_NULL;
    if (N > 0 && !frame_entropy) return SSD_ERR_NULL;
    return launch_gate(frame_entropy, frame_off, B, N, tau_ctc, gate_accept, max_entropy,
                       argmax_frame, static_cast<cudaStream_t>(stream));
}

int32_t ssd_verify(const void *logits, ssd_dtype dtype, int32_t V, int64_t ld,
                   const int64_t *tok_off, const int32_t *draft_ids, int32_t B, int64_t M,
                   float tau_slm, const uint8_t *skip,
                   float *token_logp, float *row_lse,
                   int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                   void *workspace, size_t workspace_bytes, void *stream,
                   const ssd_launch_opts *opts) {
    if (dtype != SSD_F32 && dtype != SSD_BF16) return SSD_ERR_DTYPE;
    if (B < 0 || M < 0 || V < 1 || ld < V) return SSD_ERR_ARG;
    if (!tok_off) return SSD_ERR_NULL;
    if (M > 0 && (!logits || !draft_ids || !token_logp)) return SSD_ERR_NULL;
    if (B > 0 && (!accepted_len || !all_accepted || !utt_status)) return SSD_ERR_NULL;
    const int es = dtype == SSD_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(logits) % es) return SSD_ERR_ALIGN;
    VerifyPlan plan;
    int rc = plan_for_query(B, M, V, dtype, opts, &plan);
    if (rc != SSD_OK) return rc;
    if (B > 0 && (!workspace || workspace_bytes < plan.workspace_bytes ||
                  reinterpret_cast<uintptr_t>(workspace) % 256))
        return SSD_ERR_WORKSPACE;
    Launch L{static_cast<cudaStream_t>(stream), opts};
    return launch_verify(logits, dtype, V, ld, M, tok_off, draft_ids, B, tau_slm, skip, workspace,
                         token_logp, row_lse, accepted_len, all_accepted, utt_status, plan, L);
}

int32_t ssd_verify_shard(const void *logits, ssd_dtype dtype, int32_t V_local, int64_t ld,
                         int64_t col0, const int64_t *tok_off, const int32_t *draft_ids,
                         int32_t B, int64_t M, const uint8_t *skip, float *shard_stats,
                         void *workspace, size_t workspace_bytes, void *stream,
                         const ssd_launch_opts *opts) {
    if (dtype != SSD_F32 && dtype != SSD_BF16) return SSD_ERR_DTYPE;
    if (B < 0 || M < 0 || V_local < 1 || ld < V_local || col0 < 0) return SSD_ERR_ARG;
    if (!tok_off) return SSD_ERR_NULL;
    if (M > 0 && (!logits || !draft_ids || !shard_stats)) return SSD_ERR_NULL;
    const int es = dtype == SSD_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(logits) % es) return SSD_ERR_ALIGN;
    VerifyPlan plan;
    int rc = plan_for_query(B, M, V_local, dtype, opts, &plan);
    if (rc != SSD_OK) return rc;
    if (B > 0 && (!workspace || workspace_bytes < plan.workspace_bytes ||
                  reinterpret_cast<uintptr_t>(workspace) % 256))
        return SSD_ERR_WORKSPACE;
    Launch L{static_cast<cudaStream_t>(stream), opts};
    return launch_verify_shard(logits, dtype, V_local, ld, M, col0, tok_off, draft_ids, B, skip,
                               workspace, shard_stats, plan, L);
}

int32_t ssd_verify_combine(const float *stats_all, int32_t R, int64_t V_total,
                           const int64_t *tok_off, const int32_t *draft_ids, int32_t B, int64_t M,
                           float tau_slm, const uint8_t *skip,
                           float *token_logp, float *row_lse,
                           int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                           void *stream) {
    if (B < 0 || M < 0 || R < 1 || V_total < 1) return SSD_ERR_ARG;
    if (!tok_off || (B > 0 && (!accepted_len || !all_accepted || !utt_status))) return SSD_ERR_NULL;
    if (M > 0 && (!stats_all || !draft_ids || !token_logp)) return SSD_ERR_NULL;
    return launch_verify_combine(stats_all, R, V_total, tok_off, draft_ids, B, M, tau_slm, skip,
                                 token_logp, row_lse, accepted_len, all_accepted, utt_status,
                                 static_cast<cudaStream_t>(stream));
}

int32_t ssd_threshold_sweep(const float *utt_max_entropy, const float *token_logp,
                            const int64_t *tok_off, int32_t B, int64_t M,
                            const float *tau_ctc, const float *tau_slm, int32_t P,
                            uint8_t *gate_accept, int32_t *accepted_len, uint8_t *all_accepted,
                            int32_t *counts, void *stream) {
    if (B < 0 || M < 0 || P < 0) return SSD_ERR_ARG;
    if (!tok_off) return SSD_ERR_NULL;
    if (P > 0 && (!tau_ctc || !tau_slm)) return SSD_ERR_NULL;
    if (P > 0 && B > 0 && (!utt_max_entropy || !gate_accept || !accepted_len || !all_accepted))
        return SSD_ERR_NULL;
    if (M > 0 && !token_logp) return SSD_ERR_NULL;
    return launch_sweep(utt_max_entropy, token_logp, tok_off, B, M, tau_ctc, tau_slm, P,
                        gate_accept, accepted_len, all_accepted, counts,
                        static_cast<cudaStream_t>(stream));
}

int32_t ssd_assemble(const int32_t *tokens, const int64_t *tok_off, int32_t B, int64_t M,
                     const uint8_t *gate_accept, const int32_t *accepted_len,
                     const uint8_t *all_accepted,
                     int32_t *final_tokens, int32_t *final_len, uint8_t *is_final,
                     int32_t *ar_count, int32_t *ar_utt, int32_t *ar_resume, void *stream) {
    if (B < 0 || M < 0) return SSD_ERR_ARG;
    if (!tok_off || !ar_count) return SSD_ERR_NULL;
    if (M > 0 && (!tokens || !final_tokens)) return SSD_ERR_NULL;
    if (B > 0 && (!gate_accept || !accepted_len || !all_accepted || !final_len || !is_final ||
                  !ar_utt || !ar_resume))
        return SSD_ERR_NULL;
    return launch_assemble(tokens, tok_off, B, M, gate_accept, accepted_len, all_accepted,
                           final_tokens, final_len, is_final, ar_count, ar_utt, ar_resume,
                           static_cast<cudaStream_t>(stream));
}

size_t ssd_verify_early_exit_workspace_bytes(int32_t B, int64_t M, int32_t V, ssd_dtype dtype,
                                             const ssd_launch_opts *opts) {
    if (B < 0 || M < 0 || V < 1 || (dtype != SSD_F32 && dtype != SSD_BF16)) return 0;
    VerifyPlan plan;
    if (plan_for_query(B, M, V, dtype, opts, &plan) != SSD_OK) return 0;
    return verify_ee_workspace_bytes(B, plan);
}

int32_t ssd_verify_early_exit(const void *logits, ssd_dtype dtype, int32_t V, int64_t ld,
                              const int64_t *tok_off, const int32_t *draft_ids, int32_t B,
                              int64_t M, float tau_slm, const uint8_t *skip,
                              float *token_logp, float *row_lse,
                              int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                              int32_t *rows_read,
                              void *workspace, size_t workspace_bytes, void *stream,
                              const ssd_launch_opts *opts) {
    if (dtype != SSD_F32 && dtype != SSD_BF16) return SSD_ERR_DTYPE;
    if (B < 0 || M < 0 || V < 1 || ld < V) return SSD_ERR_ARG;
    if (!tok_off) return SSD_ERR_NULL;
    if (M > 0 && (!logits || !draft_ids || !token_logp)) return SSD_ERR_NULL;
    if (B > 0 && (!accepted_len || !all_accepted || !utt_status)) return SSD_ERR_NULL;
    const int es = dtype == SSD_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(logits) % es) return SSD_ERR_ALIGN;
    VerifyPlan plan;
    int rc = plan_for_query(B, M, V, dtype, opts, &plan);
    if (rc != SSD_OK) return rc;
    if (B > 0 && (!workspace || workspace_bytes < verify_ee_workspace_bytes(B, plan) ||
                  reinterpret_cast<uintptr_t>(workspace) % 256))
        return SSD_ERR_WORKSPACE;
    Launch L{static_cast<cudaStream_t>(stream), opts};
    if (!verify_ee_applicable(B, M, plan)) {
        // too few rows to deal out position by position: the full kernel, whose outputs
        // are a superset; every row of a verified utterance is then read
        rc = launch_verify(logits, dtype, V, ld, M, tok_off, draft_ids, B, tau_slm, skip, workspace,
                           token_logp, row_lse, accepted_len, all_accepted, utt_status, plan, L);
        if (rc == SSD_OK && rows_read && B > 0) {
            cudaError_t e = cudaMemsetAsync(rows_read, 0xff, (size_t)B * sizeof(int32_t), L.stream);
            if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
        }
        return rc;
    }
    return launch_verify_ee(logits, dtype, V, ld, M, tok_off, draft_ids, B, tau_slm, skip, workspace,
                            token_logp, row_lse, accepted_len, all_accepted, utt_status, rows_read,
                            plan, L);
}

size_t ssd_greedy_step_workspace_bytes(int64_t R, int32_t V, ssd_dtype dtype,
                                       const ssd_launch_opts *opts) {
    if (R < 0 || V < 1 || (dtype != SSD_F32 && dtype != SSD_BF16)) return 0;
    VerifyPlan plan;
    if (plan_for_query(0, R, V, dtype, opts, &plan) != SSD_OK) return 0;
    return greedy_workspace_bytes(R, plan);
}

int32_t ssd_greedy_step(const void *logits, ssd_dtype dtype, int32_t V, int64_t ld, int64_t R,
                        int32_t *next_token, float *next_logp, float *row_lse,
                        uint32_t *row_status, void *workspace, size_t workspace_bytes,
                        void *stream, const ssd_launch_opts *opts) {
    if (dtype != SSD_F32 && dtype != SSD_BF16) return SSD_ERR_DTYPE;
    if (R < 0 || V < 1 || ld < V) return SSD_ERR_ARG;
    if (R > 0 && (!logits || !next_token)) return SSD_ERR_NULL;
    const int es = dtype == SSD_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(logits) % es) return SSD_ERR_ALIGN;
    VerifyPlan plan;
    int rc = plan_for_query(0, R, V, dtype, opts, &plan);
    if (rc != SSD_OK) return rc;
    if (plan.kernel != 2) return SSD_ERR_ARG;
    if (R > 0 && (!workspace || workspace_bytes < greedy_workspace_bytes(R, plan) ||
                  reinterpret_cast<uintptr_t>(workspace) % 256))
        return SSD_ERR_WORKSPACE;
    Launch L{static_cast<cudaStream_t>(stream), opts};
    return launch_greedy(logits, dtype, V, ld, R, workspace, next_token, next_logp, row_lse,
                         row_status, plan, L);
}

}  // extern "C"
