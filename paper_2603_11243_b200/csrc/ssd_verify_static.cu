// ssd_verify_static: ssd_verify for callers that have no device allocator at hand.
//
// The streaming verify kernel leaves partial (reference, sum) pairs per logits row in scratch
// memory that ssd_verify takes from the caller.  Here that scratch is a fixed array in the
// library's own device image, so the call needs no workspace argument and performs no
// allocation of any kind.
#include <mutex>

#include "ssd_common.cuh"

namespace ssd {
namespace {

constexpr size_t kStaticScratchBytes = SSD_VERIFY_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// Lives in every device that loads the library, from load to exit.  All calls on a device
// share it.  Nothing in it has to start at zero: every partial pair a call reads was written
// by the same call, and the error word is compared with a per-call epoch.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void *g_scratch_ptr[kMaxDevices];      // device address of g_static_scratch, per device

// The array's name is only a host-side handle; the address kernels can use has to be asked
// for, once per device and with that device current.
int static_scratch(void **ptr) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return SSD_ERR_ARG;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) {
            record_cuda_error(e);
            return SSD_ERR_CUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    *ptr = g_scratch_ptr[dev];
    return SSD_OK;
}

}  // namespace
}  // namespace ssd

extern "C" int32_t ssd_verify_static(const void *logits, ssd_dtype dtype, int32_t V, int64_t ld,
                                     const int64_t *tok_off, const int32_t *draft_ids, int32_t B,
                                     int64_t M, float tau_slm, const uint8_t *skip,
                                     float *token_logp, float *row_lse, int32_t *accepted_len,
                                     uint8_t *all_accepted, uint32_t *utt_status, void *stream,
                                     const ssd_launch_opts *opts) {
    using namespace ssd;
    if (dtype != SSD_F32 && dtype != SSD_BF16) return SSD_ERR_DTYPE;
    if (B < 0 || M < 0 || V < 1 || ld < V) return SSD_ERR_ARG;
    VerifyPlan plan;
    int rc = device_sm_count() > 0 ? plan_verify(B, M, V, dtype, opts, &plan) : SSD_ERR_CUDA;
    if (rc == SSD_ERR_CUDA) {              // no device to ask: the size check still works
        PlanReplay replay;
        rc = plan_verify(B, M, V, dtype, opts, &plan);
    }
    if (rc != SSD_OK) return rc;
    if (plan.workspace_bytes > kStaticScratchBytes) return SSD_ERR_TOO_LARGE;
    void *scratch = nullptr;
    rc = static_scratch(&scratch);
    if (rc != SSD_OK) return rc;
    return ssd_verify(logits, dtype, V, ld, tok_off, draft_ids, B, M, tau_slm, skip, token_logp,
                      row_lse, accepted_len, all_accepted, utt_status, scratch,
                      kStaticScratchBytes, stream, opts);
}
