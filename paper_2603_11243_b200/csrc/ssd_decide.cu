// Decision kernels around the two verification stages: the operating-point sweep of
// Section 3.2 (Eq. 3 and the first-reject rule of Section 2.3 re-evaluated for many threshold
// pairs from stored per-utterance maxima and per-token log-likelihoods, without touching the
// logits again) and the assembly of the final hypothesis (Eq. 7) with the list of utterances
// the auto-regressive pass has to continue.  Integer and compare work only.
#include <limits.h>
#include <math.h>

#include "ssd_common.cuh"

namespace ssd {
namespace {

constexpr int kSweepPairsPerLaunch = 128;

struct SweepPairs {
    float tau_ctc[kSweepPairsPerLaunch];
    float log_tau_slm[kSweepPairsPerLaunch];
    uint8_t reject_none[kSweepPairsPerLaunch];
    int count;
    int first;           // index of pair 0 of this launch in the caller's list
};

// One warp per (pair, utterance): 32 log-likelihoods per step, stops at the first reject.
__global__ void __launch_bounds__(256) sweep_kernel(
    const float *__restrict__ utt_max_entropy, const float *__restrict__ token_logp,
    const int64_t *__restrict__ tok_off, int B, int64_t M, const SweepPairs pairs,
    uint8_t *__restrict__ gate_accept, int32_t *__restrict__ accepted_len,
    uint8_t *__restrict__ all_accepted, int32_t *__restrict__ counts) {
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t items = (int64_t)pairs.count * B;
    for (int64_t it = warp; it < items; it += nwarps) {
        const int pi = (int)(it / B), b = (int)(it - (int64_t)pi * B);
        const float lt = pairs.log_tau_slm[pi];
        const bool none = pairs.reject_none[pi] != 0;
        const int64_t i0 = tok_off[b], i1 = tok_off[b + 1];
        const bool ok = !(i0 < 0 || i1 < i0 || i1 > M);
        const int K = ok ? (int)min(i1 - i0, (int64_t)INT_MAX) : 0;
        int first = K;
        if (!none) {
            for (int base = 0; base < K; base += 32) {
                const int i = base + lane;
                bool rej = false;
                if (i < K) rej = !(token_logp[i0 + i] > lt);     // p <= tau; NaN rejects
                const unsigned bal = __ballot_sync(0xffffffffu, rej);
                if (bal) { first = base + __ffs(bal) - 1; break; }
            }
        }
        if (lane == 0) {
            const bool g = utt_max_entropy[b] < pairs.tau_ctc[pi];   // Eq. 3, strict; NaN fails
            const bool all = ok && first == K;
            const int64_t o = (int64_t)(pairs.first + pi) * B + b;
            gate_accept[o] = g ? 1 : 0;
            accepted_len[o] = first;
            all_accepted[o] = all ? 1 : 0;
            if (counts) atomicAdd(&counts[3 * (pairs.first + pi) + (g ? 0 : all ? 1 : 2)], 1);
        }
    }
}

// Eq. 7.  CTA b < B copies the final tokens of utterance b; CTA B builds the ordered list of
// utterances left to the auto-regressive pass (a block scan over the utterances).
constexpr int kAssembleThreads = 256;
__global__ void __launch_bounds__(kAssembleThreads) assemble_kernel(
    const int32_t *__restrict__ tokens, const int64_t *__restrict__ tok_off, int B, int64_t M,
    const uint8_t *__restrict__ gate_accept, const int32_t *__restrict__ accepted_len,
    const uint8_t *__restrict__ all_accepted, int32_t *__restrict__ final_tokens,
    int32_t *__restrict__ final_len, uint8_t *__restrict__ is_final,
    int32_t *__restrict__ ar_count, int32_t *__restrict__ ar_utt, int32_t *__restrict__ ar_resume) {
    __shared__ int warp_tot[2][kAssembleThreads / 32];
    pdl_enter();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    auto prefix_len = [&](int b, bool &fin) {
        const int64_t i0 = tok_off[b], i1 = tok_off[b + 1];
        const int K = (i0 < 0 || i1 < i0 || i1 > M) ? 0 : (int)min(i1 - i0, (int64_t)INT_MAX);
        fin = gate_accept[b] != 0 || all_accepted[b] != 0;
        return fin ? K : max(0, min(accepted_len[b], K));
    };
    if ((int)blockIdx.x < B) {
        const int b = blockIdx.x;
        bool fin;
        const int len = prefix_len(b, fin);
        const int64_t i0 = tok_off[b];
        for (int i = tid; i < len; i += blockDim.x) final_tokens[i0 + i] = tokens[i0 + i];
        if (tid == 0) { final_len[b] = len; is_final[b] = fin ? 1 : 0; }
        return;
    }
    int base = 0, buf = 0;
    for (int tile = 0; tile < B; tile += blockDim.x, buf ^= 1) {
        const int b = tile + tid;
        bool fin = true;
        int len = 0;
        if (b < B) len = prefix_len(b, fin);
        const bool need = b < B && !fin;
        const unsigned bal = __ballot_sync(0xffffffffu, need);
        if (lane == 0) warp_tot[buf][warp] = __popc(bal);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < kAssembleThreads / 32; ++w) {
            const int c = warp_tot[buf][w];
            if (w < warp) before += c;
            total += c;
        }
        if (need) {
            const int pos = base + before + __popc(bal & ((1u << lane) - 1));
            ar_utt[pos] = b;
            ar_resume[pos] = len;
        }
        base += total;
    }
    if (tid == 0) *ar_count = base;
}

}  // namespace

int launch_sweep(const float *utt_max_entropy, const float *token_logp, const int64_t *tok_off,
                 int B, int64_t M, const float *tau_ctc, const float *tau_slm, int P,
                 uint8_t *gate_accept, int32_t *accepted_len, uint8_t *all_accepted,
                 int32_t *counts, cudaStream_t stream) {
    if (P == 0 || B == 0) return SSD_OK;
    cudaError_t e;
    if (counts) {
        e = cudaMemsetAsync(counts, 0, (size_t)P * 3 * sizeof(int32_t), stream);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    }
    for (int first = 0; first < P; first += kSweepPairsPerLaunch) {
        SweepPairs sp{};
        sp.count = P - first < kSweepPairsPerLaunch ? P - first : kSweepPairsPerLaunch;
        sp.first = first;
        for (int i = 0; i < sp.count; ++i) {
            const double tau = (double)tau_slm[first + i];
            sp.tau_ctc[i] = tau_ctc[first + i];
            sp.reject_none[i] = !(tau > 0.0);
            // tau >= 1 rejects everything (p <= 1), whatever rounding made of a stored log p
            sp.log_tau_slm[i] = sp.reject_none[i] ? -INFINITY : tau >= 1.0 ? INFINITY : (float)log(tau);
        }
        const int64_t warps = (int64_t)sp.count * B;
        int64_t ctas = (warps + 7) / 8;
        const int sms = device_sm_count();
        if (sms <= 0) return SSD_ERR_CUDA;
        if (ctas > (int64_t)sms * 8) ctas = (int64_t)sms * 8;
        e = launch_pdl(sweep_kernel, (unsigned)ctas, 256u, 0, stream, utt_max_entropy, token_logp,
                       tok_off, B, M, sp, gate_accept, accepted_len, all_accepted, counts);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

int launch_assemble(const int32_t *tokens, const int64_t *tok_off, int B, int64_t M,
                    const uint8_t *gate_accept, const int32_t *accepted_len,
                    const uint8_t *all_accepted, int32_t *final_tokens, int32_t *final_len,
                    uint8_t *is_final, int32_t *ar_count, int32_t *ar_utt, int32_t *ar_resume,
                    cudaStream_t stream) {
    cudaError_t e = launch_pdl(assemble_kernel, (unsigned)(B + 1), (unsigned)kAssembleThreads, 0,
                               stream, tokens, tok_off, B, M, gate_accept, accepted_len,
                               all_accepted, final_tokens, final_len, is_final, ar_count, ar_utt,
                               ar_resume);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

}  // namespace ssd
