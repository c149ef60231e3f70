// Stage 1 kernels: per-frame softmax statistics of the CTC head (Eq. 2, Eq. 3), the collapse
// B of Section 2.1, and the entropy gate of Eq. 3.
//
// Frame statistics are one streaming read of the [N, V] logits.  Two kernels compute them:
//   ctc_rows_tma    each warp owns a small ring of shared-memory stages that it fills with 1-D
//                   bulk asynchronous copies (TMA) of a few consecutive rows and drains itself:
//                   no block-level synchronisation at all.  A row sits in shared memory while it
//                   is reduced, so the exact two-pass softmax (max, then exponentials) costs one
//                   HBM read and one exponential per logit.
//   ctc_rows_plain  one warp per row with scalar global loads; any alignment, any V.  Fallback.
#include <limits.h>
#include <math.h>

#include "ssd_common.cuh"

namespace ssd {

namespace {

constexpr uint32_t kNanInternal = 0x7fc0dead;  // entropy payload written when a wait ran out

struct CtcParams {
    const char *logits;
    int V;
    int64_t ld;
    int64_t N;
    int64_t total_bytes;   // bytes from the first to one past the last logit of the matrix
    int64_t num_tiles;
    int rows_per_tile;
    int stages;
    int stage_stride;      // bytes, multiple of 128
    int warps;
    float *frame_entropy;
    int32_t *frame_argmax;
    float *frame_lse;
    float *frame_logprob;
};

// Statistics of one row held by one warp.
struct RowStats {
    float lse, entropy;
    int arg;
};

template <typename T>
__device__ __forceinline__ void accumulate(float x, float mh, float &S, float &A) {
    float t2 = fmaf(x, kLog2e, -mh);
    float e = ex2(t2);
    S += e;
    A = fmaf(fmaxf(t2, -200.f), e, A);   // the clamp turns (-inf)*0 into 0
}

// Reduces one row that lies in shared memory at byte address `row_addr` (element aligned).
// Exact two-pass softmax: pass 1 finds the maximum and where it first occurs, pass 2 sums
// e = 2^((x-m)*log2e) and (x-m)*log2e*e.  With mh = fl(m*log2e) and ml = m*log2e - mh (exact,
// by fma) every exponent carries the same +ml, which cancels in the entropy and is removed
// from the log-sum-exp at the end.
template <typename T>
__device__ __forceinline__ RowStats reduce_row_smem(uint32_t stage_addr, uint32_t row_off,
                                                    int V, int lane) {
    constexpr int ES = Elem<T>::kBytes, EPC = Elem<T>::kPerChunk;
    const int e0 = row_off / ES;                 // element offset of the row inside the stage
    int c0 = (e0 + EPC - 1) / EPC;               // first full 16-byte chunk
    int c1 = (e0 + V) / EPC;                     // one past the last full chunk
    int nhead, ntail;
    if (c1 > c0) { nhead = c0 * EPC - e0; ntail = e0 + V - c1 * EPC; }
    else { c0 = c1 = 0; nhead = V; ntail = 0; }
    const int tail0 = c1 * EPC - e0;             // row-relative index of the first tail element

    // ---- pass 1: maximum and its first position among this lane's elements ----
    float vmax = -INFINITY;
    int vidx = INT_MAX;
    bool vchunk = false;
    for (int i = lane; i < nhead; i += 32) {
        float x = Elem<T>::load_shared(stage_addr + (e0 + i) * ES);
        if (x > vmax) { vmax = x; vidx = i; }
    }
#pragma unroll 4
    for (int c = c0 + lane; c < c1; c += 32) {
        uint4 w = lds128(stage_addr + c * 16);
        float cm = chunk_max<T>(w);
        if (cm > vmax) { vmax = cm; vidx = c * EPC - e0; vchunk = true; }
    }
    for (int i = lane; i < ntail; i += 32) {
        float x = Elem<T>::load_shared(stage_addr + (e0 + tail0 + i) * ES);
        if (x > vmax) { vmax = x; vidx = tail0 + i; vchunk = false; }
    }
    const float m = warp_max(vmax);
    int cand = INT_MAX;
    if (vmax == m && vidx != INT_MAX) {
        cand = vidx;
        if (vchunk) {
            uint4 w = lds128(stage_addr + (e0 + vidx) * ES);
            float x[EPC];
            chunk_unpack<T>(w, x);
            int j = EPC - 1;
#pragma unroll
            for (int k = EPC - 2; k >= 0; --k) if (x[k] == m) j = k;
            cand = vidx + j;
        }
    }
    int arg = __reduce_min_sync(0xffffffffu, cand);
    if (arg == INT_MAX) arg = 0;

    // ---- pass 2: sums ----
    const float mh = m * kLog2e;
    const float ml = fmaf(m, kLog2e, -mh);
    float S0 = 0.f, S1 = 0.f, A0 = 0.f, A1 = 0.f;
    for (int i = lane; i < nhead; i += 32)
        accumulate<T>(Elem<T>::load_shared(stage_addr + (e0 + i) * ES), mh, S0, A0);
    for (int i = lane; i < ntail; i += 32)
        accumulate<T>(Elem<T>::load_shared(stage_addr + (e0 + tail0 + i) * ES), mh, S1, A1);
#pragma unroll 4
    for (int c = c0 + lane; c < c1; c += 32) {
        uint4 w = lds128(stage_addr + c * 16);
        float x[EPC];
        chunk_unpack<T>(w, x);
#pragma unroll
        for (int k = 0; k < EPC; k += 2) {
            accumulate<T>(x[k], mh, S0, A0);
            accumulate<T>(x[k + 1], mh, S1, A1);
        }
    }
    const float S = warp_sum(S0 + S1);
    const float A2 = warp_sum(A0 + A1);
    RowStats r;
    const float lnS = logf(S);
    r.lse = m + (lnS - ml * kLn2);
    r.entropy = fmaxf(lnS - kLn2 * (A2 / S), 0.f);
    if (!(S > 0.5f) || !(S < INFINITY) || !(fabsf(m) < INFINITY))
        r.entropy = __int_as_float(0x7fc00000);   // NaN / +inf / all -inf: flagged downstream
    r.arg = arg;
    return r;
}

template <typename T>
__global__ void __launch_bounds__(512, 1) ctc_rows_tma(const CtcParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int ES = Elem<T>::kBytes;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int W = p.warps, S = p.stages, R = p.rows_per_tile;
    const int64_t gw = (int64_t)blockIdx.x * W + warp, GW = (int64_t)gridDim.x * W;
    const int64_t my_tiles = gw < p.num_tiles ? (p.num_tiles - gw + GW - 1) / GW : 0;
    if (my_tiles == 0) return;

    const uint32_t bar0 = smem_u32(smem) + (warp * S) * 8;
    const uint32_t stage_region = (uint32_t)((W * S * 8 + 127) & ~127);
    const uint32_t stage0 = smem_u32(smem) + stage_region + (uint32_t)(warp * S) * p.stage_stride;
    unsigned char *stage0_ptr = smem + stage_region + (size_t)(warp * S) * p.stage_stride;

    if (lane == 0) {
        for (int s = 0; s < S; ++s) mbar_init(bar0 + s * 8, 1);
        mbar_init_fence();
    }
    __syncwarp();

    const uintptr_t base = reinterpret_cast<uintptr_t>(p.logits);
    const uintptr_t lo_bound = base, hi_bound = base + (uintptr_t)p.total_bytes;
    const int64_t row_pitch = p.ld * ES;

    // Brings tile k of this warp into stage s.  The tile's rows are one contiguous byte range
    // (padding between rows included); the 16-byte-aligned superset of the range is fetched with
    // one bulk copy where that superset stays inside the matrix, so that interior tiles need no
    // scalar fix-up; bytes of neighbouring rows that come along are never looked at.
    auto issue = [&](int64_t k, int s) {
        const int64_t tile = gw + k * GW;
        const int64_t r0 = tile * R;
        const int nrows = (int)min((int64_t)R, p.N - r0);
        const uintptr_t gstart = base + (uintptr_t)(r0 * row_pitch);
        const uintptr_t gend = gstart + (uintptr_t)((nrows - 1) * row_pitch + (int64_t)p.V * ES);
        const uintptr_t f0 = gstart & ~(uintptr_t)15;
        const uintptr_t c1 = (gend + 15) & ~(uintptr_t)15;
        const uintptr_t bulk_lo = f0 >= lo_bound ? f0 : f0 + 16;
        const uintptr_t bulk_hi = c1 <= hi_bound ? c1 : c1 - 16;
        const bool has_bulk = bulk_hi > bulk_lo;
        unsigned char *dst = stage0_ptr + (size_t)s * p.stage_stride;
        if (!has_bulk || bulk_lo > gstart || bulk_hi < gend) {
            // first / last tile of the matrix only: elements outside the bulk range by plain loads
            const uintptr_t h_end = has_bulk ? min(bulk_lo, gend) : gend;
            for (uintptr_t a = gstart + (uintptr_t)lane * ES; a < h_end; a += 32 * ES) {
                if (ES == 4) *reinterpret_cast<uint32_t *>(dst + (a - f0)) =
                        *reinterpret_cast<const uint32_t *>(a);
                else *reinterpret_cast<uint16_t *>(dst + (a - f0)) =
                        *reinterpret_cast<const uint16_t *>(a);
            }
            if (has_bulk) {
                for (uintptr_t a = max(bulk_hi, gstart) + (uintptr_t)lane * ES; a < gend;
                     a += 32 * ES) {
                    if (ES == 4) *reinterpret_cast<uint32_t *>(dst + (a - f0)) =
                            *reinterpret_cast<const uint32_t *>(a);
                    else *reinterpret_cast<uint16_t *>(dst + (a - f0)) =
                            *reinterpret_cast<const uint16_t *>(a);
                }
            }
            __syncwarp();
        }
        if (lane == 0) {
            const uint32_t bar = bar0 + s * 8;
            if (has_bulk) {
                const uint32_t bytes = (uint32_t)(bulk_hi - bulk_lo);
                fence_proxy_async();
                mbar_arrive_expect_tx(bar, bytes);
                bulk_g2s(stage0 + (uint32_t)s * p.stage_stride + (uint32_t)(bulk_lo - f0),
                         reinterpret_cast<const void *>(bulk_lo), bytes, bar);
            } else {
                mbar_arrive(bar);
            }
        }
    };

    const int prologue = (int)min((int64_t)S, my_tiles);
    for (int k = 0; k < prologue; ++k) issue(k, k);

    bool failed = false;
    for (int64_t k = 0; k < my_tiles; ++k) {
        const int s = (int)(k % S);
        const uint32_t parity = (uint32_t)((k / S) & 1);
        if (!mbar_wait_bounded(bar0 + s * 8, parity)) { failed = true; break; }
        const int64_t tile = gw + k * GW;
        const int64_t r0 = tile * R;
        const int nrows = (int)min((int64_t)R, p.N - r0);
        const uintptr_t gstart = base + (uintptr_t)(r0 * row_pitch);
        const uint32_t head = (uint32_t)(gstart & 15);
        const uint32_t stage_addr = stage0 + (uint32_t)s * p.stage_stride;
        float myH = 0.f, myL = 0.f;
        int myA = 0;
        for (int i = 0; i < nrows; ++i) {
            const uint32_t row_off = head + (uint32_t)(i * row_pitch);
            RowStats rs = reduce_row_smem<T>(stage_addr, row_off, p.V, lane);
            if (lane == i) { myH = rs.entropy; myL = rs.lse; myA = rs.arg; }
            if (p.frame_logprob) {
                float *out = p.frame_logprob + (r0 + i) * p.ld;
                for (int a = lane; a < p.V; a += 32)
                    out[a] = Elem<T>::load_shared(stage_addr + row_off + a * ES) - rs.lse;
            }
        }
        if (lane < nrows) {
            p.frame_entropy[r0 + lane] = myH;
            p.frame_argmax[r0 + lane] = myA;
            if (p.frame_lse) p.frame_lse[r0 + lane] = myL;
        }
        __syncwarp();
        if (k + S < my_tiles) issue(k + S, s);
    }
    if (failed) {
        // A wait ran out: poison every frame this warp still owed so that the per-utterance
        // kernel reports SSD_UTT_INTERNAL, then let copies that may be in flight land.
        for (int64_t k = 0; k < my_tiles; ++k) {
            const int64_t r0 = (gw + k * GW) * R;
            const int nrows = (int)min((int64_t)R, p.N - r0);
            if (lane < nrows) {
                p.frame_entropy[r0 + lane] = __uint_as_float(kNanInternal);
                p.frame_argmax[r0 + lane] = 0;
                if (p.frame_lse) p.frame_lse[r0 + lane] = __uint_as_float(kNanInternal);
            }
        }
        drain_after_error();
    }
}

template <typename T>
__global__ void __launch_bounds__(256) ctc_rows_plain(const CtcParams p) {
    constexpr int ES = Elem<T>::kBytes;
    const int lane = threadIdx.x & 31;
    const int64_t gw = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t GW = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t row = gw; row < p.N; row += GW) {
        const char *rp = p.logits + row * p.ld * ES;
        float vmax = -INFINITY;
        int vidx = INT_MAX;
        for (int a = lane; a < p.V; a += 32) {
            float x = Elem<T>::load(rp + (size_t)a * ES);
            if (x > vmax) { vmax = x; vidx = a; }
        }
        const float m = warp_max(vmax);
        int arg = __reduce_min_sync(0xffffffffu, (vmax == m) ? vidx : INT_MAX);
        if (arg == INT_MAX) arg = 0;
        float S = 0.f, A = 0.f;
        for (int a = lane; a < p.V; a += 32) {
            float t = Elem<T>::load(rp + (size_t)a * ES) - m;
            float e = expf(t);
            S += e;
            A += (e > 0.f) ? t * e : 0.f;
        }
        S = warp_sum(S);
        A = warp_sum(A);
        const float lnS = logf(S);
        const float lse = m + lnS;
        float H = fmaxf(lnS - A / S, 0.f);
        if (!(S > 0.5f) || !(S < INFINITY) || !(fabsf(m) < INFINITY)) H = __int_as_float(0x7fc00000);
        if (lane == 0) {
            p.frame_entropy[row] = H;
            p.frame_argmax[row] = arg;
            if (p.frame_lse) p.frame_lse[row] = lse;
        }
        if (p.frame_logprob) {
            float *out = p.frame_logprob + row * p.ld;
            for (int a = lane; a < p.V; a += 32) out[a] = Elem<T>::load(rp + (size_t)a * ES) - lse;
        }
    }
}

// ---- collapse B and per-utterance maximum entropy: one CTA per utterance ----------------------
constexpr int kUttThreads = 256;

struct MaxAt {
    float v;
    int at;
};
__device__ __forceinline__ MaxAt better(MaxAt a, MaxAt b) {
    // larger value wins; on equal values the earlier frame; "at < 0" means empty
    if (b.at >= 0 && (a.at < 0 || b.v > a.v || (b.v == a.v && b.at < a.at))) return b;
    return a;
}
__device__ MaxAt block_max_at(MaxAt x, MaxAt *scratch /* [32] shared */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MaxAt y;
        y.v = __shfl_xor_sync(0xffffffffu, x.v, o);
        y.at = __shfl_xor_sync(0xffffffffu, x.at, o);
        x = better(x, y);
    }
    __syncthreads();
    if (lane == 0) scratch[warp] = x;
    __syncthreads();
    MaxAt r = scratch[0];
    for (int w = 1; w < nw; ++w) r = better(r, scratch[w]);
    return r;
}

__global__ void __launch_bounds__(kUttThreads) collapse_kernel(
    const int32_t *__restrict__ frame_argmax, const float *__restrict__ frame_entropy,
    const int64_t *__restrict__ frame_off, int B, int64_t N, int blank_id, int cap,
    int32_t *__restrict__ draft_tokens, int32_t *__restrict__ draft_frames,
    int32_t *__restrict__ draft_len, int32_t *__restrict__ draft_full_len,
    float *__restrict__ utt_max_entropy, uint32_t *__restrict__ utt_status) {
    __shared__ int warp_tot[32];
    __shared__ MaxAt scratch[32];
    __shared__ unsigned flags;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nw = blockDim.x >> 5;
    const int64_t t0 = frame_off[b], t1 = frame_off[b + 1];
    if (t0 < 0 || t1 < t0 || t1 > N) {
        if (tid == 0) {
            draft_len[b] = 0; draft_full_len[b] = 0; utt_max_entropy[b] = 0.f;
            utt_status[b] = SSD_UTT_BAD_OFFSETS;
        }
        return;
    }
    if (tid == 0) flags = 0;
    __syncthreads();
    const int64_t T = t1 - t0;
    int base = 0;
    MaxAt best{0.f, -1};
    unsigned myflags = 0;
    for (int64_t tile = 0; tile < T; tile += blockDim.x) {
        const int64_t t = tile + tid;
        const bool valid = t < T;
        int a = blank_id, prev = -1;
        if (valid) {
            a = frame_argmax[t0 + t];
            if (t > 0) prev = frame_argmax[t0 + t - 1];
            const float h = frame_entropy[t0 + t];
            if (h != h) {
                myflags |= (__float_as_uint(h) == kNanInternal) ? SSD_UTT_INTERNAL : SSD_UTT_NONFINITE;
            } else {
                best = better(best, MaxAt{h, (int)t});
            }
        }
        const bool keep = valid && a != blank_id && (t == 0 || a != prev);
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
        const int prefix = __popc(bal & ((1u << lane) - 1));
        __syncthreads();                       // previous tile's totals fully consumed
        if (lane == 0) warp_tot[warp] = __popc(bal);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < nw; ++w) {
            const int c = warp_tot[w];
            if (w < warp) before += c;
            total += c;
        }
        const int pos = base + before + prefix;
        if (keep && pos < cap) {
            draft_tokens[t0 + pos] = a;
            if (draft_frames) draft_frames[t0 + pos] = (int)t;
        }
        base += total;
    }
    best = block_max_at(best, scratch);
    if (myflags) atomicOr(&flags, myflags);
    __syncthreads();
    if (tid == 0) {
        draft_full_len[b] = base;
        draft_len[b] = min(base, cap);
        utt_max_entropy[b] = best.at >= 0 ? best.v : 0.f;
        utt_status[b] = flags;
    }
}

__global__ void __launch_bounds__(kUttThreads) gate_kernel(
    const float *__restrict__ frame_entropy, const int64_t *__restrict__ frame_off, int B,
    int64_t N, float tau, uint8_t *__restrict__ gate_accept, float *__restrict__ max_entropy,
    int32_t *__restrict__ argmax_frame) {
    __shared__ MaxAt scratch[32];
    __shared__ int not_below;
    const int b = blockIdx.x, tid = threadIdx.x;
    const int64_t t0 = frame_off[b], t1 = frame_off[b + 1];
    if (t0 < 0 || t1 < t0 || t1 > N) {
        if (tid == 0) {
            gate_accept[b] = 0; max_entropy[b] = 0.f;
            if (argmax_frame) argmax_frame[b] = -1;
        }
        return;
    }
    if (tid == 0) not_below = 0;
    __syncthreads();
    const int64_t T = t1 - t0;
    MaxAt best{0.f, -1};
    int bad = 0;
    for (int64_t t = tid; t < T; t += blockDim.x) {
        const float h = frame_entropy[t0 + t];
        if (!(h < tau)) bad = 1;             // Eq. 3 is strict; NaN never passes
        if (h == h) best = better(best, MaxAt{h, (int)t});
    }
    if (bad) atomicOr(&not_below, 1);
    best = block_max_at(best, scratch);       // contains __syncthreads
    if (tid == 0) {
        const bool accept = (T == 0) ? (0.f < tau) : (not_below == 0);
        gate_accept[b] = accept ? 1 : 0;
        max_entropy[b] = best.at >= 0 ? best.v : 0.f;
        if (argmax_frame) argmax_frame[b] = best.at;
    }
}

int g_sm_count = 0;
int sm_count() {
    if (g_sm_count == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
        g_sm_count = n;
    }
    return g_sm_count;
}

}  // namespace

int device_sm_count() { return sm_count(); }

unsigned long long next_epoch() {
    static unsigned long long counter = 0;
    unsigned long long c = __atomic_add_fetch(&counter, 1ull, __ATOMIC_RELAXED);
    return 0x55D0000000000000ull | (c & 0x0000ffffffffffffull);
}

int launch_ctc_rows(const void *logits, ssd_dtype dtype, int V, int64_t ld, int64_t N,
                    const int64_t *frame_off, int B, float *frame_entropy, int32_t *frame_argmax,
                    float *frame_lse, float *frame_logprob, uint32_t *utt_status,
                    const Launch &L) {
    (void)frame_off; (void)B; (void)utt_status;
    if (N == 0) return SSD_OK;
    const ssd_launch_opts *o = L.opts;
    const int es = dtype == SSD_F32 ? 4 : 2;
    CtcParams p{};
    p.logits = static_cast<const char *>(logits);
    p.V = V; p.ld = ld; p.N = N;
    p.total_bytes = (N - 1) * ld * es + (int64_t)V * es;
    p.frame_entropy = frame_entropy; p.frame_argmax = frame_argmax; p.frame_lse = frame_lse;
    p.frame_logprob = frame_logprob;

    // ---- choose the kernel and its shape ----
    int kernel = o ? o->kernel : 0;
    const int64_t row_pitch = ld * es;
    const int64_t row_bytes = (int64_t)V * es;
    const int smem_budget = 200 * 1024;
    int warps = 0, stages = (o && o->stages > 0) ? o->stages : 3, R = 0;
    if (stages < 2) stages = 2;
    if (stages > 8) stages = 8;
    if (kernel != 1) {
        const int cand[] = {16, 8, 4, 2, 1};
        for (int w : cand) {
            if (o && o->warps > 0 && o->warps != w) continue;
            const int64_t per_stage = ((smem_budget - 1024) / ((int64_t)w * stages)) & ~127ll;
            if (row_bytes + 48 > per_stage) continue;
            warps = w;
            int64_t r = 1 + (per_stage - 48 - row_bytes) / row_pitch;
            if (r > 32) r = 32;
            // a row pitch much wider than the row would drag the padding along: one row a tile
            if (row_pitch > 2 * row_bytes) r = 1;
            if (o && o->stage_bytes > 0 && o->stage_bytes < r) r = o->stage_bytes;
            R = (int)r;
            break;
        }
        if (warps == 0) {
            if (kernel == 2) return SSD_ERR_ARG;   // forced, but a row does not fit a stage
            kernel = 1;
        } else {
            kernel = 2;
        }
    }
    cudaError_t e;
    if (o && o->ev_begin) {
        e = cudaEventRecord(static_cast<cudaEvent_t>(o->ev_begin), L.stream);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    }
    if (kernel == 2) {
        p.rows_per_tile = R; p.stages = stages; p.warps = warps;
        p.stage_stride = (int)(((R - 1) * row_pitch + row_bytes + 32 + 127) & ~127ll);
        p.num_tiles = (N + R - 1) / R;
        const size_t smem = (size_t)((warps * stages * 8 + 127) & ~127) +
                            (size_t)warps * stages * p.stage_stride;
        int64_t ctas = (p.num_tiles + warps - 1) / warps;
        const int max_ctas = (o && o->ctas > 0) ? o->ctas : sm_count();
        if (ctas > max_ctas) ctas = max_ctas;
        auto kern = dtype == SSD_F32 ? ctc_rows_tma<float> : ctc_rows_tma<bf16_t>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
        kern<<<(unsigned)ctas, warps * 32, smem, L.stream>>>(p);
    } else {
        int64_t ctas = (N + 7) / 8;
        const int64_t cap = (o && o->ctas > 0) ? o->ctas : (int64_t)sm_count() * 8;
        if (ctas > cap) ctas = cap;
        if (dtype == SSD_F32) ctc_rows_plain<float><<<(unsigned)ctas, 256, 0, L.stream>>>(p);
        else ctc_rows_plain<bf16_t><<<(unsigned)ctas, 256, 0, L.stream>>>(p);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    if (o && o->ev_end) {
        e = cudaEventRecord(static_cast<cudaEvent_t>(o->ev_end), L.stream);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    }
    return SSD_OK;
}

int launch_collapse(const int32_t *frame_argmax, const float *frame_entropy,
                    const int64_t *frame_off, int B, int64_t N, int blank_id, int max_draft_len,
                    int32_t *draft_tokens, int32_t *draft_frames, int32_t *draft_len,
                    int32_t *draft_full_len, float *utt_max_entropy, uint32_t *utt_status,
                    cudaStream_t stream) {
    if (B == 0) return SSD_OK;
    collapse_kernel<<<B, kUttThreads, 0, stream>>>(
        frame_argmax, frame_entropy, frame_off, B, N, blank_id, max_draft_len, draft_tokens,
        draft_frames, draft_len, draft_full_len, utt_max_entropy, utt_status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

int launch_gate(const float *frame_entropy, const int64_t *frame_off, int B, int64_t N,
                float tau, uint8_t *gate_accept, float *max_entropy, int32_t *argmax_frame,
                cudaStream_t stream) {
    if (B == 0) return SSD_OK;
    gate_kernel<<<B, kUttThreads, 0, stream>>>(frame_entropy, frame_off, B, N, tau, gate_accept,
                                               max_entropy, argmax_frame);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

}  // namespace ssd
