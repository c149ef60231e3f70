// Shared device helpers of libssd: mbarrier / bulk-copy PTX wrappers for sm_100a, bounded
// waits, logit unpacking and small warp reductions.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ssd.h"

namespace ssd {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kNegInit = -1.0e30f;          // "no value yet" for a running maximum
constexpr long long kWaitLimitCycles = 1ll << 31;  // ~1 s at 2 GHz: bound of every spin wait

// ---- host-side launch bookkeeping ----------------------------------------------------------
struct Launch {
    cudaStream_t stream;
    const ssd_launch_opts *opts;
};

// ---- programmatic dependent launch ------------------------------------------------------------
// Every kernel of the library is launched so that it may be scheduled while its predecessor in
// the stream is still running, which takes the launch latency of the short per-utterance
// kernels off the critical path.  A kernel first lets its own successor be scheduled, then
// waits until every earlier grid has completed and its writes are visible; nothing before
// pdl_enter() / pdl_wait() touches global memory.  The streaming kernels call the two halves
// apart, with their shared-memory set-up in between, so that the set-up (and the cold
// instruction fetches that come with it) overlaps the predecessor's tail.
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void pdl_enter() {
    pdl_launch_dependents();
    pdl_wait();
}

void count_launch();     // one more kernel launched by this host thread (ssd_launch_count)

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem,
                       cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- shared-memory addresses and mbarriers ---------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

// Makes freshly initialised barriers visible to the async (bulk-copy) proxy.
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}

// Waits for the phase with the given parity to complete, for at most kWaitLimitCycles.
// Called by all 32 lanes of a warp; the answer is the same in every lane.  Returns false when
// the limit ran out (the caller records the error and winds down).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    bool ok = mbar_try_wait(bar, parity);
    if (!ok) {
        const long long t0 = clock64();
        while (!(ok = mbar_try_wait(bar, parity))) {
            if (clock64() - t0 > kWaitLimitCycles) break;
        }
    }
    return __all_sync(0xffffffffu, ok);
}

// 1-D bulk asynchronous copy global -> shared, completion counted in bytes on `bar`.
// dst, src 16-byte aligned; bytes a positive multiple of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes,
                                         uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}

// After a bounded wait has failed: give copies that may still be in flight time to land before
// the CTA's shared memory is released (bounded as well).
__device__ __forceinline__ void drain_after_error() {
    const long long t0 = clock64();
    while (clock64() - t0 < (1ll << 22)) __nanosleep(1000);
}

// ---- scratch words that need no clearing ------------------------------------------------------
// The 32-bit tag of call number n.  A word that this call has not written is told from one it
// has by the tag alone, and a workspace may hold anything.  Taken as it is, a small call number
// is what the upper half of such a word may well hold by chance: two int32 of an array that
// lived there before (seen: once in 80,000 calls on 1,000 utterances a status word of another
// tensor's leftovers passed for this call's).  With 0x9 in the top four bits the tag reads as
// an int32 below -1.6e9, a float of magnitude below 1e-28 or a bf16 pair whose upper half is
// one, none of which logits, token ids, offsets or lengths leave behind; the other 28 bits tell
// 268 million consecutive calls apart.
__host__ __device__ inline uint32_t scratch_tag(uint32_t n) { return 0x90000000u | (n & 0x0fffffffu); }

// Adds k to a {epoch : 32 | count : 32} word and returns the count before the add.  A word
// whose epoch is not this call's is a leftover (of an earlier call, or never written) and counts
// as {epoch, 0}.  Epochs grow from call to call, so one atomic max with {epoch, 0} replaces a
// leftover of an earlier call and leaves a word of this call alone; the add follows it without
// waiting.  Only a leftover with a larger epoch field (memory that held something else) takes
// the slow way: whoever sees it swaps {epoch, 0} in, and nobody adds before that has happened.
__device__ __forceinline__ uint32_t tagged_finish(unsigned long long *w, uint32_t epoch, uint32_t k,
                                                  unsigned long long old, bool &ok) {
    if ((uint32_t)(old >> 32) == epoch) return (uint32_t)old;
    const unsigned long long tag = (unsigned long long)epoch << 32;
    for (int tries = 0; tries < (1 << 16); ++tries) {
        const unsigned long long cur = *reinterpret_cast<volatile unsigned long long *>(w);
        if ((uint32_t)(cur >> 32) == epoch) return (uint32_t)atomicAdd(w, (unsigned long long)k);
        atomicCAS(w, cur, tag);
    }
    ok = false;
    return 0xffffffffu;
}
__device__ __forceinline__ unsigned long long tagged_begin(unsigned long long *w, uint32_t epoch,
                                                           uint32_t k) {
    atomicMax(w, (unsigned long long)epoch << 32);
    return atomicAdd(w, (unsigned long long)k);
}
__device__ __forceinline__ uint32_t tagged_add(unsigned long long *w, uint32_t epoch, uint32_t k,
                                               bool &ok) {
    return tagged_finish(w, epoch, k, tagged_begin(w, epoch, k), ok);
}
// Lowers a {epoch : 32 | value : 32} word to `value` (a leftover counts as "no value yet"), and
// ORs bits into one (a leftover counts as 0).  Compare-and-swap loops: for updates that are rare.
__device__ __forceinline__ void tagged_min(unsigned long long *w, uint32_t epoch, uint32_t value,
                                           bool &ok) {
    const unsigned long long mine = ((unsigned long long)epoch << 32) | value;
    unsigned long long cur = *reinterpret_cast<volatile unsigned long long *>(w);
    for (int tries = 0; tries < (1 << 12); ++tries) {
        if ((uint32_t)(cur >> 32) == epoch && (uint32_t)cur <= value) return;
        const unsigned long long old = atomicCAS(w, cur, mine);
        if (old == cur) return;
        cur = old;
    }
    ok = false;
}
__device__ __forceinline__ void tagged_or(unsigned long long *w, uint32_t epoch, uint32_t bits,
                                          bool &ok) {
    unsigned long long cur = *reinterpret_cast<volatile unsigned long long *>(w);
    for (int tries = 0; tries < (1 << 12); ++tries) {
        const uint32_t have = (uint32_t)(cur >> 32) == epoch ? (uint32_t)cur : 0u;
        if ((uint32_t)(cur >> 32) == epoch && (have | bits) == have) return;
        const unsigned long long old =
            atomicCAS(w, cur, ((unsigned long long)epoch << 32) | have | bits);
        if (old == cur) return;
        cur = old;
    }
    ok = false;
}

// ---- arithmetic -------------------------------------------------------------------------------
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Packed pairs of fp32 (sm_100 executes one instruction for both halves).
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
        "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
__device__ __forceinline__ float2 fmul2(float2 a, float2 b) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "mul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// max of two packed bf16 pairs (NaN operands lose)
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// the same, but a NaN operand wins (so that a NaN logit is not swallowed by a clamp)
__device__ __forceinline__ uint32_t bf16x2_max_nan(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ float fmax_nan(float a, float b) {
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

__device__ __forceinline__ float fmin_nan(float a, float b) {
    float d;
    asm("min.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

// 2^t for a pair, on the FMA pipe: round t to the nearest integer n with the 1.5*2^23 trick,
// evaluate a degree-4 polynomial for 2^f on f = t - n in [-1/2, 1/2] (relative error 3.6e-6)
// and add n to the exponent field.  t is clamped to [-126, 128] first: below, the result is at
// most 2^-126 where the true value is smaller; above, it is +inf (without the clamp the
// exponent field would wrap), which the callers' range checks catch.  NaN passes the clamps.
__device__ __forceinline__ float2 exp2_fma_pair(float2 t) {
    const float kMagic = 12582912.f;
    t.x = fmin_nan(fmax_nan(t.x, -126.f), 128.f);
    t.y = fmin_nan(fmax_nan(t.y, -126.f), 128.f);
    const float2 r = fadd2(t, make_float2(kMagic, kMagic));
    const float2 n = fadd2(r, make_float2(-kMagic, -kMagic));
    const float2 f = ffma2(n, make_float2(-1.f, -1.f), t);
    float2 p = make_float2(0.00966636836528778f, 0.00966636836528778f);
    p = ffma2(p, f, make_float2(0.055921975523233414f, 0.055921975523233414f));
    p = ffma2(p, f, make_float2(0.2402234971523285f, 0.2402234971523285f));
    p = ffma2(p, f, make_float2(0.6931210160255432f, 0.6931210160255432f));
    p = ffma2(p, f, make_float2(1.0f, 1.0f));
    float2 y;
    y.x = __int_as_float(__float_as_int(r.x) * (1 << 23) + __float_as_int(p.x));
    y.y = __int_as_float(__float_as_int(r.y) * (1 << 23) + __float_as_int(p.y));
    return y;
}

// order-preserving map float -> int32 (for integer warp reductions of float maxima)
__device__ __forceinline__ int32_t float_key(float f) {
    int32_t b = __float_as_int(f);
    return b >= 0 ? b : (b ^ 0x7fffffff);
}
__device__ __forceinline__ float key_float(int32_t k) {
    return __int_as_float(k >= 0 ? k : (k ^ 0x7fffffff));
}

__device__ __forceinline__ float warp_max(float v) {
    return key_float(__reduce_max_sync(0xffffffffu, float_key(v)));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kBytes = 4;
    static constexpr int kPerChunk = 4;  // elements in a 16-byte chunk
    __device__ static __forceinline__ float load(const void *p) {
        return *reinterpret_cast<const float *>(p);
    }
    __device__ static __forceinline__ float load_shared(uint32_t addr) {
        float v;
        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
        return v;
    }
    static constexpr uint32_t kNegInfBits = 0xff800000u;
};
struct bf16_t { uint16_t bits; };
template <> struct Elem<bf16_t> {
    static constexpr int kBytes = 2;
    static constexpr int kPerChunk = 8;
    __device__ static __forceinline__ float load(const void *p) {
        return __uint_as_float(static_cast<uint32_t>(*reinterpret_cast<const uint16_t *>(p)) << 16);
    }
    __device__ static __forceinline__ float load_shared(uint32_t addr) {
        uint16_t v;
        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
        return __uint_as_float(static_cast<uint32_t>(v) << 16);
    }
    static constexpr uint32_t kNegInfBits = 0xff80ff80u;
};

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(addr));
    return v;
}

// maximum of the elements of one 16-byte chunk
template <typename T> __device__ __forceinline__ float chunk_max(const uint4 &w);
template <> __device__ __forceinline__ float chunk_max<float>(const uint4 &w) {
    return fmaxf(fmaxf(__uint_as_float(w.x), __uint_as_float(w.y)),
                 fmaxf(__uint_as_float(w.z), __uint_as_float(w.w)));
}
template <> __device__ __forceinline__ float chunk_max<bf16_t>(const uint4 &w) {
    uint32_t h = bf16x2_max(bf16x2_max(w.x, w.y), bf16x2_max(w.z, w.w));
    return fmaxf(bf16_lo(h), bf16_hi(h));
}

// element j of a 16-byte chunk as float
template <typename T> __device__ __forceinline__ void chunk_unpack(const uint4 &w, float *x);
template <> __device__ __forceinline__ void chunk_unpack<float>(const uint4 &w, float *x) {
    x[0] = __uint_as_float(w.x); x[1] = __uint_as_float(w.y);
    x[2] = __uint_as_float(w.z); x[3] = __uint_as_float(w.w);
}
template <> __device__ __forceinline__ void chunk_unpack<bf16_t>(const uint4 &w, float *x) {
    x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
    x[4] = bf16_lo(w.z); x[5] = bf16_hi(w.z); x[6] = bf16_lo(w.w); x[7] = bf16_hi(w.w);
}

// index b in [0,B) with off[b] <= r < off[b+1] for monotone offsets; stays inside [0,B) for
// any offsets.  Returns -1 when B == 0.
__device__ __forceinline__ int utterance_of_row(const int64_t *off, int B, int64_t r) {
    if (B <= 0) return -1;
    int lo = 0, hi = B - 1;
    while (lo < hi) {
        int mid = (lo + hi + 1) >> 1;
        if (off[mid] <= r) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// ---- launchers implemented in the .cu files ---------------------------------------------------
struct CtcPlan {
    int kernel;          // 1 plain loads, 2 bulk-copy tiles
    int lanes_per_row;   // G
    int rows_per_tile;   // R
    int warps, stages, stage_stride;
    int iters, tail_from;   // chunk iterations per lane and row; first one that may be a row's last
    int fma_exp;            // pairs per bf16 chunk whose exponential runs on the FMA pipe
    int64_t num_tiles;
    size_t smem_bytes, workspace_bytes;
};
int plan_ctc(ssd_dtype dtype, int V, int64_t ld, int64_t N, int B, const ssd_launch_opts *opts,
             CtcPlan *plan);
int launch_ctc_rows(const void *logits, ssd_dtype dtype, int V, int64_t ld, int64_t N,
                    float *frame_entropy, int32_t *frame_argmax, float *frame_lse,
                    float *frame_logprob, void *workspace, const CtcPlan &plan, const Launch &L);
int launch_collapse(const int32_t *frame_argmax, const float *frame_entropy,
                    const int64_t *frame_off, int B, int64_t N, int blank_id, int max_draft_len,
                    int32_t *draft_tokens, int32_t *draft_frames, int32_t *draft_len,
                    int32_t *draft_full_len, float *utt_max_entropy, uint32_t *utt_status,
                    void *workspace, cudaStream_t stream);
int launch_gate(const float *frame_entropy, const int64_t *frame_off, int B, int64_t N,
                float tau, uint8_t *gate_accept, float *max_entropy, int32_t *argmax_frame,
                cudaStream_t stream);
int launch_gate_from_maxima(const float *utt_max_entropy, const uint32_t *utt_status, int B,
                            float tau, uint8_t *gate_accept, float *max_entropy,
                            cudaStream_t stream);

struct VerifyPlan {
    int kernel;        // 1 plain loads, 2 bulk-copy pipeline
    int ctas;
    int warps;         // consumer warps per CTA
    int stages;
    int stage_bytes;
    int split;         // column spans per row
    int fma_exp;       // pairs per chunk whose exponential runs on the FMA pipe (bf16 only)
    int partials;      // partial (max, sum) pairs per row = split * warps
    int finish_inside; // rows are finalised inside the streaming kernel (no closing kernel)
    size_t smem_bytes;
    size_t fin_smem_bytes;
    size_t workspace_bytes;
};
int plan_verify(int B, int64_t M, int V, ssd_dtype dtype, const ssd_launch_opts *opts,
                VerifyPlan *plan);
int launch_verify_shard(const void *logits, ssd_dtype dtype, int V_local, int64_t ld, int64_t M,
                        int64_t col0, const int64_t *tok_off, const int32_t *draft_ids, int B,
                        const uint8_t *skip, void *workspace, float *shard_stats,
                        const VerifyPlan &plan, const Launch &L);
int launch_verify_combine(const float *stats_all, int R, int64_t V_total, const int64_t *tok_off,
                          const int32_t *draft_ids, int B, int64_t M, float tau_slm,
                          const uint8_t *skip, float *token_logp, float *row_lse,
                          int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                          cudaStream_t stream);
int launch_verify(const void *logits, ssd_dtype dtype, int V, int64_t ld, int64_t M,
                  const int64_t *tok_off, const int32_t *draft_ids, int B, float tau_slm,
                  const uint8_t *skip, void *workspace, float *token_logp, float *row_lse,
                  int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                  const VerifyPlan &plan, const Launch &L);

size_t greedy_workspace_bytes(int64_t R, const VerifyPlan &plan);
int launch_greedy(const void *logits, ssd_dtype dtype, int V, int64_t ld, int64_t R,
                  void *workspace, int32_t *next_token, float *next_logp, float *row_lse,
                  uint32_t *row_status, const VerifyPlan &plan, const Launch &L);

int launch_sweep(const float *utt_max_entropy, const float *token_logp, const int64_t *tok_off,
                 int B, int64_t M, const float *tau_ctc, const float *tau_slm, int P,
                 uint8_t *gate_accept, int32_t *accepted_len, uint8_t *all_accepted,
                 int32_t *counts, cudaStream_t stream);
int launch_assemble(const int32_t *tokens, const int64_t *tok_off, int B, int64_t M,
                    const uint8_t *gate_accept, const int32_t *accepted_len,
                    const uint8_t *all_accepted, int32_t *final_tokens, int32_t *final_len,
                    uint8_t *is_final, int32_t *ar_count, int32_t *ar_utt, int32_t *ar_resume,
                    cudaStream_t stream);

size_t verify_ee_workspace_bytes(int B, const VerifyPlan &full_plan);
bool verify_ee_applicable(int B, int64_t M, const VerifyPlan &plan);
int launch_verify_ee(const void *logits, ssd_dtype dtype, int V, int64_t ld, int64_t M,
                     const int64_t *tok_off, const int32_t *draft_ids, int B, float tau_slm,
                     const uint8_t *skip, void *workspace, float *token_logp, float *row_lse,
                     int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                     int32_t *rows_read, const VerifyPlan &plan, const Launch &L);

void record_cuda_error(cudaError_t e);

// Multiprocessors of the current device (looked up once per device); <= 0 when the device cannot
// be asked.  The host-only read-span hooks replay the plans without any device: while one of
// them runs on this thread, the count of the part the kernels are tuned for (148) stands in.
int device_sm_count();
struct PlanReplay {
    PlanReplay();
    ~PlanReplay();
};

// cudaFuncAttributeMaxDynamicSharedMemorySize, set once per kernel and device (and again only
// if a launch needs more than any before it).
cudaError_t ensure_dynamic_smem(const void *kernel, size_t bytes);

}  // namespace ssd
