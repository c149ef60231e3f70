// Pieces shared by the kernels that stream rows of LLM logits through a ring of shared-memory
// stages (ssd_verify, its early-exit variant, ssd_greedy_step): the stage descriptor, the
// per-thread running sum of exponentials and its once-per-stage range check, the FMA-pipe
// exponential split, the optional running arg max, and the warp-level merge.
#pragma once

#include <limits.h>
#include <math.h>

#include "ssd_common.cuh"

namespace ssd {
namespace stream {

constexpr int kOffCacheMax = 2048;     // utterance offsets kept in shared memory up to this many
constexpr uint32_t kFlagLast = 1u, kFlagEnd = 2u;
constexpr float kSumLimit = 1.0e30f;   // a running sum at or above this (or NaN) is recomputed


struct StageDesc {
    int32_t nchunks;
    uint32_t flags;
    int64_t slot;         // index of this item's first partial
    int32_t elem0;        // row-relative index of the first element of the stage's first chunk
    int32_t gather;       // early-exit variant: byte offset of the draft token's logit, or -1
};

// Running arg max of one thread (the greedy-step variant): the largest value so far, the
// row-relative index of its first occurrence (vidx), and, while a stage is being consumed, the
// stage's chunk in which the maximum last rose (vc, -1: not in this stage).  The chunk loop only
// keeps (vmax, vc) with a predicated select: no branch, since with 32 lanes some lane's maximum
// rises in most steps and a branch would be taken nearly always.  The position inside the chunk
// is looked up once per stage (resolve_arg), while the chunk is still in shared memory.
struct ArgTrack {
    float vmax;
    int vidx, vc;
    __device__ __forceinline__ void reset() { vmax = -INFINITY; vidx = INT_MAX; vc = -1; }
};
__device__ __forceinline__ float max3f(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
template <typename T>
__device__ __forceinline__ void resolve_arg(uint32_t a0, int elem0, ArgTrack &a) {
    constexpr int EPC = Elem<T>::kPerChunk;
    if (a.vc >= 0) {
        float x[EPC];
        chunk_unpack<T>(lds128(a0 + (uint32_t)a.vc * 16), x);
        int j = EPC - 1;
#pragma unroll
        for (int k = EPC - 2; k >= 0; --k) if (x[k] == a.vmax) j = k;
        a.vidx = elem0 + a.vc * EPC + j;
        a.vc = -1;
    }
}

// Running sum of exponentials of one thread, relative to a reference logit m that is one of the
// thread's own elements (or -inf while it has seen none).  fp32 keeps full relative precision
// over its whole exponent range, so m need not be the maximum: a thread only has to notice when
// a sum came near overflow (an element far above m), which it does once per stage, and then
// redoes that stage from shared memory with the proper maximum.  The common case therefore
// costs one exponential and no comparison per logit.
struct Online {
    float m, mh;
    float2 Sa, Sb;
    __device__ __forceinline__ void reset() {
        m = -INFINITY; mh = -INFINITY; Sa = Sb = make_float2(0.f, 0.f);
    }
    __device__ __forceinline__ float total() const { return (Sa.x + Sa.y) + (Sb.x + Sb.y); }
    __device__ __forceinline__ void raise_to(float nm) {
        const float sc = ex2(fmaf(m, kLog2e, -nm * kLog2e));      // 0 when m is still -inf
        Sa = fmul2(Sa, make_float2(sc, sc));
        Sb = fmul2(Sb, make_float2(sc, sc));
        m = nm; mh = nm * kLog2e;
    }
};

__device__ __forceinline__ float2 exp2_pair(float2 x, float2 scale, float2 nmh) {
    const float2 t = ffma2(x, scale, nmh);
    return make_float2(ex2(t.x), ex2(t.y));
}
__device__ __forceinline__ float2 exp2_pair_fma(float2 x, float2 scale, float2 nmh) {
    return exp2_fma_pair(ffma2(x, scale, nmh));
}

// kF of the 4 pairs of a bf16 chunk take the FMA-pipe exponential: the special-function unit
// (16 results per clock per SM) is what bounds this kernel for bf16 logits, and the FMA pipe
// has slots to spare.
template <typename T, int kF, bool kArg>
__device__ __forceinline__ void add_chunk(const uint4 &w, float nmh, Online &st, int c, ArgTrack &at) {
    const float2 sc = make_float2(kLog2e, kLog2e), nm = make_float2(nmh, nmh);
    if (Elem<T>::kBytes == 4) {
        const float2 x0 = make_float2(__uint_as_float(w.x), __uint_as_float(w.y));
        const float2 x1 = make_float2(__uint_as_float(w.z), __uint_as_float(w.w));
        if (kArg) {
            const float v = max3f(max3f(at.vmax, x0.x, x0.y), x1.x, x1.y);
            if (v > at.vmax) at.vc = c;
            at.vmax = v;
        }
        st.Sa = fadd2(st.Sa, exp2_pair(x0, sc, nm));
        st.Sb = fadd2(st.Sb, exp2_pair(x1, sc, nm));
    } else {
        const float2 x0 = make_float2(bf16_lo(w.x), bf16_hi(w.x)), x1 = make_float2(bf16_lo(w.y), bf16_hi(w.y));
        const float2 x2 = make_float2(bf16_lo(w.z), bf16_hi(w.z)), x3 = make_float2(bf16_lo(w.w), bf16_hi(w.w));
        if (kArg) {
            const float v = max3f(max3f(max3f(max3f(at.vmax, x0.x, x0.y), x1.x, x1.y), x2.x, x2.y), x3.x, x3.y);
            if (v > at.vmax) at.vc = c;
            at.vmax = v;
        }
        st.Sa = fadd2(st.Sa, kF >= 1 ? exp2_pair_fma(x0, sc, nm) : exp2_pair(x0, sc, nm));
        st.Sb = fadd2(st.Sb, kF >= 3 ? exp2_pair_fma(x1, sc, nm) : exp2_pair(x1, sc, nm));
        st.Sa = fadd2(st.Sa, kF >= 2 ? exp2_pair_fma(x2, sc, nm) : exp2_pair(x2, sc, nm));
        st.Sb = fadd2(st.Sb, exp2_pair(x3, sc, nm));
    }
}

// Adds this thread's chunks (ct, ct + NT, ...) of a stage holding n chunks to its running sum.
// Four chunks are fetched before any is used; the last, partial group of up to three is fetched
// together as well.
// With kArg the running arg max is updated as well.
template <typename T, int kF, bool kArg>
__device__ __forceinline__ void add_chunks(uint32_t a0, int n, int ct, int NT, Online &st,
                                           ArgTrack &at) {
    const float nmh = -st.mh;
    const uint32_t step = (uint32_t)NT * 16;
    uint32_t a = a0 + (uint32_t)ct * 16;
    int c = ct;
    for (; c + 3 * NT < n; c += 4 * NT, a += 4 * step) {
        const uint4 w0 = lds128(a), w1 = lds128(a + step), w2 = lds128(a + 2 * step),
                    w3 = lds128(a + 3 * step);
        add_chunk<T, kF, kArg>(w0, nmh, st, c, at);
        add_chunk<T, kF, kArg>(w1, nmh, st, c + NT, at);
        add_chunk<T, kF, kArg>(w2, nmh, st, c + 2 * NT, at);
        add_chunk<T, kF, kArg>(w3, nmh, st, c + 3 * NT, at);
    }
    if (c < n) {
        const bool h1 = c + NT < n, h2 = c + 2 * NT < n;
        const uint4 w0 = lds128(a);
        uint4 w1 = w0, w2 = w0;
        if (h1) w1 = lds128(a + step);
        if (h2) w2 = lds128(a + 2 * step);
        add_chunk<T, kF, kArg>(w0, nmh, st, c, at);
        if (h1) add_chunk<T, kF, kArg>(w1, nmh, st, c + NT, at);
        if (h2) add_chunk<T, kF, kArg>(w2, nmh, st, c + 2 * NT, at);
    }
}

template <typename T, int kF, bool kArg>
__device__ __forceinline__ void consume_stage(uint32_t a0, int n, int ct, int NT, Online &st,
                                              int elem0, ArgTrack &at) {
    if (ct >= n) return;
    if (!(st.m > -INFINITY)) {
        // no reference yet (start of a row): the largest element of the first chunk
        const float cm = chunk_max<T>(lds128(a0 + (uint32_t)ct * 16));
        if (cm > -INFINITY) { st.m = cm; st.mh = cm * kLog2e; }
    }
    const Online saved = st;
    add_chunks<T, kF, kArg>(a0, n, ct, NT, st, at);
    if (!(st.total() < kSumLimit)) {
        // an element far above the reference, a NaN or +inf, or only -inf so far: redo the
        // stage relative to the maximum of this thread's chunks
        st = saved;
        float cm = -INFINITY;
        for (int c = ct; c < n; c += NT) cm = fmaxf(cm, chunk_max<T>(lds128(a0 + (uint32_t)c * 16)));
        if (cm > st.m) st.raise_to(cm);
        if (st.m > -INFINITY) add_chunks<T, kF, kArg>(a0, n, ct, NT, st, at);
    }
    if (kArg) resolve_arg<T>(a0, elem0, at);
}

// Warp-level merge of the lanes' (m, S) into one pair relative to the warp maximum.
__device__ __forceinline__ float2 warp_merge(const Online &st) {
    const float S = st.total();
    const float ml = fmaf(st.m, kLog2e, -st.mh);        // exponents carried +ml: take it out
    const float M = warp_max(st.m);
    // S == 0 covers lanes that saw nothing (their m is -inf); a NaN sum still propagates
    const float Sw = warp_sum(S == 0.f ? 0.f : S * ex2(fmaf(st.m - M, kLog2e, -ml)));
    return make_float2(M, Sw);
}

}  // namespace stream
}  // namespace ssd
