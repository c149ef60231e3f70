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

// Running arg max of one thread (the greedy-step variant): value and row-relative index of the
// first element that attains it.
struct ArgTrack {
    float vmax;
    int vidx;
    __device__ __forceinline__ void reset() { vmax = -INFINITY; vidx = INT_MAX; }
};
template <typename T>
__device__ __forceinline__ void track_chunk(const uint4 &w, int elem, ArgTrack &a) {
    constexpr int EPC = Elem<T>::kPerChunk;
    const float cm = chunk_max<T>(w);
    if (cm > a.vmax) {                   // rare: a running maximum rises O(log n) times
        float x[EPC];
        chunk_unpack<T>(w, x);
        int j = EPC - 1;
#pragma unroll
        for (int k = EPC - 2; k >= 0; --k) if (x[k] == cm) j = k;
        a.vmax = cm;
        a.vidx = elem + j;
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
template <typename T, int kF>
__device__ __forceinline__ void add_chunk(const uint4 &w, float nmh, Online &st) {
    const float2 sc = make_float2(kLog2e, kLog2e), nm = make_float2(nmh, nmh);
    if (Elem<T>::kBytes == 4) {
        st.Sa = fadd2(st.Sa, exp2_pair(make_float2(__uint_as_float(w.x), __uint_as_float(w.y)), sc, nm));
        st.Sb = fadd2(st.Sb, exp2_pair(make_float2(__uint_as_float(w.z), __uint_as_float(w.w)), sc, nm));
    } else {
        const float2 x0 = make_float2(bf16_lo(w.x), bf16_hi(w.x)), x1 = make_float2(bf16_lo(w.y), bf16_hi(w.y));
        const float2 x2 = make_float2(bf16_lo(w.z), bf16_hi(w.z)), x3 = make_float2(bf16_lo(w.w), bf16_hi(w.w));
        st.Sa = fadd2(st.Sa, kF >= 1 ? exp2_pair_fma(x0, sc, nm) : exp2_pair(x0, sc, nm));
        st.Sb = fadd2(st.Sb, kF >= 3 ? exp2_pair_fma(x1, sc, nm) : exp2_pair(x1, sc, nm));
        st.Sa = fadd2(st.Sa, kF >= 2 ? exp2_pair_fma(x2, sc, nm) : exp2_pair(x2, sc, nm));
        st.Sb = fadd2(st.Sb, exp2_pair(x3, sc, nm));
    }
}

// Adds this thread's chunks (ct, ct + NT, ...) of a stage holding n chunks to its running sum.
// Four chunks are fetched before any is used; the last, partial group of up to three is fetched
// together as well.
// With kArg the running arg max is updated as well (elem0: row-relative element index of the
// stage's chunk 0).
template <typename T, int kF, bool kArg>
__device__ __forceinline__ void add_chunks(uint32_t a0, int n, int ct, int NT, Online &st,
                                           int elem0, ArgTrack &at) {
    constexpr int EPC = Elem<T>::kPerChunk;
    const float nmh = -st.mh;
    const uint32_t step = (uint32_t)NT * 16;
    uint32_t a = a0 + (uint32_t)ct * 16;
    int c = ct;
    for (; c + 3 * NT < n; c += 4 * NT, a += 4 * step) {
        const uint4 w0 = lds128(a), w1 = lds128(a + step), w2 = lds128(a + 2 * step),
                    w3 = lds128(a + 3 * step);
        if (kArg) {
            track_chunk<T>(w0, elem0 + c * EPC, at);
            track_chunk<T>(w1, elem0 + (c + NT) * EPC, at);
            track_chunk<T>(w2, elem0 + (c + 2 * NT) * EPC, at);
            track_chunk<T>(w3, elem0 + (c + 3 * NT) * EPC, at);
        }
        add_chunk<T, kF>(w0, nmh, st);
        add_chunk<T, kF>(w1, nmh, st);
        add_chunk<T, kF>(w2, nmh, st);
        add_chunk<T, kF>(w3, nmh, st);
    }
    if (c < n) {
        const bool h1 = c + NT < n, h2 = c + 2 * NT < n;
        const uint4 w0 = lds128(a);
        uint4 w1 = w0, w2 = w0;
        if (h1) w1 = lds128(a + step);
        if (h2) w2 = lds128(a + 2 * step);
        if (kArg) {
            track_chunk<T>(w0, elem0 + c * EPC, at);
            if (h1) track_chunk<T>(w1, elem0 + (c + NT) * EPC, at);
            if (h2) track_chunk<T>(w2, elem0 + (c + 2 * NT) * EPC, at);
        }
        add_chunk<T, kF>(w0, nmh, st);
        if (h1) add_chunk<T, kF>(w1, nmh, st);
        if (h2) add_chunk<T, kF>(w2, nmh, st);
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
    add_chunks<T, kF, kArg>(a0, n, ct, NT, st, elem0, at);
    if (!(st.total() < kSumLimit)) {
        // an element far above the reference, a NaN or +inf, or only -inf so far: redo the
        // stage relative to the maximum of this thread's chunks
        st = saved;
        float cm = -INFINITY;
        for (int c = ct; c < n; c += NT) cm = fmaxf(cm, chunk_max<T>(lds128(a0 + (uint32_t)c * 16)));
        if (cm > st.m) st.raise_to(cm);
        if (st.m > -INFINITY) add_chunks<T, kF, kArg>(a0, n, ct, NT, st, elem0, at);
    }
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
