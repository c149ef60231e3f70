// Stage 1 kernels: per-frame softmax statistics of the CTC head (Eq. 2, Eq. 3), the collapse
// B of Section 2.1, and the entropy gate of Eq. 3.
//
// Frame statistics are one streaming read of the [N, V] logits.  Two kernels compute them:
//   ctc_rows_tma    each warp owns a shared-memory stage that it fills with one 1-D bulk
//                   asynchronous copy (TMA) of a few consecutive rows and drains itself: no
//                   block-level synchronisation after set-up.  G lanes share a row; one fused
//                   pass per row keeps a running maximum and the sums of 2^t and t*2^t
//                   relative to a per-lane reference, so a logit costs one exponential; rows
//                   that pass cannot take (masked -inf logits, NaN, +inf, a range beyond fp32)
//                   are redone from shared memory by an exact two-pass routine.
//   ctc_rows_plain  one warp per row with scalar global loads; any alignment, any V.  Fallback.
#include <limits.h>
#include <math.h>

#include "ssd_common.cuh"
#include "ssd_ranges.cuh"

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
    int iters;             // chunk iterations per lane and row: ceil(most chunks a row touches / G)
    int tail_from;         // first iteration (>= 1) in which a lane may meet its row's last chunk
    float *frame_entropy;
    int32_t *frame_argmax;
    float *frame_lse;
    float *frame_logprob;
    // tiles are handed out from up to four counters in the caller's workspace, 256 bytes
    // apart (NULL: tile j to warp j mod the number of warps).  A word is {epoch : 32 | count :
    // 32}, so a call needs no clearing of what the last one left there.
    unsigned long long *tile_counter;
    const unsigned long long *launch_gen;   // launches this workspace has seen (see launch_ctc_rows)
    uint32_t epoch;
    int counters;          // C
    int claim;             // tiles per claim
};

// Replaces the elements of a 16-byte chunk outside [e_lo, e_hi) (they belong to a neighbouring
// row, to the padding between rows, or were never written) by -inf.
template <typename T> __device__ __forceinline__ void mask_chunk(uint4 &w, int e_lo, int e_hi);
template <> __device__ __forceinline__ void mask_chunk<float>(uint4 &w, int e_lo, int e_hi) {
    const uint32_t fill = 0xff800000u;
    if (0 < e_lo || 0 >= e_hi) w.x = fill;
    if (1 < e_lo || 1 >= e_hi) w.y = fill;
    if (2 < e_lo || 2 >= e_hi) w.z = fill;
    if (3 < e_lo || 3 >= e_hi) w.w = fill;
}
__device__ __forceinline__ uint32_t mask_pair(uint32_t v, int j, int e_lo, int e_hi) {
    const uint32_t fill = 0xff80u;
    if (j < e_lo || j >= e_hi) v = (v & 0xffff0000u) | fill;
    if (j + 1 < e_lo || j + 1 >= e_hi) v = (v & 0x0000ffffu) | (fill << 16);
    return v;
}
template <> __device__ __forceinline__ void mask_chunk<bf16_t>(uint4 &w, int e_lo, int e_hi) {
    w.x = mask_pair(w.x, 0, e_lo, e_hi);
    w.y = mask_pair(w.y, 2, e_lo, e_hi);
    w.z = mask_pair(w.z, 4, e_lo, e_hi);
    w.w = mask_pair(w.w, 6, e_lo, e_hi);
}

// S += 2^t, A += t * 2^t for the elements of one chunk, t = x*log2e - mh.  Elements are first
// clamped from below so that a masked (-inf) logit gives t*2^t = 0 instead of NaN.
template <typename T>
__device__ __forceinline__ void entropy_chunk(const uint4 &w, float nmh, float2 &Sa, float2 &Sb,
                                              float2 &Aa, float2 &Ab);
__device__ __forceinline__ void entropy_pair(float2 x, float nmh, float2 &S, float2 &A) {
    const float2 t = ffma2(x, make_float2(kLog2e, kLog2e), make_float2(nmh, nmh));
    const float2 e = make_float2(ex2(t.x), ex2(t.y));
    S = fadd2(S, e);
    A = ffma2(t, e, A);
}
template <>
__device__ __forceinline__ void entropy_chunk<float>(const uint4 &w, float nmh, float2 &Sa,
                                                     float2 &Sb, float2 &Aa, float2 &Ab) {
    const float lo = -1.0e30f;
    entropy_pair(make_float2(fmax_nan(__uint_as_float(w.x), lo), fmax_nan(__uint_as_float(w.y), lo)),
                 nmh, Sa, Aa);
    entropy_pair(make_float2(fmax_nan(__uint_as_float(w.z), lo), fmax_nan(__uint_as_float(w.w), lo)),
                 nmh, Sb, Ab);
}
template <>
__device__ __forceinline__ void entropy_chunk<bf16_t>(const uint4 &w, float nmh, float2 &Sa,
                                                      float2 &Sb, float2 &Aa, float2 &Ab) {
    const uint32_t lo = 0xf149f149u;      // bf16 pair of -1.0e30 (rounded)
    const uint32_t x = bf16x2_max_nan(w.x, lo), y = bf16x2_max_nan(w.y, lo);
    const uint32_t z = bf16x2_max_nan(w.z, lo), u = bf16x2_max_nan(w.w, lo);
    entropy_pair(make_float2(bf16_lo(x), bf16_hi(x)), nmh, Sa, Aa);
    entropy_pair(make_float2(bf16_lo(y), bf16_hi(y)), nmh, Sb, Ab);
    entropy_pair(make_float2(bf16_lo(z), bf16_hi(z)), nmh, Sa, Aa);
    entropy_pair(make_float2(bf16_lo(u), bf16_hi(u)), nmh, Sb, Ab);
}

template <int G> __device__ __forceinline__ float group_max(float v) {
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
template <int G> __device__ __forceinline__ int group_min(int v) {
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
template <int G> __device__ __forceinline__ float group_sum(float v) {
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

struct RowOut {
    float lse, H;
    int arg;
};

// Geometry of one row inside a stage: the 16-byte chunks [cf, cl] it touches and which
// elements of the first and last chunk are its own.
struct RowSpan {
    int cf, cl, e_lo, e_hi;
};

// Exact two-pass softmax of one row by the G lanes of a group (all 32 lanes call it).  Pass 1
// finds the maximum m and where it first occurs, pass 2 sums e = 2^((x-m)*log2e) and
// (x-m)*log2e*e with masked logits clamped.  With mh = fl(m*log2e) and ml = m*log2e - mh
// (exact, by fma) every exponent carries the same +ml, which cancels in the entropy and is
// removed from the log-sum-exp at the end.  This is the path for rows the fused pass below
// cannot take (masked -inf logits, NaN, +inf, a dynamic range beyond fp32's exponent).
template <typename T, int G>
__device__ __noinline__ RowOut reduce_row_exact(uint32_t stage_addr, RowSpan r, int sub) {
    constexpr int EPC = Elem<T>::kPerChunk;
    const int cf = r.cf, cl = r.cl, e_lo = r.e_lo, e_hi = r.e_hi;
    float vmax = -INFINITY;
    int vc = -1;
    for (int c = cf + sub; c <= cl; c += G) {
        uint4 w = lds128(stage_addr + (uint32_t)c * 16);
        if (c == cf || c == cl) mask_chunk<T>(w, c == cf ? e_lo : 0, c == cl ? e_hi : EPC);
        const float cm = chunk_max<T>(w);
        if (cm > vmax) { vmax = cm; vc = c; }
    }
    const float m = group_max<G>(vmax);
    int cand = INT_MAX;
    if (vc >= 0 && vmax == m) {
        uint4 w = lds128(stage_addr + (uint32_t)vc * 16);
        if (vc == cf || vc == cl) mask_chunk<T>(w, vc == cf ? e_lo : 0, vc == cl ? e_hi : EPC);
        float x[EPC];
        chunk_unpack<T>(w, x);
        int j = EPC - 1;
#pragma unroll
        for (int k = EPC - 2; k >= 0; --k) if (x[k] == m) j = k;
        cand = (vc - cf) * EPC + j - e_lo;
    }
    RowOut out;
    out.arg = group_min<G>(cand);
    if (out.arg == INT_MAX) out.arg = 0;
    const float mh = m * kLog2e;
    const float ml = fmaf(m, kLog2e, -mh);
    float2 Sa = make_float2(0.f, 0.f), Sb = Sa, Aa = Sa, Ab = Sa;
    for (int c = cf + sub; c <= cl; c += G) {
        uint4 w = lds128(stage_addr + (uint32_t)c * 16);
        if (c == cf || c == cl) mask_chunk<T>(w, c == cf ? e_lo : 0, c == cl ? e_hi : EPC);
        entropy_chunk<T>(w, -mh, Sa, Sb, Aa, Ab);
    }
    const float S = group_sum<G>((Sa.x + Sa.y) + (Sb.x + Sb.y));
    const float A2 = group_sum<G>((Aa.x + Aa.y) + (Ab.x + Ab.y));
    const float lnS = logf(S);
    out.lse = m + (lnS - ml * kLn2);
    out.H = fmaxf(lnS - kLn2 * (A2 / S), 0.f);
    if (!(S > 0.5f) || !(S < INFINITY) || !(fabsf(m) < INFINITY))
        out.H = __int_as_float(0x7fc00000);       // NaN / +inf / all -inf: flagged downstream
    return out;
}

// ---- the fused pass with a uniform trip count ---------------------------------------------------
// Every lane makes the same number of chunk iterations per row (p.iters, fixed by V and G alone),
// so a pass over 32/G rows has no data-dependent control flow.  Iteration 0 and the iterations
// from p.tail_from on may meet a row's first or last chunk, or lie past the row's end: their
// chunk goes through a keep mask looked up in a small shared-memory table (which elements
// [lo, hi) of a chunk are the row's own; hi = 0 keeps nothing), and what is not kept becomes a
// finite fill value near -1e30 whose exponential is 0.  The iterations in between are interior
// chunks and take no mask at all.
template <typename T> struct FillWord;
template <> struct FillWord<float> { static constexpr uint32_t v = 0xf149f2cau; };
template <> struct FillWord<bf16_t> { static constexpr uint32_t v = 0xf149f149u; };

// table entry (lo, hi) at index lo * (EPC + 1) + hi: all-ones in the bytes of elements [lo, hi)
template <typename T>
__device__ __forceinline__ void build_keep_table(uint4 *tab, int tid, int nthreads) {
    constexpr int EPC = Elem<T>::kPerChunk, ES = Elem<T>::kBytes;
    for (int e = tid; e < EPC * (EPC + 1); e += nthreads) {
        const int lo = e / (EPC + 1), hi = e - lo * (EPC + 1);
        uint32_t k[4];
#pragma unroll
        for (int wd = 0; wd < 4; ++wd) {
            if (ES == 4) {
                k[wd] = (lo <= wd && wd < hi) ? 0xffffffffu : 0u;
            } else {
                k[wd] = ((lo <= 2 * wd && 2 * wd < hi) ? 0x0000ffffu : 0u) |
                        ((lo <= 2 * wd + 1 && 2 * wd + 1 < hi) ? 0xffff0000u : 0u);
            }
        }
        tab[e] = make_uint4(k[0], k[1], k[2], k[3]);
    }
}

template <typename T> __device__ __forceinline__ uint4 lds_keep(uint32_t addr, uint32_t entry) {
    constexpr uint32_t F = FillWord<T>::v;
    uint4 w = lds128(addr);
    const uint4 k = lds128(entry);
    w.x = (w.x & k.x) | (F & ~k.x);
    w.y = (w.y & k.y) | (F & ~k.y);
    w.z = (w.z & k.z) | (F & ~k.z);
    w.w = (w.w & k.w) | (F & ~k.w);
    return w;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// 2^t for a pair on the FMA pipe, for t already known to be >= -126 (the caller clamps the
// logits from below) and not checked from above (the caller tests its largest exponent once
// per row): nearest integer n by the 1.5*2^23 trick, a degree-4 polynomial for 2^f on
// f = t - n in [-1/2, 1/2] (relative error 3.6e-6), n added into the exponent field.
__device__ __forceinline__ float2 exp2_fma_pair_inrange(float2 t) {
    const float kMagic = 12582912.f;
    const float2 r = fadd2(t, make_float2(kMagic, kMagic));
    const float2 n = fadd2(r, make_float2(-kMagic, -kMagic));
    const float2 f = ffma2(n, make_float2(-1.f, -1.f), t);
    float2 q = make_float2(0.00966636836528778f, 0.00966636836528778f);
    q = ffma2(q, f, make_float2(0.055921975523233414f, 0.055921975523233414f));
    q = ffma2(q, f, make_float2(0.2402234971523285f, 0.2402234971523285f));
    q = ffma2(q, f, make_float2(0.6931210160255432f, 0.6931210160255432f));
    q = ffma2(q, f, make_float2(1.0f, 1.0f));
    float2 y;
    y.x = __int_as_float(__float_as_int(r.x) * (1 << 23) + __float_as_int(q.x));
    y.y = __int_as_float(__float_as_int(r.y) * (1 << 23) + __float_as_int(q.y));
    return y;
}

// S += 2^t, A += t*2^t over one chunk (t = x*log2e + nrh) and the running maximum with the
// chunk it was first met in.  With kF, that many of a bf16 chunk's four pairs take the FMA-pipe
// exponential; `floor2` is then a packed pair of a bf16 value below which those logits are
// raised first (their exponentials are below 2^-124 either way).
template <int kF> __device__ __forceinline__ void entropy_pair2(float2 x, float nrh, float2 &S, float2 &A) {
    const float2 t = ffma2(x, make_float2(kLog2e, kLog2e), make_float2(nrh, nrh));
    const float2 e = kF ? exp2_fma_pair_inrange(t) : make_float2(ex2(t.x), ex2(t.y));
    S = fadd2(S, e);
    A = ffma2(t, e, A);
}
template <typename T, int kF> struct FusedChunk;
template <int kF> struct FusedChunk<float, kF> {
    static __device__ __forceinline__ void run(const uint4 &w, int c, float nrh, uint32_t, float &vmax,
                                               int &vc, float2 &Sa, float2 &Sb, float2 &Aa, float2 &Ab) {
        const float x0 = __uint_as_float(w.x), x1 = __uint_as_float(w.y);
        const float x2 = __uint_as_float(w.z), x3 = __uint_as_float(w.w);
        const float nm = max3(max3(vmax, x0, x1), x2, x3);
        if (nm > vmax) vc = c;
        vmax = nm;
        entropy_pair2<0>(make_float2(x0, x1), nrh, Sa, Aa);
        entropy_pair2<0>(make_float2(x2, x3), nrh, Sb, Ab);
    }
};
template <int kF> struct FusedChunk<bf16_t, kF> {
    static __device__ __forceinline__ void run(const uint4 &w, int c, float nrh, uint32_t floor2,
                                               float &vmax, int &vc, float2 &Sa, float2 &Sb,
                                               float2 &Aa, float2 &Ab) {
        const float x0 = bf16_lo(w.x), x1 = bf16_hi(w.x), x2 = bf16_lo(w.y), x3 = bf16_hi(w.y);
        const float x4 = bf16_lo(w.z), x5 = bf16_hi(w.z), x6 = bf16_lo(w.w), x7 = bf16_hi(w.w);
        const float nm = max3(max3(max3(max3(vmax, x0, x1), x2, x3), x4, x5), x6, x7);
        if (nm > vmax) vc = c;
        vmax = nm;
        if (kF >= 1) {
            const uint32_t u = bf16x2_max_nan(w.x, floor2);
            entropy_pair2<1>(make_float2(bf16_lo(u), bf16_hi(u)), nrh, Sa, Aa);
        } else {
            entropy_pair2<0>(make_float2(x0, x1), nrh, Sa, Aa);
        }
        if (kF >= 2) {
            const uint32_t u = bf16x2_max_nan(w.y, floor2);
            entropy_pair2<1>(make_float2(bf16_lo(u), bf16_hi(u)), nrh, Sb, Ab);
        } else {
            entropy_pair2<0>(make_float2(x2, x3), nrh, Sb, Ab);
        }
        entropy_pair2<0>(make_float2(x4, x5), nrh, Sa, Aa);
        entropy_pair2<0>(make_float2(x6, x7), nrh, Sb, Ab);
    }
};

// Frame statistics of the rows of one tile that lies in shared memory.  G lanes share a row and
// a warp works on 32/G rows at a time; a row is walked in the 16-byte chunks of the stage (whose
// alignment is that of global memory), lane `sub` taking chunks sub, sub + G, ...
//
// Fused single pass: a lane takes the largest element of its first chunk as reference (rh =
// fl(ref*log2e), in log2 units) and, for every chunk, updates its running maximum and adds 2^t
// and t*2^t, t = x*log2e - rh (one fma).  fp32 keeps full relative precision whatever the
// reference, so the sums only have to stay in range; at the end the lanes' sums are re-based to
// mh = fl(m*log2e) of the row maximum m (S' = S*2^d, A' = (A + d*S)*2^d with d = rh - mh, an
// exact difference) and added; ml = m*log2e - mh (exact, by fma) is taken out of the log-sum-exp
// and cancels in the entropy.  One exponential per logit.  A group whose sums left the range or
// turned NaN (a logit far above the reference, masked -inf logits, NaN, +inf) is redone by the
// exact two-pass routine above.
template <typename T, int G, int kF>
__device__ __forceinline__ void reduce_tile(const CtcParams &p, uint32_t stage_addr, uint32_t keep_tab,
                                            uint32_t head, int64_t r0, int nrows, int lane) {
    constexpr int ES = Elem<T>::kBytes, EPC = Elem<T>::kPerChunk, RPW = 32 / G;
    constexpr uint32_t STEP = (uint32_t)G * 16;
    const int sub = lane % G, grp = lane / G;
    const uint32_t pitch = (uint32_t)(p.ld * ES), row_bytes = (uint32_t)p.V * ES;
    constexpr int kDepth = 8;       // interior chunks in flight per lane
    const int ITER = p.iters, KT = p.tail_from;
    for (int g0 = 0; g0 < nrows; g0 += RPW) {
        const int i = g0 + grp;
        const bool valid = i < nrows;
        const uint32_t off = head + (uint32_t)(valid ? i : 0) * pitch;
        RowSpan r;
        r.cf = (int)(off >> 4);
        r.cl = valid ? (int)((off + row_bytes - 1) >> 4) : r.cf - 1;
        r.e_lo = (int)(off & 15) / ES;
        r.e_hi = (int)((off + row_bytes - 1) & 15) / ES + 1;
        const int cf = r.cf, cl = r.cl;

        int c = cf + sub;
        const bool has = c <= cl;
        uint32_t a = stage_addr + (uint32_t)c * 16;
        float vmax = -INFINITY;
        int vc = -1;
        float2 Sa = make_float2(0.f, 0.f), Sb = Sa, Aa = Sa, Ab = Sa;
        float nrh;
        uint32_t floor2 = 0;
        bool coarse = false;
        {
            // iteration 0: the row's first chunk for lane 0 of the group (and, for a very short
            // row, possibly its last one, or nothing at all)
            const int lo = sub == 0 ? r.e_lo : 0;
            const int hi = c < cl ? EPC : (c == cl ? r.e_hi : 0);
            const uint4 w = lds_keep<T>(a, keep_tab + (uint32_t)(lo * (EPC + 1) + hi) * 16);
            const float cm = chunk_max<T>(w);
            const float ref = cm > -1.0e29f ? cm : 0.f;
            nrh = -(ref * kLog2e);
            if (kF) {
                // bf16 (rounded up) of ref - 85: t = (x - ref)*log2e stays above -126.  For
                // |ref| < 4096 a bf16 step is at most 16, so the floor stays 69 below ref.
                coarse = !(fabsf(ref) < 4096.f);
                uint32_t fb = __float_as_uint(ref - 85.f);
                fb = (fb & 0x80000000u) ? fb : fb + 0xffffu;
                floor2 = (fb >> 16) * 0x10001u;
            }
            FusedChunk<T, kF>::run(w, c, nrh, floor2, vmax, vc, Sa, Sb, Aa, Ab);
        }
        a += STEP; c += G;
        int k = 1;
        {
            // kDepth chunks in flight: with at most 16 warps per SM (128 registers each) the
            // arithmetic hides its own latencies only if a warp has many independent chunks
            // to work on (four in flight at 24 warps and 80 registers ran 8 % slower)
#pragma unroll 1
            for (; k + kDepth <= KT; k += kDepth) {
                uint4 w[kDepth];
#pragma unroll
                for (int j = 0; j < kDepth; ++j) w[j] = lds128(a + j * STEP);
                // The block's terms are summed on their own and added to the lane's sums once:
                // a row with one logit far above the rest leaves 2^17 and more in a sum, and a
                // thousand equal small terms added to that one by one each lose the same
                // fraction of an ulp (seen: 1.4e-4 in the entropy of 5,000 bf16 logits with
                // four lanes per row; 1.5e-5 this way).
                float2 sa = make_float2(0.f, 0.f), sb = sa, aa = sa, ab = sa;
#pragma unroll
                for (int j = 0; j < kDepth; ++j)
                    FusedChunk<T, kF>::run(w[j], c + j * G, nrh, floor2, vmax, vc, sa, sb, aa, ab);
                Sa = fadd2(Sa, sa); Sb = fadd2(Sb, sb); Aa = fadd2(Aa, aa); Ab = fadd2(Ab, ab);
                a += kDepth * STEP; c += kDepth * G;
            }
        }
#pragma unroll 1
        for (; k + 4 <= KT; k += 4) {           // interior chunks, four in flight
            const uint4 w0 = lds128(a), w1 = lds128(a + STEP), w2 = lds128(a + 2 * STEP),
                        w3 = lds128(a + 3 * STEP);
            FusedChunk<T, kF>::run(w0, c, nrh, floor2, vmax, vc, Sa, Sb, Aa, Ab);
            FusedChunk<T, kF>::run(w1, c + G, nrh, floor2, vmax, vc, Sa, Sb, Aa, Ab);
            FusedChunk<T, kF>::run(w2, c + 2 * G, nrh, floor2, vmax, vc, Sa, Sb, Aa, Ab);
            FusedChunk<T, kF>::run(w3, c + 3 * G, nrh, floor2, vmax, vc, Sa, Sb, Aa, Ab);
            a += 4 * STEP; c += 4 * G;
        }
#pragma unroll 1
        for (; k < KT; ++k) {
            const uint4 w = lds128(a);
            FusedChunk<T, kF>::run(w, c, nrh, floor2, vmax, vc, Sa, Sb, Aa, Ab);
            a += STEP; c += G;
        }
#pragma unroll 1
        for (; k < ITER; ++k) {                  // may hold the row's last chunk, or lie past it
            const int hi = c < cl ? EPC : (c == cl ? r.e_hi : 0);
            const uint4 w = lds_keep<T>(a, keep_tab + (uint32_t)hi * 16);
            FusedChunk<T, kF>::run(w, c, nrh, floor2, vmax, vc, Sa, Sb, Aa, Ab);
            a += STEP; c += G;
        }
        const float Sl = (Sa.x + Sa.y) + (Sb.x + Sb.y), Al = (Aa.x + Aa.y) + (Ab.x + Ab.y);
        // out of range, NaN, or a lane whose own elements are all below the fill value
        // (with the FMA-pipe exponential also: a logit 2^120 above the reference, which that
        // exponential does not represent, or a reference too large for the bf16 floor)
        const bool bad = valid && has && (!(Sl < 1.0e30f) || Al != Al || !(vmax > -1.0e29f) ||
                                          (kF && (coarse || !(fmaf(vmax, kLog2e, nrh) < 120.f))));
        RowOut out;
        if (__any_sync(0xffffffffu, bad)) {
            out = reduce_row_exact<T, G>(stage_addr, r, sub);
        } else {
            const float m = group_max<G>(has ? vmax : -INFINITY);
            int cand = INT_MAX;
            if (has && vmax == m) {
                const int lo = vc == cf ? r.e_lo : 0;
                const int hi = vc == cl ? r.e_hi : EPC;
                const uint4 w = lds_keep<T>(stage_addr + (uint32_t)vc * 16,
                                            keep_tab + (uint32_t)(lo * (EPC + 1) + hi) * 16);
                float x[EPC];
                chunk_unpack<T>(w, x);
                int j = EPC - 1;
#pragma unroll
                for (int q = EPC - 2; q >= 0; --q) if (x[q] == m) j = q;
                cand = (vc - cf) * EPC + j - r.e_lo;
            }
            out.arg = group_min<G>(cand);
            if (out.arg == INT_MAX) out.arg = 0;
            const float mh = m * kLog2e;
            const float ml = fmaf(m, kLog2e, -mh);
            const float d = -nrh - mh;                   // <= 0 for a lane that holds chunks
            const float sc = has ? ex2(d) : 0.f;         // a lane without chunks adds nothing
            const float S = group_sum<G>(Sl * sc);
            const float A2 = group_sum<G>(fmaf(d, Sl, Al) * sc);
            // fast logarithm and division: absolute error near 1e-6, far inside the tolerance
            const float lnS = __logf(S);
            out.lse = m + (lnS - ml * kLn2);
            out.H = fmaxf(lnS - kLn2 * __fdividef(A2, S), 0.f);
            if (!(S > 0.5f) || !(S < INFINITY) || !(fabsf(m) < INFINITY))
                out.H = __int_as_float(0x7fc00000);
        }
        if (valid && sub == 0) {
            p.frame_entropy[r0 + i] = out.H;
            p.frame_argmax[r0 + i] = out.arg;
            if (p.frame_lse) p.frame_lse[r0 + i] = out.lse;
        }
        if (p.frame_logprob && valid) {
            float *o = p.frame_logprob + (r0 + i) * p.ld;
            for (int e = sub; e < p.V; e += G)
                o[e] = Elem<T>::load_shared(stage_addr + off + e * ES) - out.lse;
        }
    }
}

struct MaxAt {
    float v;
    int at;
};
__device__ __forceinline__ MaxAt better(MaxAt a, MaxAt b) {
    // larger value wins; on equal values the earlier frame; "at < 0" means empty
    if (b.at >= 0 && (a.at < 0 || b.v > a.v || (b.v == a.v && b.at < a.at))) return b;
    return a;
}
__device__ __forceinline__ MaxAt warp_max_at(MaxAt x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MaxAt y;
        y.v = __shfl_xor_sync(0xffffffffu, x.v, o);
        y.at = __shfl_xor_sync(0xffffffffu, x.at, o);
        x = better(x, y);
    }
    return x;
}

// Shared memory: one mbarrier per warp | keep table | the warps' stages.
//
// Tiles: a warp's first tile is tile number (its index among all warps); further tiles are
// claimed one at a time from counters in the workspace, so that SMs that run ahead take more and
// all finish together.  One counter could not keep up (atomics on one address retire about 190
// per microsecond; tiles of 16 KB are finished at twice that rate), so there are C of them, C
// the largest of 4, 3, 2, 1 that divides the warps per CTA: counter c hands out the tiles GW +
// c, GW + c + C, ... and serves warps c, c + C, ... of every CTA, so that all counters have the
// same number of tiles and of warps and run out together.  The claim for the tile after the
// current one is in flight while the current one is worked on.
template <typename T, int G, int kF>
__global__ void __launch_bounds__(512, 1) ctc_rows_tma(const CtcParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int ES = Elem<T>::kBytes, EPC = Elem<T>::kPerChunk;
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int W = p.warps, R = p.rows_per_tile;
    const int64_t gw = (int64_t)blockIdx.x + (int64_t)gridDim.x * warp, GW = (int64_t)gridDim.x * W;

    const uint32_t bar = smem_u32(smem) + warp * 8;
    const uint32_t tab_off = (uint32_t)((W * 8 + 15) & ~15);
    const uint32_t keep_tab = smem_u32(smem) + tab_off;
    const uint32_t stage_region = (tab_off + (uint32_t)(EPC * (EPC + 1)) * 16 + 127) & ~127u;
    const uint32_t stage = smem_u32(smem) + stage_region + (uint32_t)warp * p.stage_stride;
    unsigned char *stage_ptr = smem + stage_region + (size_t)warp * p.stage_stride;

    build_keep_table<T>(reinterpret_cast<uint4 *>(smem + tab_off), (int)threadIdx.x, (int)blockDim.x);
    if (lane == 0) {
        mbar_init(bar, 1);
        mbar_init_fence();
    }
    __syncthreads();                       // the keep table is shared by all warps
    if (gw >= p.num_tiles) return;

    const uintptr_t base = reinterpret_cast<uintptr_t>(p.logits);
    const int64_t row_pitch = p.ld * ES;

    // Brings tile t into this warp's stage.  The tile's rows are one contiguous byte range
    // (padding between rows included); the 16-byte-aligned superset of the range is fetched with
    // one bulk copy, except where that superset would leave the matrix (near its two ends):
    // there the copy is one chunk shorter and the few elements outside it are fetched with
    // plain loads.  Bytes of neighbouring rows that come along are never looked at.
    auto issue = [&](int64_t t) {
        const ranges::TileReads tr = ranges::tile_reads(base, p.total_bytes, row_pitch,
                                                        (int64_t)p.V * ES, p.N, R, t);
        if (tr.head_hi > tr.head_lo || tr.tail_hi > tr.tail_lo) {
            for (int side = 0; side < 2; ++side) {
                const uintptr_t lo = side ? tr.tail_lo : tr.head_lo, hi = side ? tr.tail_hi : tr.head_hi;
                for (uintptr_t a = lo + (uintptr_t)lane * ES; a < hi; a += 32 * ES) {
                    if (ES == 4) *reinterpret_cast<uint32_t *>(stage_ptr + (a - tr.f0)) =
                            *reinterpret_cast<const uint32_t *>(a);
                    else *reinterpret_cast<uint16_t *>(stage_ptr + (a - tr.f0)) =
                            *reinterpret_cast<const uint16_t *>(a);
                }
            }
            __syncwarp();
        }
        if (lane == 0) {
            if (tr.bulk_hi > tr.bulk_lo) {
                const uint32_t bytes = (uint32_t)(tr.bulk_hi - tr.bulk_lo);
                fence_proxy_async();
                mbar_arrive_expect_tx(bar, bytes);
                bulk_g2s(stage + (uint32_t)(tr.bulk_lo - tr.f0),
                         reinterpret_cast<const void *>(tr.bulk_lo), bytes, bar);
            } else {
                mbar_arrive(bar);
            }
        }
    };

    const bool dynamic = p.tile_counter != nullptr && p.num_tiles > GW;
    uint32_t epoch = p.epoch;
    const int C = p.counters;
    unsigned long long *counter = p.tile_counter + (warp % C) * 32;
    const int64_t first = GW + warp % C;                 // tile of this counter's slot 0
    bool failed = false, ok = true;
    uint32_t parity = 0;
    // this warp's tiles: t, t + step, ... up to (not including) t_end
    int64_t t = gw, t_end = gw + 1, step = 1;
    unsigned long long pend = 0;          // lane 0: the counter word before the claim in flight
    uint32_t pend_k = 0;
    auto claim_begin = [&]() {
        pend_k = p.claim;
        if (lane == 0) pend = tagged_begin(counter, epoch, pend_k);
    };
    pdl_wait();
    issue(t);
    if (dynamic) {
        // The tag of this launch's counter words: the host's call number plus the number of
        // launches the workspace has seen, so that a launch that is replayed with the same
        // parameters (a captured graph) does not take the counts of the replay before it for
        // its own.
        epoch = scratch_tag(epoch + (uint32_t)__ldcg(p.launch_gen));
        claim_begin();
    }
    while (t < p.num_tiles) {
        if (!mbar_wait_bounded(bar, parity)) { failed = true; break; }
        parity ^= 1u;
        const int64_t r0 = t * R;
        const int nrows = (int)min((int64_t)R, p.N - r0);
        const uint32_t head = (uint32_t)((base + (uintptr_t)(r0 * row_pitch)) & 15);
        reduce_tile<T, G, kF>(p, stage, keep_tab, head, r0, nrows, lane);
        __syncwarp();
        int64_t nt = dynamic ? t + step : t + GW;
        if (dynamic && nt >= t_end) {
            // the claimed tiles are used up: take the claim in flight, start the next one
            uint32_t cnt = 0;
            if (lane == 0) cnt = tagged_finish(counter, epoch, pend_k, pend, ok);
            cnt = __shfl_sync(0xffffffffu, cnt, 0);
            if (!__shfl_sync(0xffffffffu, (int)ok, 0)) { failed = true; break; }
            step = C;
            nt = first + (int64_t)cnt * C;
            t_end = nt + (int64_t)pend_k * C;
            if (nt < p.num_tiles) claim_begin();
        }
        if (nt < p.num_tiles) issue(nt);
        t = nt;
    }
    if (failed) {
        // A wait ran out, or the tile counter could not be read: poison the frames of the tiles
        // this warp still holds and of one more, unclaimed one, so that the per-utterance
        // kernel reports SSD_UTT_INTERNAL, then let copies that may be in flight land.
        for (; t < p.num_tiles && (!dynamic || t < t_end); t += dynamic ? step : GW) {
            const int64_t r0 = t * R;
            const int nrows = (int)min((int64_t)R, p.N - r0);
            for (int i = lane; i < nrows; i += 32) {
                p.frame_entropy[r0 + i] = __uint_as_float(kNanInternal);
                p.frame_argmax[r0 + i] = 0;
                if (p.frame_lse) p.frame_lse[r0 + i] = __uint_as_float(kNanInternal);
            }
        }
        if (dynamic) {
            // the claim in flight: its tiles are this warp's as well
            uint32_t cnt = 0xffffffffu;
            if (lane == 0 && (uint32_t)(pend >> 32) == epoch) cnt = (uint32_t)pend;
            cnt = __shfl_sync(0xffffffffu, cnt, 0);
            if (cnt != 0xffffffffu) {
                t = first + (int64_t)cnt * C;
                for (t_end = t + (int64_t)pend_k * C; t < p.num_tiles && t < t_end; t += C) {
                    const int64_t r0 = t * R;
                    const int nrows = (int)min((int64_t)R, p.N - r0);
                    for (int i = lane; i < nrows; i += 32) {
                        p.frame_entropy[r0 + i] = __uint_as_float(kNanInternal);
                        p.frame_argmax[r0 + i] = 0;
                        if (p.frame_lse) p.frame_lse[r0 + i] = __uint_as_float(kNanInternal);
                    }
                }
            } else if (lane == 0) {
                p.frame_entropy[0] = __uint_as_float(kNanInternal);   // the counter itself failed
            }
        }
        drain_after_error();
    }
}

template <typename T>
__global__ void __launch_bounds__(256) ctc_rows_plain(const CtcParams p) {
    constexpr int ES = Elem<T>::kBytes;
    pdl_enter();
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
// These kernels are chains of a few dependent memory round trips; a wide CTA takes an utterance
// of up to 1024 frames in one sweep, and the loads of a sweep are issued together.
constexpr int kUttThreads = 1024;

// Maximum over the block; valid in warp 0 (all its lanes).  One __syncthreads.
__device__ __forceinline__ MaxAt block_max_at(MaxAt x, MaxAt *scratch /* [32] shared */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    x = warp_max_at(x);
    if (lane == 0) scratch[warp] = x;
    __syncthreads();
    MaxAt r{0.f, -1};
    if (warp == 0) {
        if (lane < nw) r = scratch[lane];
        r = warp_max_at(r);
    }
    return r;
}

__global__ void __launch_bounds__(kUttThreads) collapse_kernel(
    const int32_t *__restrict__ frame_argmax, const float *__restrict__ frame_entropy,
    const int64_t *__restrict__ frame_off, int B, int64_t N, int blank_id, int cap,
    int32_t *__restrict__ draft_tokens, int32_t *__restrict__ draft_frames,
    int32_t *__restrict__ draft_len, int32_t *__restrict__ draft_full_len,
    float *__restrict__ utt_max_entropy, uint32_t *__restrict__ utt_status,
    unsigned long long *launch_gen) {
    __shared__ int warp_tot[2][32];
    __shared__ MaxAt scratch[32];
    __shared__ unsigned flags_sh[32];
    pdl_enter();
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nw = blockDim.x >> 5;
    // the frame statistics kernel before this one is through, the next one has not begun
    if (launch_gen && b == 0 && tid == 0) *launch_gen = *launch_gen + 1;
    const int64_t t0 = frame_off[b], t1 = frame_off[b + 1];
    if (t0 < 0 || t1 < t0 || t1 > N) {
        if (tid == 0) {
            draft_len[b] = 0; draft_full_len[b] = 0; utt_max_entropy[b] = 0.f;
            utt_status[b] = SSD_UTT_BAD_OFFSETS;
        }
        return;
    }
    const int64_t T = t1 - t0;
    int base = 0, buf = 0;
    MaxAt best{0.f, -1};
    unsigned myflags = 0;
    for (int64_t tile = 0; tile < T; tile += blockDim.x, buf ^= 1) {
        const int64_t t = tile + tid;
        const bool valid = t < T;
        int a = blank_id, prev0 = -1;
        float h = 0.f;
        if (valid) {
            a = frame_argmax[t0 + t];
            h = frame_entropy[t0 + t];
            if (lane == 0 && t > 0) prev0 = frame_argmax[t0 + t - 1];   // issued with the others
        }
        // the previous frame's symbol: the neighbouring lane has it, except for lane 0
        int prev = __shfl_up_sync(0xffffffffu, a, 1);
        if (lane == 0) prev = prev0;
        if (valid) {
            if (h != h) {
                myflags |= (__float_as_uint(h) == kNanInternal) ? SSD_UTT_INTERNAL : SSD_UTT_NONFINITE;
            } else {
                best = better(best, MaxAt{h, (int)t});
            }
        }
        const bool keep = valid && a != blank_id && (t == 0 || a != prev);
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
        const int prefix = __popc(bal & ((1u << lane) - 1));
        if (lane == 0) warp_tot[buf][warp] = __popc(bal);
        __syncthreads();                       // the other buffer is free again after this
        // every warp scans the (at most 32) warp totals by itself
        const int mine = lane < nw ? warp_tot[buf][lane] : 0;
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += y;
        }
        const int before = __shfl_sync(0xffffffffu, incl - mine, warp);
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        const int pos = base + before + prefix;
        if (keep && pos < cap) {
            draft_tokens[t0 + pos] = a;
            if (draft_frames) draft_frames[t0 + pos] = (int)t;
        }
        base += total;
    }
    myflags = __reduce_or_sync(0xffffffffu, myflags);
    if (lane == 0) flags_sh[warp] = myflags;
    best = block_max_at(best, scratch);        // __syncthreads inside: flags_sh visible after it
    if (warp == 0) {
        unsigned f = lane < nw ? flags_sh[lane] : 0u;
        f = __reduce_or_sync(0xffffffffu, f);
        if (lane == 0) {
            draft_full_len[b] = base;
            draft_len[b] = min(base, cap);
            utt_max_entropy[b] = best.at >= 0 ? best.v : 0.f;
            utt_status[b] = f;
        }
    }
}

__global__ void __launch_bounds__(kUttThreads) gate_kernel(
    const float *__restrict__ frame_entropy, const int64_t *__restrict__ frame_off, int B,
    int64_t N, float tau, uint8_t *__restrict__ gate_accept, float *__restrict__ max_entropy,
    int32_t *__restrict__ argmax_frame) {
    __shared__ MaxAt scratch[32];
    __shared__ int bad_sh[32];
    pdl_enter();
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nw = blockDim.x >> 5;
    const int64_t t0 = frame_off[b], t1 = frame_off[b + 1];
    if (t0 < 0 || t1 < t0 || t1 > N) {
        if (tid == 0) {
            gate_accept[b] = 0; max_entropy[b] = 0.f;
            if (argmax_frame) argmax_frame[b] = -1;
        }
        return;
    }
    const int64_t T = t1 - t0;
    MaxAt best{0.f, -1};
    int bad = 0;
    for (int64_t t = tid; t < T; t += blockDim.x) {
        const float h = frame_entropy[t0 + t];
        if (!(h < tau)) bad = 1;             // Eq. 3 is strict; NaN never passes
        if (h == h) best = better(best, MaxAt{h, (int)t});
    }
    bad = __any_sync(0xffffffffu, bad);
    if (lane == 0) bad_sh[warp] = bad;
    best = block_max_at(best, scratch);       // __syncthreads inside
    if (warp == 0) {
        const int any_bad = __any_sync(0xffffffffu, lane < nw ? bad_sh[lane] : 0);
        if (lane == 0) {
            const bool accept = (T == 0) ? (0.f < tau) : !any_bad;
            gate_accept[b] = accept ? 1 : 0;
            max_entropy[b] = best.at >= 0 ? best.v : 0.f;
            if (argmax_frame) argmax_frame[b] = best.at;
        }
    }
}

// Eq. 3 from per-utterance maxima that ssd_ctc_draft left behind: utterance b passes iff its
// largest frame entropy is below tau and no frame was NaN (status bits), its offsets were sound
// and no wait ran out.  An utterance without frames has maximum 0.
__global__ void __launch_bounds__(256) gate_from_maxima_kernel(
    const float *__restrict__ utt_max_entropy, const uint32_t *__restrict__ utt_status, int B,
    float tau, uint8_t *__restrict__ gate_accept, float *__restrict__ max_entropy) {
    pdl_enter();
    for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < B; b += gridDim.x * blockDim.x) {
        const float h = utt_max_entropy[b];
        const uint32_t st = utt_status[b];
        const bool sound = (st & (SSD_UTT_NONFINITE | SSD_UTT_BAD_OFFSETS | SSD_UTT_INTERNAL)) == 0;
        gate_accept[b] = (sound && h < tau) ? 1 : 0;
        max_entropy[b] = h;
    }
}

}  // namespace

unsigned long long next_epoch() {
    static unsigned long long counter = 0;
    unsigned long long c = __atomic_add_fetch(&counter, 1ull, __ATOMIC_RELAXED);
    return 0x55D0000000000000ull | (c & 0x0000ffffffffffffull);
}

// Kernel and launch shape of the frame-statistics pass for these sizes.
// G lanes share a row, a warp works on 32/G rows at a time (one pass), and a tile is a whole
// number of passes.  Few lanes per row spread the per-pass work (row geometry, masked first and
// last iterations, lane merges, logarithms, stores) over more rows; one pass of about 16 KB per
// warp and as many warps as shared memory holds keep both the copies and the arithmetic busy.
int plan_ctc(ssd_dtype dtype, int V, int64_t ld, int64_t N, int B, const ssd_launch_opts *o,
             CtcPlan *plan) {
    const int es = dtype == SSD_F32 ? 4 : 2;
    CtcPlan pl{};
    int kernel = o ? o->kernel : 0;
    const int64_t row_pitch = ld * es;
    const int64_t row_bytes = (int64_t)V * es;
    const int64_t chunks_max = (row_bytes + 31 - es) / 16;   // most 16-byte chunks a row touches
    const int64_t chunks_min = (row_bytes + 15) / 16;
    // lanes per row: the smallest power of two for which one pass (32/G rows) is at most 16.5 KB
    int G = 2;
    while (G < 32 && (32 / G) * row_pitch > 16896) G *= 2;
    if (o && o->split > 0) {
        G = o->split;
        if (G != 2 && G != 4 && G != 8 && G != 16 && G != 32) return SSD_ERR_ARG;
    }
    const int rpw = 32 / G;
    const int iters = (int)((chunks_max + G - 1) / G);
    // a forced G that makes a lane add up thousands of terms by itself costs accuracy: refused
    if (o && o->split > 0 && iters > 160 && G < 32) return SSD_ERR_ARG;
    int tail_from = (int)((chunks_min - 1) / G);
    if (tail_from < 1) tail_from = 1;
    (void)B;
    const int epc = 16 / es;
    const int64_t fixed = 16 * 8 + 16 + (int64_t)epc * (epc + 1) * 16 + 128;
    const int64_t stage_budget = 216 * 1024 - fixed;
    int warps = 0, R = 0;
    int64_t stage_stride = 0;
    if (kernel != 1 && row_pitch <= 2 * row_bytes + 64 && row_pitch < (1 << 20)) {
        int64_t groups = 8192 / (rpw * row_pitch);
        if (groups < 1) groups = 1;
        if (o && o->stage_bytes > 0) groups = (o->stage_bytes + rpw - 1) / rpw;
        for (; groups >= 1 && warps == 0; groups = groups > 1 ? groups / 2 : 0) {
            R = (int)(groups * rpw);
            // the last row's lanes read iters * G chunks from the row's first chunk on, whether
            // the row reaches that far or not (what lies past it is masked, not used)
            stage_stride = ((R - 1) * row_pitch + 16 + (int64_t)iters * G * 16 + 127) & ~127ll;
            int64_t w = stage_budget / stage_stride;
            if (w > 16) w = 16;      // 512 threads: 128 registers each, for eight chunks in flight
            if (w >= 5 && w % 2 && w % 3) --w;      // so that 2 or more tile counters divide it
            if (o && o->warps > 0 && o->warps < w) w = o->warps;
            if (w >= 1) warps = (int)w;
        }
    }
    if (warps == 0) {
        if (kernel == 2) return SSD_ERR_ARG;   // forced, but a pass does not fit a stage
        kernel = 1;
    } else {
        kernel = 2;
    }
    pl.kernel = kernel; pl.lanes_per_row = G; pl.rows_per_tile = R; pl.warps = warps;
    pl.stages = 1; pl.stage_stride = (int)stage_stride;
    pl.iters = iters; pl.tail_from = tail_from;
    pl.fma_exp = (o && o->fma_exp > 0 && dtype == SSD_BF16) ? (o->fma_exp > 2 ? 2 : o->fma_exp) : 0;
    pl.num_tiles = kernel != 1 ? (N + R - 1) / R : 0;
    pl.smem_bytes = kernel != 1
        ? (size_t)(((((warps * 8 + 15) & ~15) + epc * (epc + 1) * 16) + 127) & ~127) +
          (size_t)warps * stage_stride
        : 0;
    pl.workspace_bytes = 2048;      // the tile counters, 256 bytes apart, and room to spare
    *plan = pl;
    return SSD_OK;
}

namespace {
template <typename T, int kF> void (*pick_ctc(int G))(const CtcParams) {
    return G == 2 ? ctc_rows_tma<T, 2, kF> : G == 4 ? ctc_rows_tma<T, 4, kF>
         : G == 8 ? ctc_rows_tma<T, 8, kF> : G == 16 ? ctc_rows_tma<T, 16, kF>
                                                     : ctc_rows_tma<T, 32, kF>;
}
}  // namespace

// Frame statistics of all N rows.  workspace: 256 bytes for the tile counter, or NULL (tiles are
// then dealt out in a fixed order).
int launch_ctc_rows(const void *logits, ssd_dtype dtype, int V, int64_t ld, int64_t N,
                    float *frame_entropy, int32_t *frame_argmax, float *frame_lse,
                    float *frame_logprob, void *workspace, const CtcPlan &plan, const Launch &L) {
    if (N == 0) return SSD_OK;
    const ssd_launch_opts *o = L.opts;
    const int es = dtype == SSD_F32 ? 4 : 2;
    CtcParams p{};
    p.logits = static_cast<const char *>(logits);
    p.V = V; p.ld = ld; p.N = N;
    p.total_bytes = (N - 1) * ld * es + (int64_t)V * es;
    p.frame_entropy = frame_entropy; p.frame_argmax = frame_argmax; p.frame_lse = frame_lse;
    p.frame_logprob = frame_logprob;
    const int kernel = plan.kernel, G = plan.lanes_per_row, R = plan.rows_per_tile;
    cudaError_t e;
    if (o && o->ev_begin) {
        e = cudaEventRecord(static_cast<cudaEvent_t>(o->ev_begin), L.stream);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    }
    if (kernel != 1) {
        p.rows_per_tile = R; p.stages = 1; p.warps = plan.warps;
        p.stage_stride = plan.stage_stride;
        p.iters = plan.iters; p.tail_from = plan.tail_from;
        p.num_tiles = (N + R - 1) / R;
        // workspace: four counter words 256 bytes apart, then the launch count at byte 1024
        p.tile_counter = static_cast<unsigned long long *>(workspace);
        p.launch_gen = workspace ? static_cast<unsigned long long *>(workspace) + 128 : nullptr;
        p.epoch = (uint32_t)next_epoch();
        p.counters = plan.warps % 4 == 0 ? 4 : plan.warps % 3 == 0 ? 3 : plan.warps % 2 == 0 ? 2 : 1;
        // small tiles are finished faster than a counter hands them out one by one
        p.claim = (int64_t)R * ld * es * p.counters < 3 * 12288 ? 2 : 1;
        int64_t ctas = (p.num_tiles + plan.warps - 1) / plan.warps;
        const int sms = device_sm_count();
        if (sms <= 0) { record_cuda_error(cudaErrorNoDevice); return SSD_ERR_CUDA; }
        const int max_ctas = (o && o->ctas > 0) ? o->ctas : sms;
        if (ctas > max_ctas) ctas = max_ctas;
        void (*kern)(const CtcParams) = nullptr;
        if (dtype == SSD_F32) kern = pick_ctc<float, 0>(G);
        else kern = plan.fma_exp == 2 ? pick_ctc<bf16_t, 2>(G)
                  : plan.fma_exp == 1 ? pick_ctc<bf16_t, 1>(G) : pick_ctc<bf16_t, 0>(G);
        e = ensure_dynamic_smem(reinterpret_cast<const void *>(kern), plan.smem_bytes);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
        e = launch_pdl(kern, (unsigned)ctas, (unsigned)(plan.warps * 32), plan.smem_bytes,
                       L.stream, p);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    } else {
        int64_t ctas = (N + 7) / 8;
        const int sms = device_sm_count();
        if (sms <= 0) { record_cuda_error(cudaErrorNoDevice); return SSD_ERR_CUDA; }
        const int64_t cap = (o && o->ctas > 0) ? o->ctas : (int64_t)sms * 8;
        if (ctas > cap) ctas = cap;
        e = launch_pdl(dtype == SSD_F32 ? ctc_rows_plain<float> : ctc_rows_plain<bf16_t>,
                       (unsigned)ctas, 256u, 0, L.stream, p);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
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
                    void *workspace, cudaStream_t stream) {
    if (B == 0) return SSD_OK;
    unsigned long long *launch_gen =
        workspace ? static_cast<unsigned long long *>(workspace) + 128 : nullptr;
    cudaError_t e = launch_pdl(collapse_kernel, (unsigned)B, (unsigned)kUttThreads, 0, stream,
        frame_argmax, frame_entropy, frame_off, B, N, blank_id, max_draft_len, draft_tokens,
        draft_frames, draft_len, draft_full_len, utt_max_entropy, utt_status, launch_gen);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

int launch_gate_from_maxima(const float *utt_max_entropy, const uint32_t *utt_status, int B,
                            float tau, uint8_t *gate_accept, float *max_entropy,
                            cudaStream_t stream) {
    if (B == 0) return SSD_OK;
    const unsigned grid = (unsigned)((B + 255) / 256 < 8 ? (B + 255) / 256 : 8);
    cudaError_t e = launch_pdl(gate_from_maxima_kernel, grid, 256u, 0, stream, utt_max_entropy,
                               utt_status, B, tau, gate_accept, max_entropy);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

int launch_gate(const float *frame_entropy, const int64_t *frame_off, int B, int64_t N,
                float tau, uint8_t *gate_accept, float *max_entropy, int32_t *argmax_frame,
                cudaStream_t stream) {
    if (B == 0) return SSD_OK;
    cudaError_t e = launch_pdl(gate_kernel, (unsigned)B, (unsigned)kUttThreads, 0, stream,
                               frame_entropy, frame_off, B, N, tau, gate_accept, max_entropy,
                               argmax_frame);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

}  // namespace ssd
