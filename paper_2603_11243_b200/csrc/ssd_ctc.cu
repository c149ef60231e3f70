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
    float *frame_entropy;
    int32_t *frame_argmax;
    float *frame_lse;
    float *frame_logprob;
};

// Replaces the elements of a 16-byte chunk outside [e_lo, e_hi) (they belong to a neighbouring
// row, to the padding between rows, or were never written) by -inf, or, with kFinite, by a
// finite value near -1e30 whose exponential is 0 and whose product with that 0 is not NaN.
template <typename T, bool kFinite>
__device__ __forceinline__ void mask_chunk(uint4 &w, int e_lo, int e_hi);
template <bool kFinite> __device__ __forceinline__ void mask_f32(uint4 &w, int e_lo, int e_hi) {
    const uint32_t fill = kFinite ? 0xf149f2cau : 0xff800000u;
    if (0 < e_lo || 0 >= e_hi) w.x = fill;
    if (1 < e_lo || 1 >= e_hi) w.y = fill;
    if (2 < e_lo || 2 >= e_hi) w.z = fill;
    if (3 < e_lo || 3 >= e_hi) w.w = fill;
}
template <bool kFinite>
__device__ __forceinline__ uint32_t mask_pair(uint32_t v, int j, int e_lo, int e_hi) {
    const uint32_t fill = kFinite ? 0xf149u : 0xff80u;
    if (j < e_lo || j >= e_hi) v = (v & 0xffff0000u) | fill;
    if (j + 1 < e_lo || j + 1 >= e_hi) v = (v & 0x0000ffffu) | (fill << 16);
    return v;
}
template <bool kFinite> __device__ __forceinline__ void mask_bf16(uint4 &w, int e_lo, int e_hi) {
    w.x = mask_pair<kFinite>(w.x, 0, e_lo, e_hi);
    w.y = mask_pair<kFinite>(w.y, 2, e_lo, e_hi);
    w.z = mask_pair<kFinite>(w.z, 4, e_lo, e_hi);
    w.w = mask_pair<kFinite>(w.w, 6, e_lo, e_hi);
}
template <> __device__ __forceinline__ void mask_chunk<float, false>(uint4 &w, int a, int b) { mask_f32<false>(w, a, b); }
template <> __device__ __forceinline__ void mask_chunk<float, true>(uint4 &w, int a, int b) { mask_f32<true>(w, a, b); }
template <> __device__ __forceinline__ void mask_chunk<bf16_t, false>(uint4 &w, int a, int b) { mask_bf16<false>(w, a, b); }
template <> __device__ __forceinline__ void mask_chunk<bf16_t, true>(uint4 &w, int a, int b) { mask_bf16<true>(w, a, b); }

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
        if (c == cf || c == cl) mask_chunk<T, false>(w, c == cf ? e_lo : 0, c == cl ? e_hi : EPC);
        const float cm = chunk_max<T>(w);
        if (cm > vmax) { vmax = cm; vc = c; }
    }
    const float m = group_max<G>(vmax);
    int cand = INT_MAX;
    if (vc >= 0 && vmax == m) {
        uint4 w = lds128(stage_addr + (uint32_t)vc * 16);
        if (vc == cf || vc == cl) mask_chunk<T, false>(w, vc == cf ? e_lo : 0, vc == cl ? e_hi : EPC);
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
        if (c == cf || c == cl) mask_chunk<T, false>(w, c == cf ? e_lo : 0, c == cl ? e_hi : EPC);
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

// One chunk of the fused pass: running maximum (with the chunk it was first met in) and the
// sums S += 2^t, A += t*2^t with t = x*log2e - rh for a per-lane reference rh (in log2 units).
template <typename T>
__device__ __forceinline__ void fused_chunk(const uint4 &w, int c, float nrh, float &vmax, int &vc,
                                            float2 &Sa, float2 &Sb, float2 &Aa, float2 &Ab);
template <>
__device__ __forceinline__ void fused_chunk<float>(const uint4 &w, int c, float nrh, float &vmax,
                                                   int &vc, float2 &Sa, float2 &Sb, float2 &Aa,
                                                   float2 &Ab) {
    const float cm = chunk_max<float>(w);
    if (cm > vmax) { vmax = cm; vc = c; }
    entropy_pair(make_float2(__uint_as_float(w.x), __uint_as_float(w.y)), nrh, Sa, Aa);
    entropy_pair(make_float2(__uint_as_float(w.z), __uint_as_float(w.w)), nrh, Sb, Ab);
}
template <>
__device__ __forceinline__ void fused_chunk<bf16_t>(const uint4 &w, int c, float nrh, float &vmax,
                                                    int &vc, float2 &Sa, float2 &Sb, float2 &Aa,
                                                    float2 &Ab) {
    const float cm = chunk_max<bf16_t>(w);
    if (cm > vmax) { vmax = cm; vc = c; }
    entropy_pair(make_float2(bf16_lo(w.x), bf16_hi(w.x)), nrh, Sa, Aa);
    entropy_pair(make_float2(bf16_lo(w.y), bf16_hi(w.y)), nrh, Sb, Ab);
    entropy_pair(make_float2(bf16_lo(w.z), bf16_hi(w.z)), nrh, Sa, Aa);
    entropy_pair(make_float2(bf16_lo(w.w), bf16_hi(w.w)), nrh, Sb, Ab);
}

// Frame statistics of the rows of one tile that lies in shared memory.  G lanes share a row
// and a warp works on 32/G rows at a time.  A row is walked in the 16-byte chunks of the stage
// (whose alignment is that of global memory); its first and last chunk may also hold foreign
// elements, which are masked.
//
// Fused single pass: a lane takes the largest element of its first chunk as reference (rh =
// fl(ref*log2e), in log2 units) and, for every chunk, updates its running maximum and adds 2^t
// and t*2^t, t = x*log2e - rh (one fma).  fp32 keeps full relative precision whatever the
// reference, so the sums only have to stay in range; at the end the lanes' sums are re-based
// to mh = fl(m*log2e) of the row maximum m (S' = S*2^d, A' = (A + d*S)*2^d with d = rh - mh,
// an exact difference) and added; ml = m*log2e - mh (exact, by fma) is taken out of the
// log-sum-exp and cancels in the entropy.  One exponential per logit, and
// the comparisons overlap with the exponentials.  A group whose sums left the range or turned
// NaN (a logit far above the reference, masked -inf logits, NaN, +inf) is redone by the exact
// two-pass routine above.
template <typename T, int G>
__device__ __forceinline__ void reduce_tile(const CtcParams &p, uint32_t stage_addr, uint32_t head,
                                            int64_t r0, int nrows, int lane) {
    constexpr int ES = Elem<T>::kBytes, EPC = Elem<T>::kPerChunk, RPW = 32 / G;
    const int sub = lane % G, grp = lane / G;
    const uint32_t pitch = (uint32_t)(p.ld * ES), row_bytes = (uint32_t)p.V * ES;
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

        float vmax = -INFINITY, ref = 0.f;
        int vc = -1;
        float2 Sa = make_float2(0.f, 0.f), Sb = Sa, Aa = Sa, Ab = Sa;
        int c = cf + sub;
        if (c <= cl) {
            // first chunk of this lane (an edge chunk for some lanes): fixes the reference
            uint4 w = lds128(stage_addr + (uint32_t)c * 16);
            if (c == cf || c == cl) mask_chunk<T, true>(w, c == cf ? r.e_lo : 0, c == cl ? r.e_hi : EPC);
            const float cm = chunk_max<T>(w);
            if (cm > -INFINITY) ref = cm * kLog2e;
            fused_chunk<T>(w, c, -ref, vmax, vc, Sa, Sb, Aa, Ab);
            c += G;
#pragma unroll 2
            for (; c < cl; c += G) {           // interior chunks: no masks
                const uint4 wi = lds128(stage_addr + (uint32_t)c * 16);
                fused_chunk<T>(wi, c, -ref, vmax, vc, Sa, Sb, Aa, Ab);
            }
            if (c == cl) {                      // the row's last chunk
                uint4 wl = lds128(stage_addr + (uint32_t)c * 16);
                mask_chunk<T, true>(wl, 0, r.e_hi);
                fused_chunk<T>(wl, c, -ref, vmax, vc, Sa, Sb, Aa, Ab);
            }
        }
        const float Sl = (Sa.x + Sa.y) + (Sb.x + Sb.y), Al = (Aa.x + Aa.y) + (Ab.x + Ab.y);
        // out of range, NaN, or a lane that saw nothing above the mask fill value
        const bool bad = !(Sl < 1.0e30f) || Al != Al || (vc >= 0 && !(vmax > -1.0e29f));
        RowOut out;
        if (__any_sync(0xffffffffu, bad)) {
            out = reduce_row_exact<T, G>(stage_addr, r, sub);
        } else {
            const float m = group_max<G>(vmax);
            int cand = INT_MAX;
            if (vc >= 0 && vmax == m) {
                uint4 w = lds128(stage_addr + (uint32_t)vc * 16);
                if (vc == cf || vc == cl)
                    mask_chunk<T, true>(w, vc == cf ? r.e_lo : 0, vc == cl ? r.e_hi : EPC);
                float x[EPC];
                chunk_unpack<T>(w, x);
                int j = EPC - 1;
#pragma unroll
                for (int k = EPC - 2; k >= 0; --k) if (x[k] == m) j = k;
                cand = (vc - cf) * EPC + j - r.e_lo;
            }
            out.arg = group_min<G>(cand);
            if (out.arg == INT_MAX) out.arg = 0;
            const float mh = m * kLog2e;
            const float ml = fmaf(m, kLog2e, -mh);
            const float d = ref - mh;                    // <= 0; lanes without chunks have S = 0
            const float sc = ex2(d);
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
            for (int a = sub; a < p.V; a += G)
                o[a] = Elem<T>::load_shared(stage_addr + off + a * ES) - out.lse;
        }
    }
}

template <typename T, int G>
__global__ void __launch_bounds__(768, 1) ctc_rows_tma(const CtcParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int ES = Elem<T>::kBytes;
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int W = p.warps, S = p.stages, R = p.rows_per_tile;
    // Tile j goes to CTA j mod grid, and within the CTA to warp (j / grid) mod W: every CTA
    // gets the same number of tiles (give or take one) whatever the size of the matrix.
    const int64_t gw = (int64_t)blockIdx.x + (int64_t)gridDim.x * warp, GW = (int64_t)gridDim.x * W;
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
    const int64_t row_pitch = p.ld * ES;

    // Brings tile k of this warp into stage s.  The tile's rows are one contiguous byte range
    // (padding between rows included); the 16-byte-aligned superset of the range is fetched with
    // one bulk copy, except where that superset would leave the matrix (near its two ends):
    // there the copy is one chunk shorter and the few elements outside it are fetched with
    // plain loads.  Bytes of neighbouring rows that come along are never looked at.
    auto issue = [&](int64_t k, int s) {
        const ranges::TileReads t = ranges::tile_reads(base, p.total_bytes, row_pitch,
                                                       (int64_t)p.V * ES, p.N, R, gw + k * GW);
        const uint32_t bar = bar0 + s * 8;
        unsigned char *dst = stage0_ptr + (size_t)s * p.stage_stride;
        if (t.head_hi > t.head_lo || t.tail_hi > t.tail_lo) {
            for (int side = 0; side < 2; ++side) {
                const uintptr_t lo = side ? t.tail_lo : t.head_lo, hi = side ? t.tail_hi : t.head_hi;
                for (uintptr_t a = lo + (uintptr_t)lane * ES; a < hi; a += 32 * ES) {
                    if (ES == 4) *reinterpret_cast<uint32_t *>(dst + (a - t.f0)) =
                            *reinterpret_cast<const uint32_t *>(a);
                    else *reinterpret_cast<uint16_t *>(dst + (a - t.f0)) =
                            *reinterpret_cast<const uint16_t *>(a);
                }
            }
            __syncwarp();
        }
        if (lane == 0) {
            if (t.bulk_hi > t.bulk_lo) {
                const uint32_t bytes = (uint32_t)(t.bulk_hi - t.bulk_lo);
                fence_proxy_async();
                mbar_arrive_expect_tx(bar, bytes);
                bulk_g2s(stage0 + (uint32_t)s * p.stage_stride + (uint32_t)(t.bulk_lo - t.f0),
                         reinterpret_cast<const void *>(t.bulk_lo), bytes, bar);
            } else {
                mbar_arrive(bar);
            }
        }
    };

    pdl_wait();
    const int prologue = (int)min((int64_t)S, my_tiles);
    for (int k = 0; k < prologue; ++k) issue(k, k);

    bool failed = false;
    int s = 0;
    uint32_t parity = 0;
    int64_t k = 0;
    for (; k < my_tiles; ++k) {
        if (!mbar_wait_bounded(bar0 + s * 8, parity)) { failed = true; break; }
        const int64_t r0 = (gw + k * GW) * R;
        const int nrows = (int)min((int64_t)R, p.N - r0);
        const uint32_t head = (uint32_t)((base + (uintptr_t)(r0 * row_pitch)) & 15);
        reduce_tile<T, G>(p, stage0 + (uint32_t)s * p.stage_stride, head, r0, nrows, lane);
        __syncwarp();
        if (k + S < my_tiles) issue(k + S, s);
        if (++s == S) { s = 0; parity ^= 1u; }
    }
    if (failed) {
        // A wait ran out: poison every frame this warp still owed so that the per-utterance
        // kernel reports SSD_UTT_INTERNAL, then let copies that may be in flight land.
        for (; k < my_tiles; ++k) {
            const int64_t r0 = (gw + k * GW) * R;
            const int nrows = (int)min((int64_t)R, p.N - r0);
            for (int i = lane; i < nrows; i += 32) {
                p.frame_entropy[r0 + i] = __uint_as_float(kNanInternal);
                p.frame_argmax[r0 + i] = 0;
                if (p.frame_lse) p.frame_lse[r0 + i] = __uint_as_float(kNanInternal);
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
    float *__restrict__ utt_max_entropy, uint32_t *__restrict__ utt_status) {
    __shared__ int warp_tot[2][32];
    __shared__ MaxAt scratch[32];
    __shared__ unsigned flags_sh[32];
    pdl_enter();
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

// Kernel and launch shape of the frame-statistics pass for these sizes.
// G lanes share a row (so that a lane walks about 8..18 chunks of 16 bytes), a warp works on
// 32/G rows at a time, and a tile is a whole number of such row groups of about 8 KB.
int plan_ctc(ssd_dtype dtype, int V, int64_t ld, int64_t N, const ssd_launch_opts *o, CtcPlan *plan) {
    const int es = dtype == SSD_F32 ? 4 : 2;
    CtcPlan pl{};
    int kernel = o ? o->kernel : 0;
    const int64_t row_pitch = ld * es;
    const int64_t row_bytes = (int64_t)V * es;
    const int64_t chunks = (row_bytes + 15) / 16 + 1;
    const int G = chunks <= 72 ? 4 : chunks <= 144 ? 8 : chunks <= 288 ? 16 : 32;
    const int rpw = 32 / G;
    const int smem_budget = 200 * 1024;
    // One stage per warp and as many warps as fit hide the copy latency behind other warps'
    // arithmetic and give the schedulers more independent work than a deeper ring with fewer
    // warps does; a small matrix (a tile or two per warp) is better off prefetching.
    const int64_t tiles_guess = N * row_pitch / 8192 + 1;
    int warps = 0, R = 0;
    int stages = (o && o->stages > 0) ? o->stages : (tiles_guess < 2ll * 24 * sm_count() ? 2 : 1);
    if (stages < 1) stages = 1;
    if (stages > 8) stages = 8;
    int64_t stage_stride = 0;
    if (kernel != 1 && row_pitch <= 2 * row_bytes + 64 && row_pitch < (1 << 20)) {
        int64_t groups = 8192 / (rpw * row_pitch);
        if (groups < 1) groups = 1;
        if (o && o->stage_bytes > 0) groups = (o->stage_bytes + rpw - 1) / rpw;
        for (; groups >= 1 && warps == 0; groups = groups > 1 ? groups / 2 : 0) {
            R = (int)(groups * rpw);
            stage_stride = ((R - 1) * row_pitch + row_bytes + 32 + 127) & ~127ll;
            int64_t w = (smem_budget - 1024) / (stages * stage_stride);
            if (w > 24) w = 24;
            if (o && o->warps > 0 && o->warps < w) w = o->warps;
            if (w >= 1) warps = (int)w;
        }
    }
    if (warps == 0) {
        if (kernel == 2) return SSD_ERR_ARG;   // forced, but a row group does not fit a stage
        kernel = 1;
    } else {
        kernel = 2;
    }
    pl.kernel = kernel; pl.lanes_per_row = G; pl.rows_per_tile = R; pl.warps = warps;
    pl.stages = stages; pl.stage_stride = (int)stage_stride;
    pl.num_tiles = kernel == 2 ? (N + R - 1) / R : 0;
    *plan = pl;
    return SSD_OK;
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
    CtcPlan plan;
    const int prc = plan_ctc(dtype, V, ld, N, o, &plan);
    if (prc != SSD_OK) return prc;
    const int kernel = plan.kernel, G = plan.lanes_per_row, R = plan.rows_per_tile;
    const int warps = plan.warps, stages = plan.stages;
    const int64_t stage_stride = plan.stage_stride;
    cudaError_t e;
    if (o && o->ev_begin) {
        e = cudaEventRecord(static_cast<cudaEvent_t>(o->ev_begin), L.stream);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    }
    if (kernel == 2) {
        p.rows_per_tile = R; p.stages = stages; p.warps = warps;
        p.stage_stride = (int)stage_stride;
        p.num_tiles = (N + R - 1) / R;
        const size_t smem = (size_t)((warps * stages * 8 + 127) & ~127) +
                            (size_t)warps * stages * p.stage_stride;
        int64_t ctas = p.num_tiles;
        const int max_ctas = (o && o->ctas > 0) ? o->ctas : sm_count();
        if (ctas > max_ctas) ctas = max_ctas;
        void (*kern)(const CtcParams) = nullptr;
        if (dtype == SSD_F32)
            kern = G == 4 ? ctc_rows_tma<float, 4> : G == 8 ? ctc_rows_tma<float, 8>
                 : G == 16 ? ctc_rows_tma<float, 16> : ctc_rows_tma<float, 32>;
        else
            kern = G == 4 ? ctc_rows_tma<bf16_t, 4> : G == 8 ? ctc_rows_tma<bf16_t, 8>
                 : G == 16 ? ctc_rows_tma<bf16_t, 16> : ctc_rows_tma<bf16_t, 32>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
        e = launch_pdl(kern, (unsigned)ctas, (unsigned)(warps * 32), smem, L.stream, p);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    } else {
        int64_t ctas = (N + 7) / 8;
        const int64_t cap = (o && o->ctas > 0) ? o->ctas : (int64_t)sm_count() * 8;
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
                    cudaStream_t stream) {
    if (B == 0) return SSD_OK;
    cudaError_t e = launch_pdl(collapse_kernel, (unsigned)B, (unsigned)kUttThreads, 0, stream,
        frame_argmax, frame_entropy, frame_off, B, N, blank_id, max_draft_len, draft_tokens,
        draft_frames, draft_len, draft_full_len, utt_max_entropy, utt_status);
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
