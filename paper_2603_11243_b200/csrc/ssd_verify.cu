// Stage 2 kernels: vocabulary-wide log-sum-exp of the LLM logits at the draft positions, the
// draft token's log-likelihood (Eq. 5), and the first rejected position (Section 2.3).
//
// The LLM logits [M, V] are read once by a streaming kernel that leaves, for every row, a few
// partial (max, sum-of-exponentials) pairs in the workspace; a small per-utterance kernel merges
// them, gathers x[i, draft_i], applies the acceptance rule and finds the first reject.
//
//   verify_rows_tma    persistent CTAs; warp 0 is the producer: it walks this CTA's work items
//                      (a row, or a column span of a row), and feeds a ring of shared-memory
//                      stages with 1-D bulk asynchronous copies (TMA) signalled through
//                      mbarriers.  The other warps consume: each thread keeps a sum of
//                      2^((x-m)*log2e) relative to a reference logit m of its own and checks
//                      once per stage that the sum stayed in range (see Online), so the common
//                      case is one exponential and no comparison per logit.
//   verify_rows_plain  one CTA per item with scalar global loads; any alignment.  Fallback.
//
// The same streaming kernel with a running arg max serves the greedy decoding step (Eq. 6),
// and with a closing kernel that leaves (maximum, sum, draft logit) per row instead of the
// decision it serves an LLM head whose columns are split over several ranks (ssd_verify_shard,
// ssd_verify_combine).
#include <limits.h>
#include <math.h>

#include "ssd_common.cuh"
#include "ssd_ranges.cuh"
#include "ssd_stream.cuh"

namespace ssd {


namespace {

using namespace stream;

struct VerifyParams {
    const char *logits;
    int V;
    int64_t ld;
    int64_t M;
    int split;
    int64_t num_items;
    const int64_t *tok_off;
    int B;
    const uint8_t *skip;
    float2 *partials;
    int partials_per_row;
    int warps;            // consumer warps
    int stages;
    int stage_bytes;
    unsigned long long *err_word;
    unsigned long long epoch;
};

template <typename T, int kF, bool kArg>
__global__ void __launch_bounds__(544, 1) verify_rows_tma(const VerifyParams p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    constexpr int ES = Elem<T>::kBytes, EPC = Elem<T>::kPerChunk;
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int S = p.stages, CW = p.warps;
    // layout: full[S] | empty[S] | desc[S] | offsets cache | stages
    unsigned char *smem = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t full0 = sbase, empty0 = sbase + S * 8;
    StageDesc *desc = reinterpret_cast<StageDesc *>(smem + 2 * S * 8);
    const bool cache_off = p.skip != nullptr && p.B + 1 <= kOffCacheMax;
    int64_t *off_cache = reinterpret_cast<int64_t *>(smem + 2 * S * 8 + S * sizeof(StageDesc));
    const uint32_t hdr = (uint32_t)((2 * S * 8 + S * sizeof(StageDesc) +
                                     (cache_off ? (size_t)(p.B + 1) * 8 : 0) + 127) & ~(size_t)127);
    const uint32_t stage0 = sbase + hdr;
    unsigned char *stage0_ptr = smem + hdr;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full0 + s * 8, 1); mbar_init(empty0 + s * 8, CW); }
        mbar_init_fence();
    }
    pdl_wait();
    if (cache_off)
        for (int i = threadIdx.x; i <= p.B; i += blockDim.x) off_cache[i] = p.tok_off[i];
    __syncthreads();

    const int64_t row_bytes = (int64_t)p.V * ES;

    if (warp == 0) {
        // =============================== producer ===============================
        const int64_t *offs = cache_off ? off_cache : p.tok_off;
        int s = 0;                  // stage to fill next, and the phase of its barriers
        uint32_t ph = 0;
        bool failed = false;
        const int max_chunks = p.stage_bytes >> 4;
        for (int64_t k0 = 0; !failed; k0 += 32) {
            const int64_t first = (int64_t)blockIdx.x + k0 * gridDim.x;
            if (first >= p.num_items) break;
            const int64_t mine = first + (int64_t)lane * gridDim.x;
            const int64_t my_row = mine / p.split;
            bool active = mine < p.num_items;
            if (active && p.skip) {
                const int b = utterance_of_row(offs, p.B, my_row);
                active = !(b >= 0 && p.skip[b]);
            }
            unsigned todo = __ballot_sync(0xffffffffu, active);
            while (todo && !failed) {
                const int src = __ffs(todo) - 1;
                todo &= todo - 1;
                const int64_t row = __shfl_sync(0xffffffffu, my_row, src);
                const int sp = (int)(__shfl_sync(0xffffffffu, mine, src) - row * p.split);
                const ranges::RowGeom geom = ranges::row_geom(
                    reinterpret_cast<uintptr_t>(p.logits), row, p.ld * ES, row_bytes);
                const uintptr_t g0 = geom.g0, g1 = geom.g1, f0 = geom.f0;
                const ranges::SpanCut cut = ranges::span_cut(geom.row_chunks, p.split, sp, max_chunks);
                const int sc1 = cut.sc1, parts = cut.parts, per_part = cut.per_part;
                const int64_t slot = row * p.partials_per_row + (int64_t)sp * CW;
                for (int part = 0; part < parts; ++part) {
                    if (!mbar_wait_bounded(empty0 + s * 8, ph ^ 1u)) { failed = true; break; }
                    const int pc0 = cut.sc0 + part * per_part;
                    const int pc1 = min(sc1, pc0 + per_part);
                    // chunks that are only partly inside the row (row start / end not on a
                    // 16-byte boundary) are filled here with plain loads and -inf padding; the
                    // bulk copy takes the fully valid chunks only, so it never leaves the row.
                    const ranges::PartReads pr = ranges::part_reads(geom, pc0, pc1);
                    const int b0 = pr.b0, b1 = pr.b1;
                    unsigned char *dst = stage0_ptr + (size_t)s * p.stage_bytes;
                    if (pr.head_plain) {
                        if (lane < EPC) {
                            const uintptr_t a = f0 + (uintptr_t)lane * ES;
                            const bool ok = a >= g0 && a < g1;
                            if (ES == 4) reinterpret_cast<uint32_t *>(dst)[lane] =
                                ok ? *reinterpret_cast<const uint32_t *>(a) : 0xff800000u;
                            else reinterpret_cast<uint16_t *>(dst)[lane] =
                                ok ? *reinterpret_cast<const uint16_t *>(a) : (uint16_t)0xff80u;
                        }
                    }
                    if (pr.tail_plain) {
                        if (lane < EPC) {
                            const uintptr_t a = f0 + (uintptr_t)(pc1 - 1) * 16 + (uintptr_t)lane * ES;
                            const bool ok = a >= g0 && a < g1;
                            unsigned char *d = dst + (size_t)(pc1 - 1 - pc0) * 16;
                            if (ES == 4) reinterpret_cast<uint32_t *>(d)[lane] =
                                ok ? *reinterpret_cast<const uint32_t *>(a) : 0xff800000u;
                            else reinterpret_cast<uint16_t *>(d)[lane] =
                                ok ? *reinterpret_cast<const uint16_t *>(a) : (uint16_t)0xff80u;
                        }
                    }
                    __syncwarp();
                    if (lane == 0) {
                        desc[s].nchunks = pc1 - pc0;
                        desc[s].flags = (part == parts - 1) ? kFlagLast : 0u;
                        desc[s].slot = slot;
                        desc[s].elem0 = (int32_t)(((int64_t)pc0 * 16 - (int64_t)(g0 - f0)) / ES);
                        const uint32_t bar = full0 + s * 8;
                        if (b1 > b0) {
                            const uint32_t bytes = (uint32_t)(b1 - b0) << 4;
                            fence_proxy_async();
                            mbar_arrive_expect_tx(bar, bytes);
                            bulk_g2s(stage0 + (uint32_t)s * p.stage_bytes + ((uint32_t)(b0 - pc0) << 4),
                                     reinterpret_cast<const void *>(f0 + ((uintptr_t)b0 << 4)),
                                     bytes, bar);
                        } else {
                            mbar_arrive(bar);
                        }
                    }
                    __syncwarp();
                    if (++s == S) { s = 0; ph ^= 1u; }
                }
            }
        }
        if (!failed) {
            if (mbar_wait_bounded(empty0 + s * 8, ph ^ 1u)) {
                if (lane == 0) {
                    desc[s].nchunks = 0; desc[s].flags = kFlagEnd; desc[s].slot = 0;
                    mbar_arrive(full0 + s * 8);
                }
            } else {
                failed = true;
            }
        }
        if (failed) {
            if (lane == 0) atomicExch(p.err_word, p.epoch);
            drain_after_error();
        }
    } else {
        // =============================== consumers ===============================
        const int cw = warp - 1;
        const int ct = cw * 32 + lane, NT = CW * 32;
        Online st;
        st.reset();
        ArgTrack at;
        at.reset();
        bool failed = false;
        int s = 0;
        uint32_t ph = 0;
        for (;;) {
            if (!mbar_wait_bounded(full0 + s * 8, ph)) { failed = true; break; }
            const int n = desc[s].nchunks;
            const uint32_t flags = desc[s].flags;
            if (flags & kFlagEnd) break;
            consume_stage<T, kF, kArg>(stage0 + (uint32_t)s * p.stage_bytes, n, ct, NT, st,
                                       kArg ? desc[s].elem0 : 0, at);
            int64_t slot = 0;
            if (flags & kFlagLast) slot = desc[s].slot;
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + s * 8);
            if (flags & kFlagLast) {
                const float2 r = warp_merge(st);
                if (kArg) {
                    // warp arg max: largest value, lowest index among the lanes that hold it
                    const float vm = warp_max(at.vmax);
                    const int vi = __reduce_min_sync(0xffffffffu, at.vmax == vm ? at.vidx : INT_MAX);
                    if (lane == 0)
                        reinterpret_cast<float4 *>(p.partials)[slot + cw] =
                            make_float4(r.x, r.y, vm, __int_as_float(vi));
                    at.reset();
                } else {
                    if (lane == 0) p.partials[slot + cw] = r;
                }
                st.reset();
            }
            if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (failed) {
            if (lane == 0) atomicExch(p.err_word, p.epoch);
            drain_after_error();
        }
    }
}


// Merge of a row's P (reference, sum) pairs into (maximum, sum relative to it).
__device__ __forceinline__ float2 merge_partials(const float2 *pp, int P) {
    float Mx = kNegInit, S = 0.f;
    if ((P & 1) == 0 && P <= 16) {
        const float4 *p4 = reinterpret_cast<const float4 *>(pp);
        float4 v[8];
#pragma unroll
        for (int q = 0; q < 8; ++q)
            v[q] = q < P / 2 ? p4[q] : make_float4(kNegInit, 0.f, kNegInit, 0.f);
#pragma unroll
        for (int q = 0; q < 8; ++q) Mx = fmaxf(Mx, fmaxf(v[q].x, v[q].z));
#pragma unroll
        for (int q = 0; q < 8; ++q)
            S += v[q].y * ex2((v[q].x - Mx) * kLog2e) + v[q].w * ex2((v[q].z - Mx) * kLog2e);
    } else {
        for (int q = 0; q < P; ++q) Mx = fmaxf(Mx, pp[q].x);
        for (int q = 0; q < P; ++q) {
            const float2 v = pp[q];
            S += v.y * ex2((v.x - Mx) * kLog2e);
        }
    }
    return make_float2(Mx, S);
}

// Eq. 5 for one row, given its maximum Mx, ln of its sum of exponentials relative to Mx and the
// draft token's logit x: the log-likelihood, whether the position is rejected (p <= tau; NaN
// rejects; tau <= 0 rejects nothing, tau >= 1 everything), and the status bits the row raises.
struct RowDecision {
    float logp, lse;
    bool reject;
    uint32_t flags;
};
__device__ __forceinline__ RowDecision decide_row(float x, float Mx, float lnS, bool id_ok,
                                                  float log_tau, int reject_none, int reject_all) {
    RowDecision d;
    d.lse = Mx + lnS;
    d.flags = fabsf(d.lse) < INFINITY ? 0u : (uint32_t)SSD_UTT_NONFINITE;
    if (!id_ok) {
        d.flags |= SSD_UTT_BAD_DRAFT_ID;
        d.logp = -INFINITY;
        d.reject = true;
    } else {
        d.logp = (x - Mx) - lnS;      // not x - lse: keeps its accuracy when |x| is large
        d.reject = reject_none ? false : (reject_all || !(d.logp > log_tau));
    }
    return d;
}

// ---- verification finished inside the streaming kernel ----------------------------------------
// The same ring of stages as verify_rows_tma, for whole rows (no column spans).  The consumer
// warps leave a row's (reference, sum) pairs in shared memory instead of the workspace; the
// producer warp, when it next takes over the stage that held the row's last part and has the
// stage's next copy under way, merges them, adds the draft token's logit (which it fetched,
// with the draft id, one batch of rows ahead), writes the row's log-likelihood (Eq. 5) and, for
// a rejected position, lowers the utterance's first-reject word in the workspace.  The CTA that
// finishes last turns those words into accepted_len / all_accepted / utt_status (Section 2.3).
// The words are {epoch : 32 | value : 32}: nothing has to be cleared between calls.
struct FinParams {
    VerifyParams v;
    const int32_t *draft_ids;
    float log_tau;
    int reject_none, reject_all;
    float *token_logp, *row_lse;
    int32_t *accepted_len;
    uint8_t *all_accepted;
    uint32_t *utt_status;
    unsigned long long *utt_words;     // [2 * B]: first rejected position, status bits
    unsigned long long *done_ctas;
    uint32_t epoch32;
};

struct FinRow {
    int64_t row;
    int32_t b, pos, id_ok;
    float x;
};

__device__ __forceinline__ void utterance_outputs(int b, int64_t i0, int64_t i1, int64_t M,
                                                  bool skipped, int first, uint32_t flags,
                                                  uint32_t internal, int32_t *accepted_len,
                                                  uint8_t *all_accepted, uint32_t *utt_status) {
    if (i0 < 0 || i1 < i0 || i1 > M) {
        accepted_len[b] = 0; all_accepted[b] = 0;
        utt_status[b] = SSD_UTT_BAD_OFFSETS | internal;
        return;
    }
    const int64_t K64 = i1 - i0;
    const int K = K64 > 0x7fffffff ? 0x7fffffff : (int)K64;
    if (skipped) { accepted_len[b] = K; all_accepted[b] = 1; utt_status[b] = internal; return; }
    first = first < K ? first : K;
    accepted_len[b] = first;
    all_accepted[b] = first == K ? 1 : 0;
    utt_status[b] = flags | internal;
}

template <typename T, int kF>
__global__ void __launch_bounds__(544, 1) verify_rows_fin(const FinParams q) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    constexpr int ES = Elem<T>::kBytes, EPC = Elem<T>::kPerChunk;
    __shared__ int s_last;
    const VerifyParams &p = q.v;
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int S = p.stages, CW = p.warps, NR = 2 * S;
    // layout: full[S] | empty[S] | desc[S] | rows[NR] | spart[NR*CW] | pending[S] | offsets | stages
    unsigned char *smem = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t full0 = sbase, empty0 = sbase + S * 8;
    size_t o = 2 * (size_t)S * 8;
    StageDesc *desc = reinterpret_cast<StageDesc *>(smem + o);     o += S * sizeof(StageDesc);
    FinRow *rows = reinterpret_cast<FinRow *>(smem + o);           o += NR * sizeof(FinRow);
    float2 *spart = reinterpret_cast<float2 *>(smem + o);          o += (size_t)NR * CW * 8;
    int32_t *pending = reinterpret_cast<int32_t *>(smem + o);      o += S * 4;
    o = (o + 7) & ~(size_t)7;
    int64_t *offs = reinterpret_cast<int64_t *>(smem + o);         o += (size_t)(p.B + 1) * 8;
    const uint32_t hdr = (uint32_t)((o + 127) & ~(size_t)127);
    const uint32_t stage0 = sbase + hdr;
    unsigned char *stage0_ptr = smem + hdr;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full0 + s * 8, 1);
            mbar_init(empty0 + s * 8, CW);
            pending[s] = 0;
        }
        mbar_init_fence();
        s_last = 0;
    }
    pdl_wait();
    for (int i = threadIdx.x; i <= p.B; i += blockDim.x) offs[i] = p.tok_off[i];
    __syncthreads();

    const int64_t row_bytes = (int64_t)p.V * ES;
    bool failed = false;

    if (warp == 0) {
        // =============================== producer ===============================
        int s = 0;
        uint32_t ph = 0;
        int rowseq = 0;
        bool ok = true;
        const int max_chunks = p.stage_bytes >> 4;

        auto finalize = [&](int slot1) {
            if (slot1 == 0) return;
            const int slot = slot1 - 1;
            const float2 v = lane < CW ? spart[slot * CW + lane] : make_float2(kNegInit, 0.f);
            const float Mx = fmaxf(warp_max(v.x), kNegInit);
            const float Ssum = warp_sum(v.y * ex2((v.x - Mx) * kLog2e));
            if (lane == 0) {
                const FinRow rm = rows[slot];
                const RowDecision d = decide_row(rm.x, Mx, logf(Ssum), rm.id_ok != 0, q.log_tau,
                                                 q.reject_none, q.reject_all);
                const float logp = d.logp, lse = d.lse;
                const uint32_t fl = d.flags;
                const bool reject = d.reject;
                q.token_logp[rm.row] = logp;
                if (q.row_lse) q.row_lse[rm.row] = lse;
                if (fl) tagged_or(q.utt_words + 2 * rm.b + 1, q.epoch32, fl, ok);
                if (reject) tagged_min(q.utt_words + 2 * rm.b, q.epoch32, (uint32_t)rm.pos, ok);
            }
            __syncwarp();
        };

        // What a lane knows about its row of a batch of 32 rows (row first + lane * grid): the
        // utterance, the position, the draft id and the draft token's logit.  Loaded one batch
        // ahead, so that nothing here waits for memory.
        struct Mine { int64_t row; int b, pos, id; float x; bool active; };
        auto look_up = [&](int64_t k0) {
            Mine m{0, 0, 0, -1, 0.f, false};
            m.row = (int64_t)blockIdx.x + (k0 + lane) * gridDim.x;
            if (m.row < p.M) {
                m.b = utterance_of_row(offs, p.B, m.row);
                if (m.b >= 0) {
                    const int64_t i0 = offs[m.b], i1 = offs[m.b + 1];
                    m.active = i0 >= 0 && i1 <= p.M && m.row >= i0 && m.row < i1 &&
                               i1 - i0 <= 0x7fffffff && !(p.skip && p.skip[m.b]);
                    if (m.active) {
                        m.pos = (int)(m.row - i0);
                        m.id = q.draft_ids[m.row];
                        if (m.id >= 0 && m.id < p.V)
                            m.x = Elem<T>::load(p.logits + (m.row * p.ld + m.id) * ES);
                    }
                }
            }
            return m;
        };
        Mine next = look_up(0);
        for (int64_t k0 = 0; !failed; k0 += 32) {
            if ((int64_t)blockIdx.x + k0 * gridDim.x >= p.M) break;
            const Mine cur = next;
            next = look_up(k0 + 32);
            unsigned todo = __ballot_sync(0xffffffffu, cur.active);
            while (todo && !failed) {
                const int src = __ffs(todo) - 1;
                todo &= todo - 1;
                const int64_t row = __shfl_sync(0xffffffffu, cur.row, src);
                const int rslot = rowseq % NR;
                ++rowseq;
                const ranges::RowGeom geom = ranges::row_geom(
                    reinterpret_cast<uintptr_t>(p.logits), row, p.ld * ES, row_bytes);
                const uintptr_t g0 = geom.g0, g1 = geom.g1, f0 = geom.f0;
                const ranges::SpanCut cut = ranges::span_cut(geom.row_chunks, 1, 0, max_chunks);
                const int parts = cut.parts, per_part = cut.per_part;
                for (int part = 0; part < parts; ++part) {
                    if (!mbar_wait_bounded(empty0 + s * 8, ph ^ 1u)) { failed = true; break; }
                    const int done_slot1 = pending[s];     // the row this stage held last, if any
                    __syncwarp();
                    const int pc0 = part * per_part;
                    const int pc1 = min(geom.row_chunks, pc0 + per_part);
                    const ranges::PartReads pr = ranges::part_reads(geom, pc0, pc1);
                    const int b0 = pr.b0, b1 = pr.b1;
                    unsigned char *dst = stage0_ptr + (size_t)s * p.stage_bytes;
                    if (pr.head_plain) {
                        if (lane < EPC) {
                            const uintptr_t a = f0 + (uintptr_t)lane * ES;
                            const bool in = a >= g0 && a < g1;
                            if (ES == 4) reinterpret_cast<uint32_t *>(dst)[lane] =
                                in ? *reinterpret_cast<const uint32_t *>(a) : 0xff800000u;
                            else reinterpret_cast<uint16_t *>(dst)[lane] =
                                in ? *reinterpret_cast<const uint16_t *>(a) : (uint16_t)0xff80u;
                        }
                    }
                    if (pr.tail_plain) {
                        if (lane < EPC) {
                            const uintptr_t a = f0 + (uintptr_t)(pc1 - 1) * 16 + (uintptr_t)lane * ES;
                            const bool in = a >= g0 && a < g1;
                            unsigned char *d = dst + (size_t)(pc1 - 1 - pc0) * 16;
                            if (ES == 4) reinterpret_cast<uint32_t *>(d)[lane] =
                                in ? *reinterpret_cast<const uint32_t *>(a) : 0xff800000u;
                            else reinterpret_cast<uint16_t *>(d)[lane] =
                                in ? *reinterpret_cast<const uint16_t *>(a) : (uint16_t)0xff80u;
                        }
                    }
                    __syncwarp();
                    if (lane == 0) {
                        const bool last = part == parts - 1;
                        desc[s].nchunks = pc1 - pc0;
                        desc[s].flags = last ? kFlagLast : 0u;
                        desc[s].slot = rslot;
                        desc[s].elem0 = 0;
                        desc[s].gather = -1;
                        pending[s] = last ? rslot + 1 : 0;
                        const uint32_t bar = full0 + s * 8;
                        if (b1 > b0) {
                            const uint32_t bytes = (uint32_t)(b1 - b0) << 4;
                            fence_proxy_async();
                            mbar_arrive_expect_tx(bar, bytes);
                            bulk_g2s(stage0 + (uint32_t)s * p.stage_bytes + ((uint32_t)(b0 - pc0) << 4),
                                     reinterpret_cast<const void *>(f0 + ((uintptr_t)b0 << 4)),
                                     bytes, bar);
                        } else {
                            mbar_arrive(bar);
                        }
                    }
                    __syncwarp();
                    finalize(done_slot1);     // after the stage's next copy is under way
                    if (++s == S) { s = 0; ph ^= 1u; }
                }
                // what the row's finish needs; written after its copies are under way, since the
                // draft id and logit of a kernel's first rows may still be on their way
                if (lane == src) {
                    FinRow rm;
                    rm.row = cur.row; rm.b = cur.b; rm.pos = cur.pos;
                    rm.id_ok = (cur.id >= 0 && cur.id < p.V) ? 1 : 0; rm.x = cur.x;
                    rows[rslot] = rm;
                }
                __syncwarp();
            }
        }
        if (!failed) {
            // end marker into the next stage, then the rows still waiting in the other stages
            if (mbar_wait_bounded(empty0 + s * 8, ph ^ 1u)) {
                finalize(pending[s]);
                if (lane == 0) {
                    desc[s].nchunks = 0; desc[s].flags = kFlagEnd; desc[s].slot = 0; desc[s].gather = -1;
                    mbar_arrive(full0 + s * 8);
                }
                for (int t = 1; t < S && !failed; ++t) {
                    const int st = (s + t) % S;
                    const uint32_t par = st > s ? (ph ^ 1u) : ph;     // filled last round / this round
                    if (mbar_wait_bounded(empty0 + st * 8, par)) finalize(pending[st]);
                    else failed = true;
                }
            } else {
                failed = true;
            }
        }
        if (!__shfl_sync(0xffffffffu, (int)ok, 0)) failed = true;
        if (failed) {
            if (lane == 0) atomicExch(p.err_word, p.epoch);
            drain_after_error();
        }
    } else {
        // =============================== consumers ===============================
        const int cw = warp - 1;
        const int ct = cw * 32 + lane, NT = CW * 32;
        Online st;
        st.reset();
        ArgTrack unused;
        unused.reset();
        int s = 0;
        uint32_t ph = 0;
        for (;;) {
            if (!mbar_wait_bounded(full0 + s * 8, ph)) { failed = true; break; }
            const int n = desc[s].nchunks;
            const uint32_t flags = desc[s].flags;
            if (flags & kFlagEnd) break;
            consume_stage<T, kF, false>(stage0 + (uint32_t)s * p.stage_bytes, n, ct, NT, st, 0, unused);
            if (flags & kFlagLast) {
                const int slot = (int)desc[s].slot;
                const float2 r = warp_merge(st);
                if (lane == 0) spart[slot * CW + cw] = r;
                st.reset();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + s * 8);      // releases the write above as well
            if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (failed) {
            if (lane == 0) atomicExch(p.err_word, p.epoch);
            drain_after_error();
        }
    }

    // ---- the CTA that finishes last writes the per-utterance outputs --------------------------
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        bool ok2 = true;
        const uint32_t before = tagged_add(q.done_ctas, q.epoch32, 1u, ok2);
        s_last = ok2 && before + 1 == gridDim.x;
        if (!ok2) atomicExch(p.err_word, p.epoch);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const uint32_t internal = (__ldcg(p.err_word) == p.epoch) ? (uint32_t)SSD_UTT_INTERNAL : 0u;
    for (int b = threadIdx.x; b < p.B; b += blockDim.x) {
        const unsigned long long w0 = __ldcg(q.utt_words + 2 * b), w1 = __ldcg(q.utt_words + 2 * b + 1);
        const int first = (uint32_t)(w0 >> 32) == q.epoch32 ? (int)min((uint32_t)w0, 0x7fffffffu)
                                                            : 0x7fffffff;
        const uint32_t fl = (uint32_t)(w1 >> 32) == q.epoch32 ? (uint32_t)w1 : 0u;
        utterance_outputs(b, offs[b], offs[b + 1], p.M, p.skip && p.skip[b], first, fl, internal,
                          q.accepted_len, q.all_accepted, q.utt_status);
    }
}

template <typename T>
__global__ void __launch_bounds__(256) verify_rows_plain(const VerifyParams p) {
    constexpr int ES = Elem<T>::kBytes;
    pdl_enter();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    for (int64_t item = blockIdx.x; item < p.num_items; item += gridDim.x) {
        const int64_t row = item / p.split;
        const int sp = (int)(item - row * p.split);
        if (p.skip) {
            const int b = utterance_of_row(p.tok_off, p.B, row);
            if (b >= 0 && p.skip[b]) continue;
        }
        const int per = (p.V + p.split - 1) / p.split;
        const int v0 = min(p.V, sp * per), v1 = min(p.V, v0 + per);
        const char *rp = p.logits + row * p.ld * ES;
        float m = kNegInit, S = 0.f;
        for (int a = v0 + threadIdx.x; a < v1; a += blockDim.x) {
            const float x = Elem<T>::load(rp + (size_t)a * ES);
            if (x > m) { S = S * expf(m - x) + 1.f; m = x; }
            else S += expf(x - m);
        }
        const float Mw = warp_max(m);
        const float Sw = warp_sum(S * expf(m - Mw));
        if (lane == 0) p.partials[row * p.partials_per_row + (int64_t)sp * nw + warp] =
            make_float2(Mw, Sw);
    }
}

constexpr int kFinishThreads = 1024;   // one sweep for drafts of up to 1024 tokens

template <typename T>
__global__ void __launch_bounds__(kFinishThreads) verify_finish_kernel(
    const char *__restrict__ logits, int V, int64_t ld, int64_t M,
    const int64_t *__restrict__ tok_off, const int32_t *__restrict__ draft_ids, int B,
    float log_tau, int reject_none, int reject_all, const uint8_t *__restrict__ skip,
    const float2 *__restrict__ partials, int P, float *__restrict__ token_logp,
    float *__restrict__ row_lse, int32_t *__restrict__ accepted_len,
    uint8_t *__restrict__ all_accepted, uint32_t *__restrict__ utt_status,
    const unsigned long long *err_word, unsigned long long epoch) {
    constexpr int ES = Elem<T>::kBytes;
    __shared__ int first_reject;
    __shared__ unsigned flags;
    pdl_enter();
    // The kernel is a chain of dependent memory round trips, so the loads of each level are
    // issued together: offsets, skip flag and error word; then a row's draft id and its
    // partials; then the draft token's logit.
    const int b = blockIdx.x, tid = threadIdx.x;
    const int64_t i0 = tok_off[b], i1 = tok_off[b + 1];
    const unsigned long long err = *err_word;
    const bool skipped = skip != nullptr && skip[b] != 0;
    const uint32_t internal = (err == epoch) ? (uint32_t)SSD_UTT_INTERNAL : 0u;
    if (i0 < 0 || i1 < i0 || i1 > M) {
        if (tid == 0) {
            accepted_len[b] = 0; all_accepted[b] = 0;
            utt_status[b] = SSD_UTT_BAD_OFFSETS | internal;
        }
        return;
    }
    const int64_t K64 = i1 - i0;
    const int K = K64 > 0x7fffffff ? 0x7fffffff : (int)K64;
    if (skipped) {
        if (tid == 0) { accepted_len[b] = K; all_accepted[b] = 1; utt_status[b] = internal; }
        return;
    }
    if (tid == 0) { first_reject = K; flags = 0; }
    __syncthreads();
    unsigned myflags = 0;
    int myfirst = K;
    for (int i = tid; i < K; i += blockDim.x) {
        const int64_t r = i0 + i;
        const int id = draft_ids[r];
        const bool id_ok = id >= 0 && id < V;
        // the row's partials and the draft token's logit are fetched together
        float x = 0.f;
        if (id_ok) x = Elem<T>::load(logits + (r * ld + id) * ES);
        const float2 ms = merge_partials(partials + r * P, P);
        const RowDecision d = decide_row(x, ms.x, logf(ms.y), id_ok, log_tau, reject_none, reject_all);
        myflags |= d.flags;
        token_logp[r] = d.logp;
        if (row_lse) row_lse[r] = d.lse;
        const bool reject = d.reject;
        if (reject && i < myfirst) myfirst = i;
    }
    if (myfirst < K) atomicMin(&first_reject, myfirst);
    if (myflags) atomicOr(&flags, myflags);
    __syncthreads();
    if (tid == 0) {
        accepted_len[b] = first_reject;
        all_accepted[b] = first_reject == K ? 1 : 0;
        utt_status[b] = flags | internal;
    }
}

constexpr uint32_t kStatsInternal = 0x7fc0dead;   // in place of a row's maximum: a wait ran out

// Vocabulary-parallel verification, per rank: for every row of a verified utterance the
// triple (maximum of the local columns, sum of exponentials relative to it, logit of the draft
// token if its column is local, else -inf).  Rows of skipped or malformed utterances are left
// untouched; the combining kernel does not read them.
template <typename T>
__global__ void __launch_bounds__(kFinishThreads) shard_finish_kernel(
    const char *__restrict__ logits, int V_local, int64_t ld, int64_t M, int64_t col0,
    const int64_t *__restrict__ tok_off, const int32_t *__restrict__ draft_ids, int B,
    const uint8_t *__restrict__ skip, const float2 *__restrict__ partials, int P,
    float *__restrict__ stats, const unsigned long long *err_word, unsigned long long epoch) {
    constexpr int ES = Elem<T>::kBytes;
    pdl_enter();
    const int b = blockIdx.x, tid = threadIdx.x;
    const int64_t i0 = tok_off[b], i1 = tok_off[b + 1];
    const unsigned long long err = *err_word;
    const bool skipped = skip != nullptr && skip[b] != 0;
    if (i0 < 0 || i1 < i0 || i1 > M || skipped) return;
    const bool internal = err == epoch;
    for (int64_t r = i0 + tid; r < i1; r += blockDim.x) {
        const int64_t local = (int64_t)draft_ids[r] - col0;
        const bool owned = local >= 0 && local < V_local;
        float x = -INFINITY;
        if (owned) x = Elem<T>::load(logits + (r * ld + local) * ES);
        const float2 ms = merge_partials(partials + r * P, P);
        stats[3 * r + 0] = internal ? __uint_as_float(kStatsInternal) : ms.x;
        stats[3 * r + 1] = ms.y;
        stats[3 * r + 2] = x;
    }
}

// Vocabulary-parallel verification, after the exchange: stats_all holds R ranks' triples,
// [R, M, 3].  Per row the global maximum, the sum re-based to it, the draft token's logit (the
// one shard that owns the column has it), then Eq. 5 and the first reject exactly as in
// verify_finish_kernel.
__global__ void __launch_bounds__(kFinishThreads) combine_kernel(
    const float *__restrict__ stats_all, int R, int64_t V_total, int64_t M,
    const int64_t *__restrict__ tok_off, const int32_t *__restrict__ draft_ids, int B,
    float log_tau, int reject_none, int reject_all, const uint8_t *__restrict__ skip,
    float *__restrict__ token_logp, float *__restrict__ row_lse,
    int32_t *__restrict__ accepted_len, uint8_t *__restrict__ all_accepted,
    uint32_t *__restrict__ utt_status) {
    __shared__ int first_reject;
    __shared__ unsigned flags;
    pdl_enter();
    const int b = blockIdx.x, tid = threadIdx.x;
    const int64_t i0 = tok_off[b], i1 = tok_off[b + 1];
    const bool skipped = skip != nullptr && skip[b] != 0;
    if (i0 < 0 || i1 < i0 || i1 > M) {
        if (tid == 0) { accepted_len[b] = 0; all_accepted[b] = 0; utt_status[b] = SSD_UTT_BAD_OFFSETS; }
        return;
    }
    const int64_t K64 = i1 - i0;
    const int K = K64 > 0x7fffffff ? 0x7fffffff : (int)K64;
    if (skipped) {
        if (tid == 0) { accepted_len[b] = K; all_accepted[b] = 1; utt_status[b] = 0; }
        return;
    }
    if (tid == 0) { first_reject = K; flags = 0; }
    __syncthreads();
    unsigned myflags = 0;
    int myfirst = K;
    for (int i = tid; i < K; i += blockDim.x) {
        const int64_t r = i0 + i;
        const int id = draft_ids[r];
        const bool id_ok = id >= 0 && (int64_t)id < V_total;
        float Mx = kNegInit, x = -INFINITY;
        for (int q = 0; q < R; ++q) {
            const float *t = stats_all + ((int64_t)q * M + r) * 3;
            const float m = t[0];
            if (__float_as_uint(m) == kStatsInternal) myflags |= SSD_UTT_INTERNAL;
            Mx = fmaxf(Mx, m);
            x = fmaxf(x, t[2]);
        }
        float S = 0.f;
        for (int q = 0; q < R; ++q) {
            const float *t = stats_all + ((int64_t)q * M + r) * 3;
            S += t[1] * ex2((t[0] - Mx) * kLog2e);
        }
        const RowDecision d = decide_row(x, Mx, logf(S), id_ok, log_tau, reject_none, reject_all);
        myflags |= d.flags;
        token_logp[r] = d.logp;
        if (row_lse) row_lse[r] = d.lse;
        const bool reject = d.reject;
        if (reject && i < myfirst) myfirst = i;
    }
    if (myfirst < K) atomicMin(&first_reject, myfirst);
    if (myflags) atomicOr(&flags, myflags);
    __syncthreads();
    if (tid == 0) {
        accepted_len[b] = first_reject;
        all_accepted[b] = first_reject == K ? 1 : 0;
        utt_status[b] = flags;
    }
}

// Greedy step: merges the partials of a row, one warp per row.  A partial is
// (reference, sum, largest logit, index of its first occurrence).
constexpr int kGreedyWarps = 8;
__global__ void __launch_bounds__(kGreedyWarps * 32) greedy_finish_kernel(
    int V, int64_t R, const float4 *__restrict__ partials, int P, int32_t *__restrict__ next_token,
    float *__restrict__ next_logp, float *__restrict__ row_lse, uint32_t *__restrict__ row_status,
    const unsigned long long *err_word, unsigned long long epoch) {
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const int64_t r = (int64_t)blockIdx.x * kGreedyWarps + (threadIdx.x >> 5);
    if (r >= R) return;
    const float4 *pp = partials + r * P;
    float Mx = kNegInit, vm = -INFINITY;
    for (int q = lane; q < P; q += 32) {
        const float4 v = pp[q];
        Mx = fmaxf(Mx, v.x);
        vm = fmaxf(vm, v.z);
    }
    Mx = warp_max(Mx);
    vm = warp_max(vm);
    float S = 0.f;
    int vi = INT_MAX;
    for (int q = lane; q < P; q += 32) {
        const float4 v = pp[q];
        S += v.y * ex2((v.x - Mx) * kLog2e);
        if (v.z == vm) vi = min(vi, __float_as_int(v.w));
    }
    S = warp_sum(S);
    vi = __reduce_min_sync(0xffffffffu, vi);
    if (lane == 0) {
        const float lnS = logf(S);
        const float lse = Mx + lnS;
        uint32_t st = (*err_word == epoch) ? (uint32_t)SSD_UTT_INTERNAL : 0u;
        if (!(fabsf(lse) < INFINITY)) st |= SSD_UTT_NONFINITE;
        next_token[r] = (vi < 0 || vi >= V) ? 0 : vi;
        if (next_logp) next_logp[r] = (vm - Mx) - lnS;
        if (row_lse) row_lse[r] = lse;
        if (row_status) row_status[r] = st;
    }
}

}  // namespace

unsigned long long next_epoch();

// Workspace: [0,256) header (error word, finished-CTA counter), two words per utterance, then
// M * partials float2.
int plan_verify(int B, int64_t M, int V, ssd_dtype dtype, const ssd_launch_opts *o,
                VerifyPlan *plan) {
    const int es = dtype == SSD_F32 ? 4 : 2;
    VerifyPlan pl{};
    pl.kernel = (o && o->kernel) ? o->kernel : 2;
    if (pl.kernel != 1 && pl.kernel != 2) return SSD_ERR_ARG;
    const int sms = device_sm_count();
    if (sms <= 0 && !(o && o->ctas > 0)) return SSD_ERR_CUDA;
    pl.ctas = (o && o->ctas > 0) ? o->ctas : sms;
    const int64_t row_bytes = (int64_t)V * es;
    // column spans per row: enough items for a few balanced waves when there are few rows
    int split = 1;
    if (o && o->split > 0) {
        split = o->split;
    } else if (M > 0 && M < 4ll * pl.ctas) {
        // about four items per CTA, spans of 32 KB at least: every span is a stage hand-over
        // for the consumers, so more and smaller ones lose what the better balance gains
        // (250 rows of 98 KB: 13.9 us with 2 or 3 spans, 16.0 with 5, 16.9 with 6)
        const int64_t want = (4ll * pl.ctas + M - 1) / M;
        const int64_t most = row_bytes / 32768 > 1 ? row_bytes / 32768 : 1;
        split = (int)(want < most ? want : most);
    }
    if (split < 1) split = 1;
    if (split > 64) split = 64;
    pl.split = split;
    if (pl.kernel == 2) {
        pl.warps = (o && o->warps > 0) ? o->warps : (row_bytes >= 96 * 1024 ? 12 : 16);
        if (pl.warps > 16) return SSD_ERR_ARG;
        const int off_cache = (B + 1 <= kOffCacheMax) ? (B + 1) * 8 : 0;
        const int budget = 222 * 1024 - 512 - off_cache;
        const int max_stage = (budget / 2) & ~127;     // two stages must fit
        if (o && o->stage_bytes > 0) {
            pl.stage_bytes = o->stage_bytes;
        } else {
            // A span is cut into as few equal parts as a ring of two stages allows, one part per
            // stage.  Every stage costs each consumer warp about a hundred instructions of
            // hand-over whatever its size (measured: 0.33 us per stage and CTA), and two stages
            // of ~100 KB already keep enough bytes in flight, so few large stages beat a deeper
            // ring of small ones: a 98 KB row as one stage streams 6 % faster than as two.
            const int64_t span = (row_bytes + split - 1) / split + 32;
            const int64_t parts = (span + max_stage - 1) / max_stage;
            int64_t sb = ((span + parts - 1) / parts + 16 + 127) & ~127ll;
            if (sb < 4096) sb = 4096;
            if (sb > max_stage) sb = max_stage;
            pl.stage_bytes = (int)sb;
        }
        if (pl.stage_bytes < 1024 || pl.stage_bytes > max_stage || (pl.stage_bytes & 127))
            return SSD_ERR_ARG;
        pl.stages = (o && o->stages > 0) ? o->stages : budget / pl.stage_bytes;
        if (pl.stages > 16) pl.stages = 16;
        if (pl.stages < 2 || (int64_t)pl.stages * pl.stage_bytes > budget) return SSD_ERR_ARG;
        pl.smem_bytes = 128 + (size_t)((2 * pl.stages * 8 + pl.stages * sizeof(StageDesc) +
                                        off_cache + 127) & ~127) +
                        (size_t)pl.stages * pl.stage_bytes;
    } else {
        pl.warps = 8;
        pl.stages = 0; pl.stage_bytes = 0; pl.smem_bytes = 0;
    }
    // measured: one pair of four on the FMA pipe is the best split for bf16 (two lose to
    // instruction issue); fp32 logits are HBM-bound without it
    pl.fma_exp = (o && o->fma_exp) ? (o->fma_exp < 0 ? 0 : o->fma_exp) : (dtype == SSD_BF16 ? 1 : 0);
    if (pl.fma_exp > 3) return SSD_ERR_ARG;
    pl.partials = split * pl.warps;
    // header | two words per utterance | partials
    pl.workspace_bytes = 256 + (((size_t)(B > 0 ? B : 0) * 16 + 255) & ~(size_t)255) +
                         (size_t)M * pl.partials * sizeof(float2);
    // Rows can be finished inside the streaming kernel where that kernel sees whole rows and can
    // keep the utterance offsets in shared memory.  It is not the default: in a chain of calls
    // the closing kernel's few microseconds are when the next streaming kernel's CTAs (which
    // need the SM's whole shared memory) get resident and past their set-up, and without it that
    // ramp-up is exposed instead (measured: 108 against 104 us per step on 32 utterances).
    const int finish = o ? o->finish : 0;
    if (finish < 0 || finish > 2) return SSD_ERR_ARG;
    pl.finish_inside = 0;
    if (finish == 2 && pl.kernel == 2 && split == 1 && B > 0 && B + 1 <= kOffCacheMax && M > 0) {
        const int NR = 2 * pl.stages;
        size_t hdr = 2 * (size_t)pl.stages * 8 + pl.stages * sizeof(StageDesc) + NR * sizeof(FinRow) +
                     (size_t)NR * pl.warps * 8 + pl.stages * 4 + 8 + (size_t)(B + 1) * 8;
        pl.fin_smem_bytes = 128 + ((hdr + 127) & ~(size_t)127) + (size_t)pl.stages * pl.stage_bytes;
        pl.finish_inside = pl.fin_smem_bytes <= 227 * 1024 ? 1 : 0;
    }
    if (finish == 2 && !pl.finish_inside) return SSD_ERR_ARG;
    *plan = pl;
    return SSD_OK;
}

static size_t partials_offset(int B) {
    return 256 + (((size_t)(B > 0 ? B : 0) * 16 + 255) & ~(size_t)255);
}

// Launches the streaming kernel that leaves plan.partials (reference, sum) pairs per row in the
// workspace (nothing for rows of skipped utterances).
static int launch_verify_rows(const void *logits, ssd_dtype dtype, int V, int64_t ld, int64_t M,
                              const int64_t *tok_off, int B, const uint8_t *skip, void *workspace,
                              unsigned long long epoch, const VerifyPlan &plan, const Launch &L) {
    if (M == 0) return SSD_OK;
    const ssd_launch_opts *o = L.opts;
    cudaError_t e;
    VerifyParams p{};
    p.logits = static_cast<const char *>(logits);
    p.V = V; p.ld = ld; p.M = M; p.split = plan.split; p.num_items = M * plan.split;
    p.tok_off = tok_off; p.B = B; p.skip = skip;
    p.partials = reinterpret_cast<float2 *>(static_cast<char *>(workspace) + partials_offset(B));
    p.partials_per_row = plan.partials;
    p.warps = plan.warps; p.stages = plan.stages; p.stage_bytes = plan.stage_bytes;
    p.err_word = static_cast<unsigned long long *>(workspace); p.epoch = epoch;
    int64_t ctas = p.num_items < plan.ctas ? p.num_items : plan.ctas;
    if (o && o->ev_begin) {
        e = cudaEventRecord(static_cast<cudaEvent_t>(o->ev_begin), L.stream);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    }
    if (plan.kernel == 2) {
        void (*kern)(const VerifyParams) = verify_rows_tma<float, 0, false>;
        if (dtype == SSD_BF16)
            kern = plan.fma_exp == 1 ? verify_rows_tma<bf16_t, 1, false>
                 : plan.fma_exp == 2 ? verify_rows_tma<bf16_t, 2, false>
                 : plan.fma_exp == 3 ? verify_rows_tma<bf16_t, 3, false>
                                     : verify_rows_tma<bf16_t, 0, false>;
        e = ensure_dynamic_smem(reinterpret_cast<const void *>(kern), plan.smem_bytes);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
        e = launch_pdl(kern, (unsigned)ctas, (unsigned)((plan.warps + 1) * 32), plan.smem_bytes,
                       L.stream, p);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    } else {
        ctas = p.num_items < 8ll * plan.ctas ? p.num_items : 8ll * plan.ctas;
        e = launch_pdl(dtype == SSD_F32 ? verify_rows_plain<float> : verify_rows_plain<bf16_t>,
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

// Eq. 5's threshold on the host: log(tau) in fp64, rounded to fp32.  tau <= 0 rejects nothing
// (p > 0 always), tau >= 1 everything (p <= 1 always), whatever rounding does to log p.
struct Threshold {
    float log_tau;
    int reject_none, reject_all;
};
static Threshold threshold_of(float tau_slm) {
    const double tau = (double)tau_slm;
    Threshold t;
    t.reject_none = !(tau > 0.0);
    t.reject_all = tau >= 1.0;
    t.log_tau = t.reject_none ? -INFINITY : (float)log(tau);
    return t;
}

int launch_verify(const void *logits, ssd_dtype dtype, int V, int64_t ld, int64_t M,
                  const int64_t *tok_off, const int32_t *draft_ids, int B, float tau_slm,
                  const uint8_t *skip, void *workspace, float *token_logp, float *row_lse,
                  int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                  const VerifyPlan &plan, const Launch &L) {
    if (B == 0) return SSD_OK;
    const ssd_launch_opts *o = L.opts;
    unsigned long long *err_word = static_cast<unsigned long long *>(workspace);
    float2 *partials = reinterpret_cast<float2 *>(static_cast<char *>(workspace) + partials_offset(B));
    const unsigned long long epoch = next_epoch();
    const Threshold th = threshold_of(tau_slm);
    cudaError_t e;
    if (plan.finish_inside) {
        // The per-utterance words of this variant are told apart from leftovers by the host's
        // call number, which a captured launch would repeat at every replay: not while capturing.
        cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
        e = cudaStreamIsCapturing(L.stream, &capturing);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
        if (capturing != cudaStreamCaptureStatusNone) return SSD_ERR_ARG;
        FinParams q{};
        VerifyParams &p = q.v;
        p.logits = static_cast<const char *>(logits);
        p.V = V; p.ld = ld; p.M = M; p.split = 1; p.num_items = M;
        p.tok_off = tok_off; p.B = B; p.skip = skip;
        p.warps = plan.warps; p.stages = plan.stages; p.stage_bytes = plan.stage_bytes;
        p.err_word = err_word; p.epoch = epoch;
        q.draft_ids = draft_ids;
        q.log_tau = th.log_tau; q.reject_none = th.reject_none; q.reject_all = th.reject_all;
        q.token_logp = token_logp; q.row_lse = row_lse;
        q.accepted_len = accepted_len; q.all_accepted = all_accepted; q.utt_status = utt_status;
        q.utt_words = reinterpret_cast<unsigned long long *>(static_cast<char *>(workspace) + 256);
        q.done_ctas = err_word + 1;
        q.epoch32 = scratch_tag((uint32_t)epoch);
        const int64_t ctas = M < plan.ctas ? M : plan.ctas;
        if (o && o->ev_begin) {
            e = cudaEventRecord(static_cast<cudaEvent_t>(o->ev_begin), L.stream);
            if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
        }
        void (*kern)(const FinParams) = verify_rows_fin<float, 0>;
        if (dtype == SSD_BF16)
            kern = plan.fma_exp == 1 ? verify_rows_fin<bf16_t, 1>
                 : plan.fma_exp == 2 ? verify_rows_fin<bf16_t, 2>
                 : plan.fma_exp == 3 ? verify_rows_fin<bf16_t, 3>
                                     : verify_rows_fin<bf16_t, 0>;
        e = ensure_dynamic_smem(reinterpret_cast<const void *>(kern), plan.fin_smem_bytes);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
        e = launch_pdl(kern, (unsigned)ctas, (unsigned)((plan.warps + 1) * 32), plan.fin_smem_bytes,
                       L.stream, q);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
        if (o && o->ev_end) {
            e = cudaEventRecord(static_cast<cudaEvent_t>(o->ev_end), L.stream);
            if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
        }
        return SSD_OK;
    }
    const int rc = launch_verify_rows(logits, dtype, V, ld, M, tok_off, B, skip, workspace, epoch,
                                      plan, L);
    if (rc != SSD_OK) return rc;
    e = launch_pdl(
        dtype == SSD_F32 ? verify_finish_kernel<float> : verify_finish_kernel<bf16_t>,
        (unsigned)B, (unsigned)kFinishThreads, 0, L.stream,
        static_cast<const char *>(logits), V, ld, M, tok_off, draft_ids, B, th.log_tau,
        th.reject_none, th.reject_all, skip, static_cast<const float2 *>(partials), plan.partials,
        token_logp, row_lse, accepted_len, all_accepted, utt_status,
        static_cast<const unsigned long long *>(err_word), epoch);
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

// Vocabulary-parallel verification, this rank's part: the same streaming kernel over the local
// columns, then one (maximum, sum, draft logit) triple per row.
int launch_verify_shard(const void *logits, ssd_dtype dtype, int V_local, int64_t ld, int64_t M,
                        int64_t col0, const int64_t *tok_off, const int32_t *draft_ids, int B,
                        const uint8_t *skip, void *workspace, float *shard_stats,
                        const VerifyPlan &plan, const Launch &L) {
    if (B == 0) return SSD_OK;
    unsigned long long *err_word = static_cast<unsigned long long *>(workspace);
    float2 *partials = reinterpret_cast<float2 *>(static_cast<char *>(workspace) + partials_offset(B));
    const unsigned long long epoch = next_epoch();
    const int rc = launch_verify_rows(logits, dtype, V_local, ld, M, tok_off, B, skip, workspace,
                                      epoch, plan, L);
    if (rc != SSD_OK) return rc;
    cudaError_t e = launch_pdl(
        dtype == SSD_F32 ? shard_finish_kernel<float> : shard_finish_kernel<bf16_t>,
        (unsigned)B, (unsigned)kFinishThreads, 0, L.stream,
        static_cast<const char *>(logits), V_local, ld, M, col0, tok_off, draft_ids, B, skip,
        static_cast<const float2 *>(partials), plan.partials, shard_stats,
        static_cast<const unsigned long long *>(err_word), epoch);
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

int launch_verify_combine(const float *stats_all, int R, int64_t V_total, const int64_t *tok_off,
                          const int32_t *draft_ids, int B, int64_t M, float tau_slm,
                          const uint8_t *skip, float *token_logp, float *row_lse,
                          int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                          cudaStream_t stream) {
    if (B == 0) return SSD_OK;
    const Threshold th = threshold_of(tau_slm);
    cudaError_t e = launch_pdl(combine_kernel, (unsigned)B, (unsigned)kFinishThreads, 0, stream,
                               stats_all, R, V_total, M, tok_off, draft_ids, B, th.log_tau,
                               th.reject_none, th.reject_all, skip, token_logp, row_lse,
                               accepted_len, all_accepted, utt_status);
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

size_t greedy_workspace_bytes(int64_t R, const VerifyPlan &plan) {
    return 256 + (size_t)R * plan.partials * sizeof(float4);
}

int launch_greedy(const void *logits, ssd_dtype dtype, int V, int64_t ld, int64_t R,
                  void *workspace, int32_t *next_token, float *next_logp, float *row_lse,
                  uint32_t *row_status, const VerifyPlan &plan, const Launch &L) {
    if (R == 0) return SSD_OK;
    if (plan.kernel != 2) return SSD_ERR_ARG;      // only the bulk-copy kernel tracks the arg max
    const ssd_launch_opts *o = L.opts;
    unsigned long long *err_word = static_cast<unsigned long long *>(workspace);
    float4 *partials = reinterpret_cast<float4 *>(static_cast<char *>(workspace) + 256);
    const unsigned long long epoch = next_epoch();
    VerifyParams p{};
    p.logits = static_cast<const char *>(logits);
    p.V = V; p.ld = ld; p.M = R; p.split = plan.split; p.num_items = R * plan.split;
    p.tok_off = nullptr; p.B = 0; p.skip = nullptr;
    p.partials = reinterpret_cast<float2 *>(partials); p.partials_per_row = plan.partials;
    p.warps = plan.warps; p.stages = plan.stages; p.stage_bytes = plan.stage_bytes;
    p.err_word = err_word; p.epoch = epoch;
    const int64_t ctas = p.num_items < plan.ctas ? p.num_items : plan.ctas;
    cudaError_t e;
    if (o && o->ev_begin) {
        e = cudaEventRecord(static_cast<cudaEvent_t>(o->ev_begin), L.stream);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    }
    void (*kern)(const VerifyParams) = verify_rows_tma<float, 0, true>;
    if (dtype == SSD_BF16)
        kern = plan.fma_exp >= 1 ? verify_rows_tma<bf16_t, 1, true> : verify_rows_tma<bf16_t, 0, true>;
    e = ensure_dynamic_smem(reinterpret_cast<const void *>(kern), plan.smem_bytes);
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    e = launch_pdl(kern, (unsigned)ctas, (unsigned)((plan.warps + 1) * 32), plan.smem_bytes,
                   L.stream, p);
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    if (o && o->ev_end) {
        e = cudaEventRecord(static_cast<cudaEvent_t>(o->ev_end), L.stream);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    }
    e = launch_pdl(greedy_finish_kernel, (unsigned)((R + kGreedyWarps - 1) / kGreedyWarps),
                   (unsigned)(kGreedyWarps * 32), 0, L.stream, V, R,
                   static_cast<const float4 *>(partials), plan.partials, next_token, next_logp,
                   row_lse, row_status, static_cast<const unsigned long long *>(err_word), epoch);
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

}  // namespace ssd
