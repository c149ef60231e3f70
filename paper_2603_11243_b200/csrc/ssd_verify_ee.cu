// ssd_verify_early_exit: verification that stops reading an utterance's rows once its first
// rejected position is known.  The method only needs the accepted prefix length (Section 2.3:
// j is the FIRST position whose likelihood is <= tau_SLM), so every row after that position is
// bandwidth spent for nothing.
//
// Rows are visited position-major (position 0 of every utterance, then position 1, ...), claimed
// in that order by persistent CTAs from a global counter, so that all CTAs work on about the
// same position at any time and stay equally loaded although rows drop out at random.  A row
// is finalised inside the streaming kernel: the consumer warps leave their (reference, sum)
// pairs and the draft token's logit in shared memory, and the producer warp, when it is about
// to refill the stage that held the row's last part, merges them, writes the row's
// log-likelihood and, on a reject, lowers the utterance's first-reject word in global memory
// with an atomic minimum.  Before a row is fetched the producer reads that word and skips the
// row if a smaller rejected position is already known.  Positions up to the true first reject
// are therefore never skipped, and the result is exactly that of ssd_verify.
#include <limits.h>
#include <math.h>

#include "ssd_common.cuh"
#include "ssd_ranges.cuh"
#include "ssd_stream.cuh"

namespace ssd {

unsigned long long next_epoch();

namespace {

using namespace stream;

struct EeParams {
    const char *logits;
    int V;
    int64_t ld;
    int64_t M;
    const int64_t *tok_off;
    const int32_t *draft_ids;
    int B;
    const uint8_t *skip;
    float log_tau;
    int reject_none, reject_all;
    float *token_logp;
    float *row_lse;
    int32_t *first_reject;     // [B] lowest rejected position known so far (K_b: none)
    uint32_t *flags;           // [B] status bits
    int32_t *rows_read;        // [B]
    const int32_t *kmax;       // largest K_b among the utterances to verify
    unsigned long long *next_item;   // position-major items handed out so far
    int warps, stages, stage_bytes;
    unsigned long long *err_word;
    unsigned long long epoch;
};

struct RowMeta {
    int64_t row;
    int32_t b, pos, id_ok, pad;
};

// ---- set-up: per-utterance words and the largest draft length ---------------------------------
__global__ void __launch_bounds__(1024) ee_init_kernel(
    const int64_t *__restrict__ tok_off, const uint8_t *__restrict__ skip, int B, int64_t M,
    int32_t *__restrict__ first_reject, uint32_t *__restrict__ flags,
    int32_t *__restrict__ rows_read, int32_t *__restrict__ kmax,
    unsigned long long *__restrict__ next_item) {
    __shared__ int warp_max_sh[32];
    pdl_enter();
    if (threadIdx.x == 0) *next_item = 0ull;
    int mx = 0;
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        const int64_t i0 = tok_off[b], i1 = tok_off[b + 1];
        const bool ok = !(i0 < 0 || i1 < i0 || i1 > M);
        const int K = ok ? (int)min(i1 - i0, (int64_t)INT_MAX) : 0;
        first_reject[b] = K;
        flags[b] = ok ? 0u : (uint32_t)SSD_UTT_BAD_OFFSETS;
        rows_read[b] = 0;
        if (ok && !(skip && skip[b])) mx = max(mx, K);
    }
    mx = __reduce_max_sync(0xffffffffu, mx);
    if ((threadIdx.x & 31) == 0) warp_max_sh[threadIdx.x >> 5] = mx;
    __syncthreads();
    if (threadIdx.x < 32) {
        mx = __reduce_max_sync(0xffffffffu, warp_max_sh[threadIdx.x]);
        if (threadIdx.x == 0) *kmax = mx;
    }
}

// ---- the streaming kernel -------------------------------------------------------------------
template <typename T, int kF>
__global__ void __launch_bounds__(544, 1) verify_rows_ee(const EeParams p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    constexpr int ES = Elem<T>::kBytes, EPC = Elem<T>::kPerChunk;
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int S = p.stages, CW = p.warps, NR = 2 * S;
    // layout: full[S] | empty[S] | desc[S] | pending[S] | rowmeta[NR] | sx[NR] | spart[NR*CW] |
    //         offsets cache | stages
    unsigned char *smem = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t full0 = sbase, empty0 = sbase + S * 8;
    size_t o = 2 * (size_t)S * 8;
    StageDesc *desc = reinterpret_cast<StageDesc *>(smem + o);          o += S * sizeof(StageDesc);
    RowMeta *rowmeta = reinterpret_cast<RowMeta *>(smem + o);          o += NR * sizeof(RowMeta);
    float2 *spart = reinterpret_cast<float2 *>(smem + o);              o += (size_t)NR * CW * 8;
    float *sx = reinterpret_cast<float *>(smem + o);                   o += NR * 4;
    int32_t *pending = reinterpret_cast<int32_t *>(smem + o);          o += S * 4;
    o = (o + 7) & ~(size_t)7;
    const bool cache_off = p.B + 1 <= kOffCacheMax;
    int64_t *off_cache = reinterpret_cast<int64_t *>(smem + o);
    if (cache_off) o += (size_t)(p.B + 1) * 8;
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
    }
    pdl_wait();
    if (cache_off)
        for (int i = threadIdx.x; i <= p.B; i += blockDim.x) off_cache[i] = p.tok_off[i];
    __syncthreads();

    const int64_t row_bytes = (int64_t)p.V * ES;

    if (warp == 0) {
        // =============================== producer ===============================
        const int64_t *offs = cache_off ? off_cache : p.tok_off;
        const int64_t num_items = (int64_t)(*p.kmax) * p.B;
        int s = 0;
        uint32_t ph = 0;
        int rowseq = 0;
        bool failed = false;
        const int max_chunks = p.stage_bytes >> 4;

        // Merges the partials of the row in row slot slot1 - 1 (0: none), once the consumers
        // have let go of the stage that held its last part; called by all lanes.  It touches
        // the row slot only, not the stage, so it runs after the stage's next copy is under way.
        auto finalize = [&](int slot1) {
            if (slot1 == 0) return;
            const int slot = slot1 - 1;
            const float2 v = lane < CW ? spart[slot * CW + lane] : make_float2(kNegInit, 0.f);
            const float Mx = fmaxf(warp_max(v.x), kNegInit);
            const float Ssum = warp_sum(v.y * ex2((v.x - Mx) * kLog2e));
            if (lane == 0) {
                const RowMeta rm = rowmeta[slot];
                const float lnS = logf(Ssum);
                const float lse = Mx + lnS;
                uint32_t fl = 0;
                if (!(fabsf(lse) < INFINITY)) fl |= SSD_UTT_NONFINITE;
                float logp;
                bool reject;
                if (!rm.id_ok) {
                    fl |= SSD_UTT_BAD_DRAFT_ID;
                    logp = -INFINITY;
                    reject = true;
                } else {
                    logp = (sx[slot] - Mx) - lnS;
                    reject = p.reject_none ? false : (p.reject_all || !(logp > p.log_tau));   // p <= tau; NaN rejects
                }
                p.token_logp[rm.row] = logp;
                if (p.row_lse) p.row_lse[rm.row] = lse;
                if (fl) atomicOr(&p.flags[rm.b], fl);
                if (reject) atomicMin(&p.first_reject[rm.b], rm.pos);
                atomicAdd(&p.rows_read[rm.b], 1);
            }
            __syncwarp();
        };

        // Items (position-major) are claimed a few at a time from a global counter: rows are
        // skipped at random, so a fixed deal would leave the CTAs with unequal work.  The next
        // claim is made before the current batch is worked on, to hide the atomic's latency.
        // (A claim spans B/16 items at most: with few utterances a long claim would let the
        // CTAs drift many positions apart.)
        const int claim_items = max(1, min(32, p.B / 16));
        auto claim = [&]() {
            unsigned long long v = 0;
            if (lane == 0) v = atomicAdd(p.next_item, (unsigned long long)claim_items);
            return (int64_t)__shfl_sync(0xffffffffu, v, 0);
        };
        auto known_reject = [&](int b) {
            return *reinterpret_cast<const volatile int32_t *>(&p.first_reject[b]);
        };
        int64_t next_base = claim();
        while (!failed) {
            const int64_t base = next_base;
            if (base >= num_items) break;
            next_base = claim();
            const int64_t mine = base + lane;
            bool active = lane < claim_items && mine < num_items;
            int my_b = 0, my_pos = 0, my_id = -1;
            int64_t my_row = 0;
            if (active) {
                my_pos = (int)(mine / p.B);
                my_b = (int)(mine - (int64_t)my_pos * p.B);
                const int64_t i0 = offs[my_b], i1 = offs[my_b + 1];
                active = !(i0 < 0 || i1 < i0 || i1 > p.M) && my_pos < i1 - i0 &&
                         !(p.skip && p.skip[my_b]);
                if (active) {
                    my_row = i0 + my_pos;
                    my_id = p.draft_ids[my_row];
                }
            }
            unsigned todo = __ballot_sync(0xffffffffu, active);
            // the first-reject word of a row is read one row ahead of its use
            int fr_next = todo ? known_reject(__shfl_sync(0xffffffffu, my_b, __ffs(todo) - 1)) : 0;
            while (todo && !failed) {
                const int src = __ffs(todo) - 1;
                todo &= todo - 1;
                const int64_t row = __shfl_sync(0xffffffffu, my_row, src);
                const int b = __shfl_sync(0xffffffffu, my_b, src);
                const int pos = __shfl_sync(0xffffffffu, my_pos, src);
                const int fr = fr_next;
                if (todo) fr_next = known_reject(__shfl_sync(0xffffffffu, my_b, __ffs(todo) - 1));
                const int id = __shfl_sync(0xffffffffu, my_id, src);
                // a smaller rejected position already known: the row cannot matter
                if (pos > fr) continue;
                const bool id_ok = id >= 0 && id < p.V;
                const ranges::RowGeom geom = ranges::row_geom(
                    reinterpret_cast<uintptr_t>(p.logits), row, p.ld * ES, row_bytes);
                const uintptr_t g0 = geom.g0, g1 = geom.g1, f0 = geom.f0;
                const int row_chunks = geom.row_chunks;
                const ranges::SpanCut cut = ranges::span_cut(row_chunks, 1, 0, max_chunks);
                const int parts = cut.parts, per_part = cut.per_part;
                const int64_t id_byte = id_ok ? (int64_t)(g0 - f0) + (int64_t)id * ES : -1;
                const int rslot = rowseq % NR;
                ++rowseq;
                if (lane == 0) {
                    RowMeta rm;
                    rm.row = row; rm.b = b; rm.pos = pos; rm.id_ok = id_ok ? 1 : 0; rm.pad = 0;
                    rowmeta[rslot] = rm;
                }
                for (int part = 0; part < parts; ++part) {
                    if (!mbar_wait_bounded(empty0 + s * 8, ph ^ 1u)) { failed = true; break; }
                    const int done_slot1 = pending[s];     // the row this stage held last, if any
                    __syncwarp();
                    const int pc0 = part * per_part;
                    const int pc1 = min(row_chunks, pc0 + per_part);
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
                        const bool last = part == parts - 1;
                        desc[s].nchunks = pc1 - pc0;
                        desc[s].flags = last ? kFlagLast : 0u;
                        desc[s].slot = rslot;
                        desc[s].elem0 = 0;
                        // where the draft token's logit sits in this stage, if it does
                        desc[s].gather = (id_byte >= (int64_t)pc0 * 16 && id_byte < (int64_t)pc1 * 16)
                                          ? (int32_t)(id_byte - (int64_t)pc0 * 16) : -1;
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
                    finalize(done_slot1);
                    if (++s == S) { s = 0; ph ^= 1u; }
                }
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
        bool failed = false;
        int s = 0;
        uint32_t ph = 0;
        for (;;) {
            if (!mbar_wait_bounded(full0 + s * 8, ph)) { failed = true; break; }
            const int n = desc[s].nchunks;
            const uint32_t flags = desc[s].flags;
            if (flags & kFlagEnd) break;
            const uint32_t a0 = stage0 + (uint32_t)s * p.stage_bytes;
            consume_stage<T, kF, false>(a0, n, ct, NT, st, 0, unused);
            const int slot = (int)desc[s].slot;
            const int g = desc[s].gather;
            if (g >= 0 && ct == 0) sx[slot] = Elem<T>::load_shared(a0 + (uint32_t)g);
            if (flags & kFlagLast) {
                const float2 r = warp_merge(st);
                if (lane == 0) spart[slot * CW + cw] = r;
                st.reset();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + s * 8);      // releases the writes above as well
            if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (failed) {
            if (lane == 0) atomicExch(p.err_word, p.epoch);
            drain_after_error();
        }
    }
}

__global__ void __launch_bounds__(256) ee_finish_kernel(
    const int64_t *__restrict__ tok_off, const uint8_t *__restrict__ skip, int B, int64_t M,
    const int32_t *__restrict__ first_reject, const uint32_t *__restrict__ flags,
    const int32_t *__restrict__ rows_read_ws, int32_t *__restrict__ accepted_len,
    uint8_t *__restrict__ all_accepted, uint32_t *__restrict__ utt_status,
    int32_t *__restrict__ rows_read, const unsigned long long *err_word,
    unsigned long long epoch) {
    pdl_enter();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const uint32_t internal = (*err_word == epoch) ? (uint32_t)SSD_UTT_INTERNAL : 0u;
    const int64_t i0 = tok_off[b], i1 = tok_off[b + 1];
    const bool ok = !(i0 < 0 || i1 < i0 || i1 > M);
    const int K = ok ? (int)min(i1 - i0, (int64_t)INT_MAX) : 0;
    const int fr = first_reject[b];
    accepted_len[b] = ok ? fr : 0;
    all_accepted[b] = (ok && fr == K) ? 1 : 0;
    utt_status[b] = flags[b] | internal;
    if (rows_read) rows_read[b] = rows_read_ws[b];
}

size_t ee_smem_bytes(int B, const VerifyPlan &plan) {
    const int S = plan.stages, NR = 2 * S;
    size_t o = 2 * (size_t)S * 8 + S * sizeof(StageDesc) + NR * sizeof(RowMeta) +
               (size_t)NR * plan.warps * 8 + NR * 4 + S * 4 + 8;
    if (B + 1 <= kOffCacheMax) o += (size_t)(B + 1) * 8;
    return 128 + ((o + 127) & ~(size_t)127) + (size_t)S * plan.stage_bytes;
}

}  // namespace

// Workspace: [0,256) header (error word, kmax at byte 64, item counter at byte 128), then three
// int32 arrays of B.
size_t verify_ee_workspace_bytes(int B, const VerifyPlan &full_plan) {
    const size_t ee = 256 + 3 * (((size_t)B * 4 + 255) & ~(size_t)255);
    return ee > full_plan.workspace_bytes ? ee : full_plan.workspace_bytes;
}

// Whether the early-exit kernel is used for these sizes (else the call falls back to the full
// kernel, whose outputs are a superset): rows must not be split into column spans, there must
// be enough rows to balance the CTAs, and the position-major item count must fit 31 bits.
bool verify_ee_applicable(int B, int64_t M, const VerifyPlan &plan) {
    return plan.kernel == 2 && plan.split == 1 && B > 0 && M >= 4ll * plan.ctas &&
           M * 4 < (1ll << 31) && (int64_t)B * M < (1ll << 40);
}

int launch_verify_ee(const void *logits, ssd_dtype dtype, int V, int64_t ld, int64_t M,
                     const int64_t *tok_off, const int32_t *draft_ids, int B, float tau_slm,
                     const uint8_t *skip, void *workspace, float *token_logp, float *row_lse,
                     int32_t *accepted_len, uint8_t *all_accepted, uint32_t *utt_status,
                     int32_t *rows_read, const VerifyPlan &plan, const Launch &L) {
    if (B == 0) return SSD_OK;
    const ssd_launch_opts *o = L.opts;
    char *ws = static_cast<char *>(workspace);
    const size_t arr = ((size_t)B * 4 + 255) & ~(size_t)255;
    unsigned long long *err_word = reinterpret_cast<unsigned long long *>(ws);
    int32_t *kmax = reinterpret_cast<int32_t *>(ws + 64);
    unsigned long long *next_item = reinterpret_cast<unsigned long long *>(ws + 128);
    int32_t *first_reject = reinterpret_cast<int32_t *>(ws + 256);
    uint32_t *flags = reinterpret_cast<uint32_t *>(ws + 256 + arr);
    int32_t *rr = reinterpret_cast<int32_t *>(ws + 256 + 2 * arr);
    const unsigned long long epoch = next_epoch();
    cudaError_t e = launch_pdl(ee_init_kernel, 1u, 1024u, 0, L.stream, tok_off, skip, B, M,
                               first_reject, flags, rr, kmax, next_item);
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    EeParams p{};
    p.logits = static_cast<const char *>(logits);
    p.V = V; p.ld = ld; p.M = M; p.tok_off = tok_off; p.draft_ids = draft_ids; p.B = B;
    p.skip = skip;
    const double tau = (double)tau_slm;
    p.reject_none = !(tau > 0.0);
    p.reject_all = tau >= 1.0;     // p <= 1 always, whatever rounding makes of log p
    p.log_tau = p.reject_none ? -INFINITY : (float)log(tau);
    p.token_logp = token_logp; p.row_lse = row_lse;
    p.first_reject = first_reject; p.flags = flags; p.rows_read = rr; p.kmax = kmax;
    p.next_item = next_item;
    p.warps = plan.warps; p.stages = plan.stages; p.stage_bytes = plan.stage_bytes;
    p.err_word = err_word; p.epoch = epoch;
    VerifyPlan pl = plan;                      // the extra per-row slots may cost one stage
    while (ee_smem_bytes(B, pl) > 227 * 1024 && pl.stages > 2) --pl.stages;
    p.stages = pl.stages;
    const size_t smem = ee_smem_bytes(B, pl);
    if (smem > 227 * 1024) return SSD_ERR_ARG;
    if (o && o->ev_begin) {
        e = cudaEventRecord(static_cast<cudaEvent_t>(o->ev_begin), L.stream);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    }
    void (*kern)(const EeParams) = verify_rows_ee<float, 0>;
    if (dtype == SSD_BF16) kern = plan.fma_exp >= 1 ? verify_rows_ee<bf16_t, 1> : verify_rows_ee<bf16_t, 0>;
    e = ensure_dynamic_smem(reinterpret_cast<const void *>(kern), smem);
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    e = launch_pdl(kern, (unsigned)plan.ctas, (unsigned)((plan.warps + 1) * 32), smem, L.stream, p);
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    if (o && o->ev_end) {
        e = cudaEventRecord(static_cast<cudaEvent_t>(o->ev_end), L.stream);
        if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    }
    e = launch_pdl(ee_finish_kernel, (unsigned)((B + 255) / 256), 256u, 0, L.stream, tok_off, skip,
                   B, M, static_cast<const int32_t *>(first_reject),
                   static_cast<const uint32_t *>(flags), static_cast<const int32_t *>(rr),
                   accepted_len, all_accepted, utt_status, rows_read,
                   static_cast<const unsigned long long *>(err_word), epoch);
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    e = cudaGetLastError();
    if (e != cudaSuccess) { record_cuda_error(e); return SSD_ERR_CUDA; }
    return SSD_OK;
}

}  // namespace ssd
