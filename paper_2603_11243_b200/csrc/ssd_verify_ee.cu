// ssd_verify_early_exit: verification that stops reading an utterance's rows once its first
// rejected position is known.  The method only needs the accepted prefix length (Section 2.3:
// j is the FIRST position whose likelihood is <= tau_SLM), so every row after that position is
// bandwidth spent for nothing.
//
// Rows are visited position-major (position 0 of every utterance, then position 1, ...), claimed
// in that order by persistent CTAs from a global counter, so that all CTAs work on about the
// same position at any time and stay equally loaded although rows drop out at random.  A row
// is finished inside the streaming kernel: the consumer warps leave their (reference, sum)
// pairs and the draft token's logit in shared memory, and a warp of its own merges them, writes
// the row's log-likelihood and, on a reject, lowers the utterance's first-reject word in global
// memory with an atomic minimum.  Before a row is fetched the producer reads that word and
// skips the row if a smaller rejected position is already known.  Positions up to the true
// first reject are therefore never skipped, and the result is exactly that of ssd_verify.
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
    int claim_items;           // items per claim from the counter
    unsigned long long *err_word;
    unsigned long long epoch;
};

struct RowMeta {
    int64_t row;
    int32_t b, pos;
};

// Items per claim from the position-major counter.  Two limits: B/16, because with few
// utterances a long claim lets the CTAs drift many positions apart (rows get read that a reject
// a few positions earlier would have spared); and a twelfth of a CTA's share of the rows, so that
// the last claims leave the CTAs level (32-item claims on 6,144 rows: 1.5 times the time of
// 4-item ones).  One-item claims cost more in counter traffic than they gain.
inline int ee_claim_items(int B, int64_t M, int ctas) {
    int64_t n = B / 16;
    const int64_t level = M / (12ll * (ctas > 0 ? ctas : 1));
    if (n > level) n = level;
    return n < 2 ? (B >= 2 ? 2 : 1) : (n > 32 ? 32 : (int)n);
}

// Row slots of a CTA (what the consumers leave of a row until the finishing warp has taken it).
__host__ __device__ inline int ee_row_slots(int stages) { return 2 * stages + 2; }
constexpr int kEeRunning = -1, kEeAborted = -2;     // end_seq before the producer knows the count
constexpr uint32_t kFlagFirst = 4u;                 // stage flag: first stage of a row

// Loads and the claim's atomic as the producer issues them: under a predicate, straight into a
// register that already holds the value for "not loaded".  Written as `if (c) v = load` the warp
// was found waiting for the memory right there (by cycle counter: 1,100 cycles for a claim whose
// value is not needed for two rows' time), as if the result were copied where the branches
// join; issued this way it waits where the value is used.
__device__ __forceinline__ void load_volatile_s32_if(int &dst, const int32_t *ptr, bool pred) {
    asm volatile("{ .reg .pred q; setp.ne.s32 q, %2, 0; @q ld.volatile.global.s32 %0, [%1]; }"
                 : "+r"(dst) : "l"(ptr), "r"((int)pred) : "memory");
}
__device__ __forceinline__ void load_u8_if(int &dst, const uint8_t *ptr, bool pred) {
    asm volatile("{ .reg .pred q; setp.ne.s32 q, %2, 0; @q ld.global.u8 %0, [%1]; }"
                 : "+r"(dst) : "l"(ptr), "r"((int)pred) : "memory");
}
// try_wait that gives the thread back after about `ns` nanoseconds at the latest (the plain form
// may keep it for a time of the hardware's choosing: microseconds when nothing completes the phase).
__device__ __forceinline__ bool mbar_try_wait_for(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile("{ .reg .pred q; mbarrier.try_wait.parity.shared::cta.b64 q, [%1], %2, %3; selp.u32 %0, 1, 0, q; }"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void atom_add_u64_if(unsigned long long &dst, unsigned long long *ptr,
                                                unsigned long long n, bool pred) {
    asm volatile("{ .reg .pred q; setp.ne.s32 q, %3, 0; @q atom.global.add.u64 %0, [%1], %2; }"
                 : "+l"(dst) : "l"(ptr), "l"(n), "r"((int)pred) : "memory");
}

// ---- set-up: per-utterance words and the largest draft length ---------------------------------
__global__ void __launch_bounds__(1024) ee_init_kernel(
    const int64_t *__restrict__ tok_off, const uint8_t *__restrict__ skip, int B, int64_t M,
    int32_t *__restrict__ first_reject, uint32_t *__restrict__ flags,
    int32_t *__restrict__ rows_read, int32_t *__restrict__ kmax,
    unsigned long long *__restrict__ next_item, unsigned long long first_free) {
    __shared__ int warp_max_sh[32];
    pdl_enter();
    if (threadIdx.x == 0) *next_item = first_free;     // every CTA's first two batches are dealt
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
// Warp 0 produces (claims items, fetches rows), warps 1..CW consume, warp CW+1 finishes rows.
// The producer does nothing per row that it does not have to: with a ring of two row-sized
// stages every cycle it spends between a stage's release and the stage's next copy is a cycle
// with less in flight for this SM, and a single warp's dependent instructions are slow next to
// twelve streaming ones (measured with the row's closing arithmetic on the producer: 4,300
// cycles of producer work per row against 3,500 of consumer work; the stage it wanted next was
// free every single time it came to wait for it).
template <typename T, int kF>
__global__ void __launch_bounds__(576, 1) verify_rows_ee(const EeParams p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    constexpr int ES = Elem<T>::kBytes, EPC = Elem<T>::kPerChunk;
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int S = p.stages, CW = p.warps, NR = ee_row_slots(S);
    // layout: full[S] | empty[S] | rowdone[NR] | rowfree[NR] | desc[S] | rowmeta[NR] |
    //         spart[NR*CW] | sx[NR] | sid_ok[NR] | end_seq | offsets cache | stages
    unsigned char *smem = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t full0 = sbase, empty0 = sbase + S * 8;
    const uint32_t rowdone0 = sbase + 2 * S * 8, rowfree0 = rowdone0 + NR * 8;
    size_t o = 2 * (size_t)S * 8 + 2 * (size_t)NR * 8;
    StageDesc *desc = reinterpret_cast<StageDesc *>(smem + o);          o += S * sizeof(StageDesc);
    RowMeta *rowmeta = reinterpret_cast<RowMeta *>(smem + o);          o += NR * sizeof(RowMeta);
    float2 *spart = reinterpret_cast<float2 *>(smem + o);              o += (size_t)NR * CW * 8;
    float *sx = reinterpret_cast<float *>(smem + o);                   o += NR * 4;
    int32_t *sid_ok = reinterpret_cast<int32_t *>(smem + o);           o += NR * 4;
    volatile int32_t *end_seq = reinterpret_cast<volatile int32_t *>(smem + o);   o += 4;
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
        }
        for (int r = 0; r < NR; ++r) {
            mbar_init(rowdone0 + r * 8, CW);
            mbar_init(rowfree0 + r * 8, 1);
        }
        *end_seq = kEeRunning;
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
        // Items at or past kmax * B belong to no row.  The word is needed only to know when to
        // stop (a row's item is recognised by its position being inside its utterance), so the
        // first copies do not wait for it.
        const int kmax = *p.kmax;
        const int64_t item_cap = (int64_t)p.B * p.M;
        const bool small_items = item_cap < (1ll << 31);
        int s = 0;
        uint32_t ph = 0;
        int rowseq = 0;
        bool failed = false;
        const int max_chunks = p.stage_bytes >> 4;

        // Items (position-major) are claimed a few at a time from a global counter: rows are
        // skipped at random, so a fixed deal would leave the CTAs with unequal work.  Nothing
        // here waits for memory where it can be helped.  The claim for the batch after the next
        // one is in flight (its value stays in lane 0 until it is needed).  What the next
        // batch's rows need -- the skip flag and the first reject known by then, which drops
        // rows that cannot matter any more -- is loaded, one item per lane, while the current
        // batch is worked on, and looked at only when that batch's turn comes.  The first-reject
        // word a row is checked against is read while the row before it is handed to the
        // consumers, across batches too.  All of these are words every CTA keeps reading, so
        // they come from L2; the draft token's id, which comes from DRAM at a latency of more
        // than a row's time when the memory is busy, is not the producer's business at all: a
        // consumer thread fetches it while it works through the row.
        const int claim_items = p.claim_items;
        auto claim_begin = [&]() {
            unsigned long long v = 0;
            atom_add_u64_if(v, p.next_item, (unsigned long long)claim_items, lane == 0);
            return v;
        };
        auto known_reject = [&](int b, bool wanted) {
            int v = INT_MAX;
            load_volatile_s32_if(v, p.first_reject + b, wanted);
            return v;
        };
        struct Mine { int64_t row; int b, pos, fr_then, skipped; bool in_range; };
        auto look_up = [&](int64_t base, bool check) {
            Mine m{0, 0, 0, INT_MAX, 0, false};
            const int64_t mine = base + lane;
            m.in_range = lane < claim_items && mine < item_cap;
            if (m.in_range) {
                m.pos = small_items ? (int)((uint32_t)mine / (uint32_t)p.B) : (int)(mine / p.B);
                m.b = (int)(mine - (int64_t)m.pos * p.B);
                const int64_t i0 = offs[m.b], i1 = offs[m.b + 1];
                m.in_range = !(i0 < 0 || i1 < i0 || i1 > p.M) && m.pos < i1 - i0;
                m.row = i0 + m.pos;
            }
            if (!m.in_range) m.b = 0;
            load_volatile_s32_if(m.fr_then, p.first_reject + m.b, m.in_range && check);
            load_u8_if(m.skipped, p.skip + m.b, m.in_range && p.skip != nullptr);
            return m;
        };
        auto live = [&](const Mine &m) {
            return __ballot_sync(0xffffffffu, m.in_range && !m.skipped && m.pos <= m.fr_then);
        };
        // The first two batches are dealt (the set-up kernel starts the counter behind them),
        // and not checked against the first rejects: hardly any is known yet.
        Mine cur = look_up((int64_t)blockIdx.x * claim_items, false);
        int64_t next_base = ((int64_t)gridDim.x + blockIdx.x) * claim_items;
        Mine next = look_up(next_base, false);
        unsigned long long pend = claim_begin();
        unsigned todo = live(cur);
        struct Row { int64_t row; int b, pos; bool valid; };
        // the next row to look at, in claim order; moves on to the next batch when this one is used up
        auto pop = [&]() {
            Row r{0, 0, 0, false};
            for (;;) {
                if (todo) {
                    const int src = __ffs(todo) - 1;
                    todo &= todo - 1;
                    r.row = __shfl_sync(0xffffffffu, cur.row, src);
                    r.b = __shfl_sync(0xffffffffu, cur.b, src);
                    r.pos = __shfl_sync(0xffffffffu, cur.pos, src);
                    r.valid = true;
                    return r;
                }
                if (next_base >= (int64_t)kmax * p.B) return r;      // claims only grow: nothing is left
                cur = next;
                todo = live(cur);
                next_base = (int64_t)__shfl_sync(0xffffffffu, pend, 0);
                next = look_up(next_base, true);
                pend = claim_begin();
            }
        };
        Row R = pop();
        int fr = INT_MAX;
        // a row's slot and how often it has been used; the cut of a row into stages, which is the
        // same for every row unless the rows start at different offsets from a 16-byte boundary
        int rslot = 0, use = 0;
        int cut_chunks = -1, parts = 1, per_part = 0;
        while (R.valid && !failed) {
            const int64_t row = R.row;
            const int b = R.b, pos = R.pos;
            const bool wanted = pos <= fr;     // else a smaller rejected position is known already
            R = pop();
            fr = known_reject(R.b, R.valid);
            if (!wanted) continue;
            const ranges::RowGeom geom = ranges::row_geom(
                reinterpret_cast<uintptr_t>(p.logits), row, p.ld * ES, row_bytes);
            const uintptr_t g0 = geom.g0, g1 = geom.g1, f0 = geom.f0;
            const int row_chunks = geom.row_chunks;
            if (row_chunks != cut_chunks) {
                const ranges::SpanCut cut = ranges::span_cut(row_chunks, 1, 0, max_chunks);
                parts = cut.parts;
                per_part = cut.per_part;
                cut_chunks = row_chunks;
            }
            // the row's slot: free once the finishing warp is through with the row that had it
            ++rowseq;
            if (use > 0 && !mbar_wait_bounded(rowfree0 + rslot * 8, (uint32_t)((use - 1) & 1))) {
                failed = true;
                break;
            }
            if (lane == 0) {
                RowMeta rm;
                rm.row = row; rm.b = b; rm.pos = pos;
                rowmeta[rslot] = rm;
            }
            for (int part = 0; part < parts; ++part) {
                if (!mbar_wait_bounded(empty0 + s * 8, ph ^ 1u)) { failed = true; break; }
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
                    desc[s].nchunks = pc1 - pc0;
                    desc[s].flags = (part == parts - 1 ? kFlagLast : 0u) | (part == 0 ? kFlagFirst : 0u);
                    desc[s].slot = rslot;
                    desc[s].elem0 = (int32_t)(((int64_t)pc0 * 16 - (int64_t)(g0 - f0)) / ES);
                    desc[s].gather = -1;
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
            if (++rslot == NR) { rslot = 0; ++use; }
        }
        if (!failed) {
            // the end marker for the consumers, and for the finishing warp how many rows there were
            if (mbar_wait_bounded(empty0 + s * 8, ph ^ 1u)) {
                if (lane == 0) {
                    desc[s].nchunks = 0; desc[s].flags = kFlagEnd; desc[s].slot = 0; desc[s].gather = -1;
                    mbar_arrive(full0 + s * 8);
                    *end_seq = rowseq;
                }
            } else {
                failed = true;
            }
        }
        if (failed) {
            if (lane == 0) {
                *end_seq = kEeAborted;
                atomicExch(p.err_word, p.epoch);
            }
            drain_after_error();
        }
    } else if (warp <= CW) {
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
        int my_id = -1;
        for (;;) {
            if (!mbar_wait_bounded(full0 + s * 8, ph)) { failed = true; break; }
            const int n = desc[s].nchunks;
            const uint32_t flags = desc[s].flags;
            if (flags & kFlagEnd) break;
            const uint32_t a0 = stage0 + (uint32_t)s * p.stage_bytes;
            const int slot = (int)desc[s].slot;
            // one thread fetches the row's draft token id; it is back before the stage is through
            if (ct == 0 && (flags & kFlagFirst)) my_id = p.draft_ids[rowmeta[slot].row];
            consume_stage<T, kF, false>(a0, n, ct, NT, st, 0, unused);
            if (ct == 0) {
                const bool id_ok = my_id >= 0 && my_id < p.V;
                const int64_t at = (int64_t)my_id - desc[s].elem0;     // element of this stage
                if (id_ok && at >= 0 && at < (int64_t)n * EPC)
                    sx[slot] = Elem<T>::load_shared(a0 + (uint32_t)at * ES);
                if (flags & kFlagLast) sid_ok[slot] = id_ok ? 1 : 0;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + s * 8);      // the stage first: its next copy can start
            if (flags & kFlagLast) {
                const float2 r = warp_merge(st);
                if (lane == 0) {
                    spart[slot * CW + cw] = r;
                    mbar_arrive(rowdone0 + slot * 8);        // releases this and the logit above
                }
                st.reset();
            }
            if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (failed) {
            if (lane == 0) {
                *end_seq = kEeAborted;
                atomicExch(p.err_word, p.epoch);
            }
            drain_after_error();
        }
    } else {
        // =============================== finishing warp ===============================
        // Takes the rows in the order the producer issued them: merges the consumer warps'
        // pairs, writes the row's log-likelihood and, on a reject, lowers the utterance's
        // first-reject word, then hands the row's slot back to the producer.
        bool failed = false;
        for (int seq = 0;; ++seq) {
            const int slot = seq % NR;
            const uint32_t bar = rowdone0 + slot * 8, par = (uint32_t)((seq / NR) & 1);
            // Sleeps on the row's barrier half a microsecond at a time, looking for the end in
            // between.  (After the last row nothing completes the barrier: the plain wait sat out
            // its time there and the kernel ended 4 us after its last row; and a loop that only
            // tests the barrier keeps a warp spinning on every SM, which under the power cap cost
            // 3 % of the clock.)
            bool got = false;
            const long long t0 = clock64();
            for (;;) {
                got = __all_sync(0xffffffffu, mbar_try_wait_for(bar, par, 500u));
                if (got) break;
                const int e = __shfl_sync(0xffffffffu, (int)*end_seq, 0);
                if (e == kEeAborted || (e >= 0 && seq >= e)) break;
                if (__any_sync(0xffffffffu, clock64() - t0 > kWaitLimitCycles)) { failed = true; break; }
            }
            if (!got) break;
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
                if (!sid_ok[slot]) {
                    fl |= SSD_UTT_BAD_DRAFT_ID;
                    logp = -INFINITY;
                    reject = true;
                } else {
                    logp = (sx[slot] - Mx) - lnS;
                    reject = p.reject_none ? false : (p.reject_all || !(logp > p.log_tau));   // p <= tau; NaN rejects
                }
                if (reject) atomicMin(&p.first_reject[rm.b], rm.pos);
                p.token_logp[rm.row] = logp;
                if (p.row_lse) p.row_lse[rm.row] = lse;
                if (fl) atomicOr(&p.flags[rm.b], fl);
                atomicAdd(&p.rows_read[rm.b], 1);
                mbar_arrive(rowfree0 + slot * 8);
            }
            __syncwarp();
        }
        if (failed && lane == 0) atomicExch(p.err_word, p.epoch);
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
    const int S = plan.stages, NR = ee_row_slots(S);
    size_t o = 2 * (size_t)S * 8 + 2 * (size_t)NR * 8 + S * sizeof(StageDesc) + NR * sizeof(RowMeta) +
               (size_t)NR * plan.warps * 8 + 2 * NR * 4 + 4 + 8;
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
    const int claim_items = ee_claim_items(B, M, plan.ctas);
    cudaError_t e = launch_pdl(ee_init_kernel, 1u, 1024u, 0, L.stream, tok_off, skip, B, M,
                               first_reject, flags, rr, kmax, next_item,
                               2ull * (unsigned long long)plan.ctas * (unsigned long long)claim_items);
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
    p.claim_items = claim_items;
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
    e = launch_pdl(kern, (unsigned)plan.ctas, (unsigned)((plan.warps + 2) * 32), smem, L.stream, p);
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
