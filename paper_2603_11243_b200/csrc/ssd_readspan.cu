// Host-side replay of the bulk-copy kernels' address arithmetic (ssd_ranges.cuh): for a logits
// matrix that would start at a given address, which bytes would be read, do the reads of every
// tile / row part cover its bytes exactly, and do they stay inside the matrix and the stage.
// Nothing is dereferenced and no GPU is needed; the tests sweep shapes and misalignments.
#include "ssd_common.cuh"
#include "ssd_ranges.cuh"

using namespace ssd;

namespace {

struct Span {
    uint64_t lo = ~0ull, hi = 0;
    int64_t faults = 0;
    void add(uintptr_t a, uintptr_t b) {
        if (b <= a) return;
        if (a < lo) lo = a;
        if (b > hi) hi = b;
    }
};

}  // namespace

extern "C" {

int32_t ssd_ctc_draft_read_span(uint64_t base_addr, ssd_dtype dtype, int32_t V, int64_t ld,
                                int64_t N, const ssd_launch_opts *opts, ssd_read_span *out) {
    if (!out) return SSD_ERR_NULL;
    if (dtype != SSD_F32 && dtype != SSD_BF16) return SSD_ERR_DTYPE;
    if (N < 0 || V < 1 || ld < V) return SSD_ERR_ARG;
    const int es = dtype == SSD_F32 ? 4 : 2;
    if (base_addr % es) return SSD_ERR_ALIGN;
    PlanReplay replay;      // no device here: the plans use the SM count they are tuned for
    CtcPlan plan;
    const int rc = plan_ctc(dtype, V, ld, N, 0, opts, &plan);
    if (rc != SSD_OK) return rc;
    const int64_t row_pitch = ld * es, row_bytes = (int64_t)V * es;
    const int64_t total = N > 0 ? (N - 1) * row_pitch + row_bytes : 0;
    const uintptr_t base = (uintptr_t)base_addr;
    Span sp;
    if (plan.kernel == 2) {
        for (int64_t tile = 0; tile < plan.num_tiles; ++tile) {
            const ranges::TileReads t =
                ranges::tile_reads(base, total, row_pitch, row_bytes, N, plan.rows_per_tile, tile);
            bool ok = t.gstart >= base && t.gend <= base + (uintptr_t)total && t.gend > t.gstart;
            const bool bulk = t.bulk_hi > t.bulk_lo, head = t.head_hi > t.head_lo,
                       tail = t.tail_hi > t.tail_lo;
            // every read inside the matrix; the bulk copy on 16-byte boundaries; all of it
            // inside the stage, whose byte 0 is address f0
            const uintptr_t ends[3][2] = {{t.bulk_lo, t.bulk_hi}, {t.head_lo, t.head_hi},
                                          {t.tail_lo, t.tail_hi}};
            for (int i = 0; i < 3; ++i) {
                if (ends[i][1] <= ends[i][0]) continue;
                ok = ok && ends[i][0] >= base && ends[i][1] <= base + (uintptr_t)total;
                ok = ok && ends[i][0] >= t.f0 &&
                     ends[i][1] - t.f0 <= (uintptr_t)plan.stage_stride;
                sp.add(ends[i][0], ends[i][1]);
            }
            if (bulk) ok = ok && (t.bulk_lo % 16 == 0) && (t.bulk_hi % 16 == 0);
            if (head) ok = ok && (t.head_lo - t.gstart) % es == 0 && (t.head_hi - t.gstart) % es == 0;
            if (tail) ok = ok && (t.tail_lo - t.gstart) % es == 0 && (t.tail_hi - t.gstart) % es == 0;
            // head, bulk, tail in this order, without gaps or overlaps, cover [gstart, gend)
            uintptr_t at = t.gstart;
            if (head) {
                ok = ok && t.head_lo == at;
                if (bulk) ok = ok && t.head_hi == (t.bulk_lo < t.gend ? t.bulk_lo : t.gend);
                at = t.head_hi;
            }
            if (bulk) {
                ok = ok && t.bulk_lo <= at && t.bulk_hi > at;
                at = t.bulk_hi < t.gend ? t.bulk_hi : t.gend;
            }
            if (tail) { ok = ok && t.tail_lo == at; at = t.tail_hi; }
            ok = ok && at == t.gend;
            if (!ok) ++sp.faults;
        }
    } else if (N > 0) {
        sp.add(base, base + (uintptr_t)total);   // element-wise loads of the rows' own bytes
    }
    out->lo = sp.hi ? sp.lo : base_addr;
    out->hi = sp.hi ? sp.hi : base_addr;
    out->faults = sp.faults;
    out->kernel = plan.kernel;
    out->reserved = 0;
    return SSD_OK;
}

int32_t ssd_verify_read_span(uint64_t base_addr, ssd_dtype dtype, int32_t V, int64_t ld,
                             int64_t M, int32_t B, const ssd_launch_opts *opts,
                             ssd_read_span *out) {
    if (!out) return SSD_ERR_NULL;
    if (dtype != SSD_F32 && dtype != SSD_BF16) return SSD_ERR_DTYPE;
    if (B < 0 || M < 0 || V < 1 || ld < V) return SSD_ERR_ARG;
    const int es = dtype == SSD_F32 ? 4 : 2;
    if (base_addr % es) return SSD_ERR_ALIGN;
    PlanReplay replay;
    VerifyPlan plan;
    const int rc = plan_verify(B, M, V, dtype, opts, &plan);
    if (rc != SSD_OK) return rc;
    const int64_t row_pitch = ld * es, row_bytes = (int64_t)V * es;
    const uintptr_t base = (uintptr_t)base_addr;
    Span sp;
    if (plan.kernel == 2) {
        const int max_chunks = plan.stage_bytes >> 4;
        for (int64_t row = 0; row < M; ++row) {
            const ranges::RowGeom g = ranges::row_geom(base, row, row_pitch, row_bytes);
            int next_chunk = 0;        // spans and parts must tile [0, row_chunks) in order
            bool ok = true;
            for (int s = 0; s < plan.split; ++s) {
                const ranges::SpanCut c = ranges::span_cut(g.row_chunks, plan.split, s, max_chunks);
                ok = ok && c.sc0 == next_chunk && c.sc1 >= c.sc0 && c.parts >= 1;
                for (int part = 0; part < c.parts; ++part) {
                    const int pc0 = c.sc0 + part * c.per_part;
                    const int pc1 = c.sc1 < pc0 + c.per_part ? c.sc1 : pc0 + c.per_part;
                    if (c.sc1 == c.sc0) { ok = ok && c.parts == 1; break; }   // empty span
                    ok = ok && pc0 == next_chunk && pc1 > pc0 && pc1 - pc0 <= max_chunks;
                    const ranges::PartReads r = ranges::part_reads(g, pc0, pc1);
                    // the bulk copy plus the element-wise first / last chunk cover the part
                    ok = ok && (r.b0 == pc0 || (r.head_plain && r.b0 == pc0 + 1));
                    ok = ok && (r.b1 == pc1 || (r.tail_plain && r.b1 == pc1 - 1));
                    if (r.b1 > r.b0) {
                        const uintptr_t lo = g.f0 + ((uintptr_t)r.b0 << 4), hi = g.f0 + ((uintptr_t)r.b1 << 4);
                        ok = ok && lo >= g.g0 && hi <= g.g1;      // never leaves the row
                        sp.add(lo, hi);
                    }
                    // element-wise chunks read only addresses inside [g0, g1)
                    if (r.head_plain) sp.add(g.g0, g.g1 < g.f0 + 16 ? g.g1 : g.f0 + 16);
                    if (r.tail_plain) {
                        const uintptr_t c0 = g.f0 + ((uintptr_t)(pc1 - 1) << 4);
                        sp.add(c0 > g.g0 ? c0 : g.g0, g.g1);
                    }
                    next_chunk = pc1;
                }
                if (c.sc1 > c.sc0) ok = ok && next_chunk == c.sc1;
            }
            ok = ok && next_chunk == g.row_chunks;
            if (!ok) ++sp.faults;
        }
    } else if (M > 0) {
        sp.add(base, base + (uintptr_t)((M - 1) * row_pitch + row_bytes));
    }
    out->lo = sp.hi ? sp.lo : base_addr;
    out->hi = sp.hi ? sp.hi : base_addr;
    out->faults = sp.faults;
    out->kernel = plan.kernel;
    out->reserved = 0;
    return SSD_OK;
}

}  // extern "C"
