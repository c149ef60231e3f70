// Address arithmetic of the bulk-copy kernels: which bytes of the logits a tile (frame
// statistics) or a part of a row (verification, greedy step) is read from, and by which means.
// The functions compile for host and device: the kernels call them when they issue their
// copies, and the library's host-side read-span hooks replay them for any base address and
// shape, so that "no byte outside the matrix is ever read" can be checked without a GPU.
#pragma once

#include <stdint.h>

namespace ssd {
namespace ranges {

#if defined(__CUDACC__)
#define SSD_HD __host__ __device__ __forceinline__
#else
#define SSD_HD inline
#endif

SSD_HD uintptr_t align_down16(uintptr_t a) { return a & ~(uintptr_t)15; }
SSD_HD uintptr_t align_up16(uintptr_t a) { return (a + 15) & ~(uintptr_t)15; }

// ---- frame statistics: one tile = R consecutive rows, fetched as one contiguous range --------
// The tile's bytes are [gstart, gend).  Its 16-byte-aligned superset [f0, c1) is what lands in
// the stage (stage byte 0 holds address f0).  Where that superset would leave the matrix
// [lo_bound, hi_bound) -- at its first tile, its last one, or next to a last tile of a few bytes
// -- the bulk copy is shortened by one chunk on that side and the elements it no longer covers
// are fetched with plain loads.
struct TileReads {
    uintptr_t gstart, gend;     // the tile's own bytes
    uintptr_t f0;               // address that maps to stage byte 0
    uintptr_t bulk_lo, bulk_hi; // bulk copy [bulk_lo, bulk_hi); empty when bulk_hi <= bulk_lo
    uintptr_t head_lo, head_hi; // plain element loads [head_lo, head_hi)
    uintptr_t tail_lo, tail_hi; // plain element loads [tail_lo, tail_hi)
};

SSD_HD TileReads tile_reads(uintptr_t base, int64_t total_bytes, int64_t row_pitch,
                            int64_t row_bytes, int64_t N, int R, int64_t tile) {
    TileReads t;
    const int64_t first_row = tile * R;
    t.gstart = base + (uintptr_t)(first_row * row_pitch);
    t.f0 = align_down16(t.gstart);
    t.head_lo = t.head_hi = t.tail_lo = t.tail_hi = t.gstart;
    if (first_row >= R && first_row + 2 * (int64_t)R <= N) {
        // a whole tile with a whole tile on either side (a tile is never shorter than 16
        // bytes): the superset cannot leave the matrix
        t.gend = t.gstart + (uintptr_t)((int64_t)(R - 1) * row_pitch + row_bytes);
        t.bulk_lo = t.f0;
        t.bulk_hi = align_up16(t.gend);
        return t;
    }
    const uintptr_t lo_bound = base, hi_bound = base + (uintptr_t)total_bytes;
    const int64_t nrows = (N - first_row) < (int64_t)R ? (N - first_row) : (int64_t)R;
    t.gend = t.gstart + (uintptr_t)((nrows - 1) * row_pitch + row_bytes);
    const uintptr_t c1 = align_up16(t.gend);
    t.bulk_lo = t.f0 >= lo_bound ? t.f0 : t.f0 + 16;
    t.bulk_hi = c1 <= hi_bound ? c1 : c1 - 16;
    const bool has_bulk = t.bulk_hi > t.bulk_lo;
    if (!has_bulk) {
        t.bulk_lo = t.bulk_hi = t.gstart;
        t.head_lo = t.gstart;
        t.head_hi = t.gend;
        return t;
    }
    if (t.bulk_lo > t.gstart) {
        t.head_lo = t.gstart;
        t.head_hi = t.bulk_lo < t.gend ? t.bulk_lo : t.gend;
    }
    if (t.bulk_hi < t.gend) {
        t.tail_lo = t.bulk_hi > t.gstart ? t.bulk_hi : t.gstart;
        t.tail_hi = t.gend;
    }
    return t;
}

// ---- verification / greedy step: a row is cut into column spans, a span into parts -----------
// Geometry of one row: its bytes [g0, g1), the aligned start f0, and the number of 16-byte
// chunks of [f0, align_up(g1)).  Chunk 0 is ragged when the row does not start on a 16-byte
// boundary, the last chunk when it does not end on one.
struct RowGeom {
    uintptr_t g0, g1, f0;
    int row_chunks;
    bool head_ragged, tail_ragged;
};
SSD_HD RowGeom row_geom(uintptr_t base, int64_t row, int64_t row_pitch, int64_t row_bytes) {
    RowGeom g;
    g.g0 = base + (uintptr_t)(row * row_pitch);
    g.g1 = g.g0 + (uintptr_t)row_bytes;
    g.f0 = align_down16(g.g0);
    g.row_chunks = (int)((align_up16(g.g1) - g.f0) >> 4);
    g.head_ragged = g.f0 != g.g0;
    g.tail_ragged = (g.g1 & 15) != 0;
    return g;
}

// Span sp of ns: chunks [sc0, sc1), cut into `parts` parts of per_part chunks (the last one may
// be shorter), none larger than max_chunks.  A span without chunks still has one (empty) part.
struct SpanCut {
    int sc0, sc1, parts, per_part;
};
SSD_HD SpanCut span_cut(int row_chunks, int ns, int sp, int max_chunks) {
    SpanCut c;
    const int cps = (row_chunks + ns - 1) / ns;
    c.sc0 = sp * cps < row_chunks ? sp * cps : row_chunks;
    c.sc1 = c.sc0 + cps < row_chunks ? c.sc0 + cps : row_chunks;
    const int span = c.sc1 - c.sc0;
    c.parts = span > 0 ? (span + max_chunks - 1) / max_chunks : 1;
    c.per_part = span > 0 ? (span + c.parts - 1) / c.parts : 0;
    return c;
}

// Part [pc0, pc1) of a row: the bulk copy takes chunks [b0, b1), which lie wholly inside the
// row; a ragged first / last chunk that belongs to the part is instead filled element by
// element (addresses outside [g0, g1) are not read: the stage gets -inf there).
struct PartReads {
    int b0, b1;
    bool head_plain, tail_plain;
};
SSD_HD PartReads part_reads(const RowGeom &g, int pc0, int pc1) {
    PartReads r;
    r.b0 = pc0;
    r.b1 = pc1;
    r.head_plain = g.head_ragged && pc1 > pc0 && pc0 == 0;
    if (r.head_plain) r.b0 = 1;
    r.tail_plain = g.tail_ragged && pc1 > pc0 && pc1 == g.row_chunks &&
                   !(r.b0 == 1 && g.row_chunks == 1);
    if (r.tail_plain) r.b1 = pc1 - 1;
    return r;
}

}  // namespace ranges
}  // namespace ssd
