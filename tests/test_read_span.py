"""Memory safety of the bulk-copy kernels' reads, checked on the host.

The kernels fetch 16-byte-aligned ranges although rows may start at any element; the library's
read-span hooks replay the kernels' own address arithmetic (one header shared by both) for a
matrix at any address.  For every shape and misalignment below: no tile / row part breaks a rule
(faults == 0) and the union of all reads is exactly the matrix's own extent -- nothing before its
first logit, nothing past its last one, nothing left out at the ends."""
import itertools

import pytest

from paper_2603_11243_b200 import binding as ssd

BASE = 0x7F0000000000          # any 16-byte-aligned address; nothing is dereferenced


def _extent(rows, ld, V, es):
    return ((rows - 1) * ld + V) * es


VS = (1, 2, 3, 5, 7, 8, 9, 15, 16, 17, 31, 33, 129, 348, 1025, 4097)
NS = tuple(range(1, 41)) + (63, 64, 65, 100, 1000, 4095, 4096, 4097, 4099, 8191, 8192, 8193,
                            12289, 14674)


@pytest.mark.parametrize("dtype,es", [(ssd.F32, 4), (ssd.BF16, 2)])
def test_ctc_reads_stay_inside_the_matrix(dtype, es):
    checked_bulk = 0
    for V in VS:
        for pad in (0, 1, 3, 8):
            ld = V + pad
            for N in NS:
                for mis in range(0, 16, es) if N < 50 else (0, es, 16 - es):
                    base = BASE + mis
                    r = ssd.ssd_ctc_draft_read_span(base, dtype, V, ld, N)
                    assert r.faults == 0, (V, ld, N, mis)
                    assert r.lo == base and r.hi == base + _extent(N, ld, V, es), (V, ld, N, mis)
                    checked_bulk += r.kernel == 2
    assert checked_bulk > 1000          # the sweep really exercised the bulk-copy kernel


def test_ctc_reads_with_forced_shapes():
    # small stages, many warps, the shapes the launch options can force
    for V, N in itertools.product((1, 3, 129, 1025), (1, 5, 33, 1000, 4097)):
        for stage_bytes, stages, warps in ((1, 1, 1), (1, 8, 24), (64, 2, 3), (100000, 1, 24)):
            o = ssd.LaunchOpts()
            o.stage_bytes, o.stages, o.warps = stage_bytes, stages, warps
            for mis in (0, 2, 6, 14):
                try:
                    r = ssd.ssd_ctc_draft_read_span(BASE + mis, ssd.BF16, V, V + 1, N, o)
                except ssd.SsdError:
                    continue                       # a shape the library refuses
                assert r.faults == 0 and r.lo == BASE + mis
                assert r.hi == BASE + mis + _extent(N, V + 1, V, 2)


@pytest.mark.parametrize("dtype,es", [(ssd.F32, 4), (ssd.BF16, 2)])
def test_verify_reads_stay_inside_each_row(dtype, es):
    checked_bulk = 0
    for V in (1, 2, 7, 8, 9, 33, 1000, 4097, 32000, 49152, 49153, 100352, 152064, 152065):
        for pad in (0, 1, 5):
            ld = V + pad
            for M in (1, 2, 3, 17, 148, 149, 1200):
                if V > 50000 and M > 149:
                    continue
                for mis in range(0, 16, es) if M < 20 else (0, es):
                    base = BASE + mis
                    r = ssd.ssd_verify_read_span(base, dtype, V, ld, M, B=3)
                    assert r.faults == 0, (V, ld, M, mis)
                    assert r.lo == base and r.hi == base + _extent(M, ld, V, es), (V, ld, M, mis)
                    checked_bulk += r.kernel == 2
    assert checked_bulk > 300


def test_verify_reads_with_forced_shapes():
    for V, M in itertools.product((7, 1025, 49153), (1, 5, 300)):
        for split, stage_bytes, warps in ((1, 1024, 4), (3, 4096, 16), (7, 1024, 8), (64, 2048, 12),
                                          (2, 65536, 16)):
            o = ssd.LaunchOpts()
            o.split, o.stage_bytes, o.warps = split, stage_bytes, warps
            for mis in (0, 2, 10):
                r = ssd.ssd_verify_read_span(BASE + mis, ssd.BF16, V, V + 3, M, 2, o)
                assert r.faults == 0 and r.lo == BASE + mis
                assert r.hi == BASE + mis + _extent(M, V + 3, V, 2)


def test_read_span_argument_errors():
    with pytest.raises(ssd.SsdError):
        ssd.ssd_ctc_draft_read_span(BASE + 1, ssd.BF16, 8, 8, 4)        # off the element size
    with pytest.raises(ssd.SsdError):
        ssd.ssd_verify_read_span(BASE, ssd.F32, 8, 7, 4)                # ld < V
    with pytest.raises(ssd.SsdError):
        ssd.ssd_ctc_draft_read_span(BASE, 7, 8, 8, 4)                   # bad dtype
    r = ssd.ssd_ctc_draft_read_span(BASE, ssd.F32, 8, 8, 0)             # nothing to read
    assert r.faults == 0 and r.lo == r.hi == BASE
