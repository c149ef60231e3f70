"""The C-ABI library: it loads, exports every symbol the header declares, and turns bad
arguments into error codes on the host (no GPU needed: these calls return before any launch)."""
import ctypes as C
import os
import re

import pytest

from paper_2603_11243_b200 import binding as ssd
from paper_2603_11243_b200 import build as ssd_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ssd_build.build()
    return ssd.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ssd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ssd_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"ssd_ctc_draft", "ssd_entropy_gate", "ssd_verify"} <= set(names)
    for n in names:
        assert hasattr(lib, n), "libssd.so does not export " + n


def test_status_strings(lib):
    assert lib.ssd_status_string(0) == b"SSD_OK"
    for code in range(1, 7):
        assert lib.ssd_status_string(code).startswith(b"SSD_ERR_")
    assert lib.ssd_version() >= 100


def _ctc(lib, logits=8, dtype=1, V=10, ld=10, off=8, B=1, N=4, blank=0, cap=5, outs=8, ws=0,
         ws_bytes=0):
    p = C.c_void_p
    o = p(outs) if outs else None
    return lib.ssd_ctc_draft(p(logits) if logits else None, dtype, V, ld, p(off) if off else None,
                             B, N, blank, cap, o, o, o, None, o, o, o, o, o, o,
                             p(ws) if ws else None, ws_bytes, None, None)


def test_ctc_draft_rejects_bad_arguments_on_the_host(lib):
    assert _ctc(lib, dtype=7) == ssd.ERR_DTYPE
    assert _ctc(lib, V=0) == ssd.ERR_ARG
    assert _ctc(lib, ld=9) == ssd.ERR_ARG
    assert _ctc(lib, B=-1) == ssd.ERR_ARG
    assert _ctc(lib, N=-1) == ssd.ERR_ARG
    assert _ctc(lib, blank=10) == ssd.ERR_ARG
    assert _ctc(lib, blank=-1) == ssd.ERR_ARG
    assert _ctc(lib, cap=-1) == ssd.ERR_ARG
    assert _ctc(lib, logits=0) == ssd.ERR_NULL
    assert _ctc(lib, off=0) == ssd.ERR_NULL
    assert _ctc(lib, outs=0) == ssd.ERR_NULL
    assert _ctc(lib, logits=9, dtype=1) == ssd.ERR_ALIGN     # bf16 at an odd address
    assert _ctc(lib, logits=10, dtype=0) == ssd.ERR_ALIGN    # fp32 at 2 mod 4
    assert _ctc(lib, ws=256, ws_bytes=2047) == ssd.ERR_WORKSPACE     # 2048 bytes needed
    assert _ctc(lib, ws=264, ws_bytes=4096) == ssd.ERR_WORKSPACE     # not 256-byte aligned


def _verify(lib, logits=8, dtype=1, V=10, ld=10, off=8, ids=8, B=1, M=4, outs=8, ws=256, ws_bytes=1 << 20):
    p = C.c_void_p
    o = p(outs) if outs else None
    return lib.ssd_verify(p(logits) if logits else None, dtype, V, ld, p(off) if off else None,
                          p(ids) if ids else None, B, M, C.c_float(0.1), None, o, o, o, o, o,
                          p(ws) if ws else None, ws_bytes, None, None)


def test_verify_rejects_bad_arguments_on_the_host(lib):
    assert _verify(lib, dtype=2) == ssd.ERR_DTYPE
    assert _verify(lib, V=0) == ssd.ERR_ARG
    assert _verify(lib, ld=3) == ssd.ERR_ARG
    assert _verify(lib, M=-2) == ssd.ERR_ARG
    assert _verify(lib, B=-2) == ssd.ERR_ARG
    assert _verify(lib, logits=0) == ssd.ERR_NULL
    assert _verify(lib, ids=0) == ssd.ERR_NULL
    assert _verify(lib, off=0) == ssd.ERR_NULL
    assert _verify(lib, outs=0) == ssd.ERR_NULL
    assert _verify(lib, logits=7) == ssd.ERR_ALIGN
    assert _verify(lib, ws=0) == ssd.ERR_WORKSPACE
    assert _verify(lib, ws_bytes=16) == ssd.ERR_WORKSPACE
    assert _verify(lib, ws=264) == ssd.ERR_WORKSPACE           # not 256-byte aligned


def test_verify_rejects_bad_options(lib):
    o = ssd.LaunchOpts()
    o.kernel = 9
    p = C.c_void_p
    rc = lib.ssd_verify(p(8), 1, 10, 10, p(8), p(8), 1, 4, C.c_float(0.1), None, p(8), p(8), p(8),
                        p(8), p(8), p(256), 1 << 20, None, C.byref(o))
    assert rc == ssd.ERR_ARG
    o.kernel, o.stage_bytes = 2, 1000     # not a multiple of 128
    rc = lib.ssd_verify(p(8), 1, 10, 10, p(8), p(8), 1, 4, C.c_float(0.1), None, p(8), p(8), p(8),
                        p(8), p(8), p(256), 1 << 20, None, C.byref(o))
    assert rc == ssd.ERR_ARG


def test_gate_rejects_bad_arguments_on_the_host(lib):
    p = C.c_void_p
    g = lambda *a: lib.ssd_entropy_gate(*a)
    assert g(p(8), p(8), -1, 4, C.c_float(0.5), p(8), p(8), None, None, None, None) == ssd.ERR_ARG
    assert g(None, p(8), 1, 4, C.c_float(0.5), p(8), p(8), None, None, None, None) == ssd.ERR_NULL
    assert g(p(8), None, 1, 4, C.c_float(0.5), p(8), p(8), None, None, None, None) == ssd.ERR_NULL
    assert g(p(8), p(8), 1, 4, C.c_float(0.5), None, p(8), None, None, None, None) == ssd.ERR_NULL
    # the form that reads utterance maxima needs their status words as well
    assert g(None, None, 1, 0, C.c_float(0.5), p(8), p(8), None, p(8), None, None) == ssd.ERR_NULL
    assert g(None, None, 1, 0, C.c_float(0.5), None, p(8), None, p(8), p(8), None) == ssd.ERR_NULL


def test_workspace_queries(lib):
    assert ssd.ssd_ctc_draft_workspace_bytes(32, 16000, 1025, ssd.BF16) == 2048
    small = ssd.ssd_verify_workspace_bytes(1, 250, 152064, ssd.BF16)
    big = ssd.ssd_verify_workspace_bytes(32, 6400, 49152, ssd.BF16)
    assert small >= 256 + 250 * 8 * 8 and big >= 256 + 6400 * 8 * 8
    o = ssd.LaunchOpts()
    o.split, o.warps = 4, 8
    # header, two words per utterance (rounded to 256 bytes), 8-byte pairs per row, span and warp
    assert ssd.ssd_verify_workspace_bytes(32, 6400, 49152, ssd.BF16, o) == 256 + 512 + 6400 * 4 * 8 * 8


def test_binding_refuses_host_tensors(lib):
    import torch
    x = torch.zeros((4, 8), dtype=torch.float32)
    off = torch.tensor([0, 4], dtype=torch.int64)
    with pytest.raises(ValueError):
        ssd.ssd_ctc_draft(x, off, 0, 4)


def test_sweep_assemble_greedy_reject_bad_arguments_on_the_host(lib):
    p = C.c_void_p
    f = (C.c_float * 2)(0.5, 0.1)
    fp = C.cast(f, C.c_void_p)
    sw = lib.ssd_threshold_sweep
    assert sw(p(8), p(8), p(8), -1, 4, fp, fp, 2, p(8), p(8), p(8), None, None) == ssd.ERR_ARG
    assert sw(p(8), p(8), p(8), 2, 4, fp, fp, -1, p(8), p(8), p(8), None, None) == ssd.ERR_ARG
    assert sw(p(8), p(8), None, 2, 4, fp, fp, 2, p(8), p(8), p(8), None, None) == ssd.ERR_NULL
    assert sw(p(8), p(8), p(8), 2, 4, None, fp, 2, p(8), p(8), p(8), None, None) == ssd.ERR_NULL
    assert sw(None, p(8), p(8), 2, 4, fp, fp, 2, p(8), p(8), p(8), None, None) == ssd.ERR_NULL
    assert sw(p(8), None, p(8), 2, 4, fp, fp, 2, p(8), p(8), p(8), None, None) == ssd.ERR_NULL
    assert sw(p(8), p(8), p(8), 2, 4, fp, fp, 2, p(8), None, p(8), None, None) == ssd.ERR_NULL
    asm = lib.ssd_assemble
    a = [p(8)] * 2 + [3, 9] + [p(8)] * 9 + [None]
    bad = list(a); bad[2] = -1
    assert asm(*bad) == ssd.ERR_ARG
    for i in (1, 4, 5, 6, 8, 9, 10, 11, 12):
        bad = list(a); bad[i] = None
        assert asm(*bad) == ssd.ERR_NULL, i
    gs = lib.ssd_greedy_step
    ok = [p(8), ssd.BF16, 100, 100, 5, p(8), p(8), p(8), p(8), p(256), 1 << 20, None, None]
    for i, v, code in ((1, 9, ssd.ERR_DTYPE), (2, 0, ssd.ERR_ARG), (3, 99, ssd.ERR_ARG),
                       (4, -1, ssd.ERR_ARG), (0, None, ssd.ERR_NULL), (5, None, ssd.ERR_NULL),
                       (0, p(7), ssd.ERR_ALIGN), (9, None, ssd.ERR_WORKSPACE),
                       (10, 16, ssd.ERR_WORKSPACE), (9, p(264), ssd.ERR_WORKSPACE)):
        bad = list(ok); bad[i] = v
        assert gs(*bad) == code, (i, v)
    o = ssd.LaunchOpts()
    o.kernel = 1
    bad = list(ok); bad[12] = C.byref(o)
    assert gs(*bad) == ssd.ERR_ARG
    assert ssd.ssd_greedy_step_workspace_bytes(16, 152064, ssd.BF16) >= 256 + 16 * 16 * 12


def test_early_exit_rejects_bad_arguments_on_the_host(lib):
    p = C.c_void_p
    ee = lib.ssd_verify_early_exit
    ok = [p(8), ssd.BF16, 100, 100, p(8), p(8), 2, 40, C.c_float(0.1), None, p(8), p(8), p(8), p(8),
          p(8), None, p(256), 1 << 20, None, None]
    for i, v, code in ((1, 4, ssd.ERR_DTYPE), (2, 0, ssd.ERR_ARG), (3, 50, ssd.ERR_ARG),
                       (6, -1, ssd.ERR_ARG), (7, -1, ssd.ERR_ARG), (0, None, ssd.ERR_NULL),
                       (4, None, ssd.ERR_NULL), (5, None, ssd.ERR_NULL), (10, None, ssd.ERR_NULL),
                       (12, None, ssd.ERR_NULL), (0, p(7), ssd.ERR_ALIGN),
                       (16, None, ssd.ERR_WORKSPACE), (17, 64, ssd.ERR_WORKSPACE),
                       (16, p(257), ssd.ERR_WORKSPACE)):
        bad = list(ok); bad[i] = v
        assert ee(*bad) == code, (i, v)
    full = ssd.ssd_verify_workspace_bytes(64, 20000, 49152, ssd.BF16)
    assert ssd.ssd_verify_early_exit_workspace_bytes(64, 20000, 49152, ssd.BF16) >= full


def test_vocab_parallel_calls_reject_bad_arguments_on_the_host(lib):
    p = lambda n: C.c_void_p(n)
    f32 = C.c_float(0.1)
    sh = lambda logits, dtype, V, ld, col0, off, ids, B, M, stats, ws, wsb: lib.ssd_verify_shard(
        logits, dtype, V, ld, col0, off, ids, B, M, None, stats, ws, wsb, None, None)
    assert sh(p(8), 9, 10, 10, 0, p(8), p(8), 1, 4, p(8), p(256), 1 << 20) == ssd.ERR_DTYPE
    assert sh(p(8), 1, 10, 9, 0, p(8), p(8), 1, 4, p(8), p(256), 1 << 20) == ssd.ERR_ARG     # ld < V
    assert sh(p(8), 1, 10, 10, -1, p(8), p(8), 1, 4, p(8), p(256), 1 << 20) == ssd.ERR_ARG   # col0 < 0
    assert sh(p(8), 1, 10, 10, 0, None, p(8), 1, 4, p(8), p(256), 1 << 20) == ssd.ERR_NULL
    assert sh(p(8), 1, 10, 10, 0, p(8), p(8), 1, 4, None, p(256), 1 << 20) == ssd.ERR_NULL
    assert sh(p(9), 1, 10, 10, 0, p(8), p(8), 1, 4, p(8), p(256), 1 << 20) == ssd.ERR_ALIGN
    assert sh(p(8), 1, 10, 10, 0, p(8), p(8), 1, 4, p(8), p(256), 16) == ssd.ERR_WORKSPACE
    assert sh(p(8), 1, 10, 10, 0, p(8), p(8), 0, 0, p(8), None, 0) == ssd.OK                # nothing to do
    cb = lambda stats, R, V, off, ids, B, M, lp, al, aa, st: lib.ssd_verify_combine(
        stats, R, V, off, ids, B, M, f32, None, lp, None, al, aa, st, None)
    assert cb(p(8), 0, 10, p(8), p(8), 1, 4, p(8), p(8), p(8), p(8)) == ssd.ERR_ARG          # R < 1
    assert cb(p(8), 2, 0, p(8), p(8), 1, 4, p(8), p(8), p(8), p(8)) == ssd.ERR_ARG           # V < 1
    assert cb(None, 2, 10, p(8), p(8), 1, 4, p(8), p(8), p(8), p(8)) == ssd.ERR_NULL
    assert cb(p(8), 2, 10, p(8), p(8), 1, 4, p(8), None, p(8), p(8)) == ssd.ERR_NULL
    assert cb(p(8), 2, 10, p(8), p(8), 0, 0, p(8), p(8), p(8), p(8)) == ssd.OK

