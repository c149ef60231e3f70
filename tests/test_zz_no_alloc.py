"""ssd_verify_static, the entry point for callers that cannot allocate device memory (a
real-time callback, a sandboxed plugin, a runtime whose memory is handed out before start-up):
its scratch is a fixed array inside the library, so the caller passes inputs and outputs only.

This file is collected last on purpose: a run that stops at the first failure has then already
been through every other test.  The GPU test works on its own in a fresh process (its first
call does the one-time address look-up) and after the rest of the suite.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import helpers as H
from paper_2603_11243_b200 import binding as ssd
from paper_2603_11243_b200 import build as ssd_build
from paper_2603_11243_b200 import synth

RESULTS = ("token_logp", "row_lse", "accepted_len", "all_accepted", "utt_status")


def _result_buffers(M, B, device):
    out = ssd.alloc_verify_outputs(M, B, device, 0)
    del out["workspace"]                      # the point of the call: there is none to pass
    out["token_logp"].fill_(float("nan"))
    return out


@pytest.mark.gpu
def test_static_scratch_matches_ssd_verify_on_two_calls_in_a_row(cuda_device):
    """Different batches, one after the other through the same fixed scratch: each must give the
    oracle's answers (as every other entry point is held to) and reproduce what ssd_verify
    computes with a caller-provided workspace (same kernels, so the floats agree far inside the
    suite's tolerance); a call must not be disturbed by what the one before left behind, also
    when the launch options change how the scratch is laid out.  From the second call on (the
    first looks up the array's address) a call must leave the device's free memory and torch's
    allocator counters exactly as it found them: the entry point exists for callers that cannot
    allocate."""
    from oracle import ref
    dev = cuda_device
    w = synth.scaled(synth.CONFIGS[1], B=5, seed=61)
    batches = [synth.make_verify_batch(w, [17, 0, 33, 8, 21], "cpu"),
               synth.make_verify_batch(synth.scaled(w, seed=62, V_llm=32000), [5, 40, 12, 1, 9], "cpu"),
               synth.make_verify_batch(synth.scaled(w, seed=63), [9, 9, 2, 30, 4], "cpu")]
    skips = [None, torch.tensor([0, 1, 0, 0, 0], dtype=torch.uint8), None]
    options = [None, None, H.opts(split=3, warps=8)]       # column spans: partials laid out anew
    for call, (vb, skip, o) in enumerate(zip(batches, skips, options)):
        x, off, ids = vb.logits.to(dev), vb.tok_off.to(dev), vb.draft_ids.to(dev)
        M, B, V = x.shape[0], off.shape[0] - 1, x.shape[1]
        skip_dev = None if skip is None else skip.to(dev)
        want = ssd.ssd_verify(x, off, ids, w.tau_slm, skip=skip_dev, opts=o)
        bufs = _result_buffers(M, B, dev)
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info(dev)[0]
        stats0 = torch.cuda.memory_stats(dev)
        got = ssd.ssd_verify_static(x, off, ids, w.tau_slm, bufs, skip=skip_dev, opts=o)
        torch.cuda.synchronize()
        if call > 0:
            assert torch.cuda.mem_get_info(dev)[0] == free0, "device memory changed hands"
            stats1 = torch.cuda.memory_stats(dev)
            for key in ("allocation.all.allocated", "segment.all.allocated",
                        "allocated_bytes.all.allocated", "reserved_bytes.all.allocated"):
                assert stats1[key] == stats0[key], key
        sk = None if skip is None else skip.numpy()
        orc = ref.verify(H.storage_numpy(vb.logits), V, vb.tok_off.numpy(), vb.draft_ids.numpy(),
                         float(np.float32(w.tau_slm)), skip=sk)
        H.compare_stage2(got, orc, vb.tok_off.numpy(), w.tau_slm, skip=sk)
        skb = np.zeros(B, bool) if skip is None else skip.numpy().astype(bool)
        rows = np.concatenate([np.arange(int(vb.tok_off[b]), int(vb.tok_off[b + 1]))
                               for b in range(B) if not skb[b]]).astype(np.int64)
        for k in ("token_logp", "row_lse"):
            a, b = got[k].cpu().numpy()[rows], want[k].cpu().numpy()[rows]
            assert np.abs(a.astype(np.float64) - b).max() <= H.FLOAT_TOL, k
        for k in ("accepted_len", "all_accepted", "utt_status"):
            np.testing.assert_array_equal(got[k].cpu().numpy(), want[k].cpu().numpy(), err_msg=k)
        # rows of a skipped utterance stay untouched by both entry points
        skipped_rows = np.setdiff1d(np.arange(M), rows)
        assert np.isnan(got["token_logp"].cpu().numpy()[skipped_rows]).all()


def test_sizes_beyond_the_fixed_scratch_are_refused_before_any_cuda_call():
    """The size check comes first, on the host: it needs no GPU and touches none of the
    pointers."""
    ssd_build.build()
    lib = ssd.lib()
    p = C.c_void_p
    rows_that_fit = (ssd.VERIFY_STATIC_SCRATCH_BYTES - 256 - 256) // (16 * 8)
    assert ssd.ssd_verify_workspace_bytes(4, rows_that_fit, 1000, ssd.BF16) <= ssd.VERIFY_STATIC_SCRATCH_BYTES
    too_many = rows_that_fit + 1
    rc = lib.ssd_verify_static(p(8), ssd.BF16, 1000, 1000, p(8), p(8), 4, too_many, C.c_float(0.1),
                               None, p(8), p(8), p(8), p(8), p(8), None, None)
    assert rc == ssd.ERR_TOO_LARGE
    assert b"SSD_ERR_TOO_LARGE" in lib.ssd_status_string(rc)
    # argument errors are reported as for ssd_verify
    assert lib.ssd_verify_static(p(8), 5, 1000, 1000, p(8), p(8), 4, 10, C.c_float(0.1), None,
                                 p(8), p(8), p(8), p(8), p(8), None, None) == ssd.ERR_DTYPE
    assert lib.ssd_verify_static(p(8), ssd.BF16, 1000, 999, p(8), p(8), 4, 10, C.c_float(0.1), None,
                                 p(8), p(8), p(8), p(8), p(8), None, None) == ssd.ERR_ARG
