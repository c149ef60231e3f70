"""GPU parity of stage 2 (ssd_verify) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import helpers as H
from oracle import ref
from paper_2603_11243_b200 import binding as ssd
from paper_2603_11243_b200 import synth

pytestmark = pytest.mark.gpu

# plain loads; bulk copies with rows finished inside the streaming kernel; bulk copies with the
# closing kernel of its own
KERNELS = {"plain": dict(kernel=1), "tma": dict(kernel=2, finish=2, split=1),
           "tma_closing": dict(kernel=2, finish=1)}


def _kopts(kernel, okw):
    k = dict(kernel) if isinstance(kernel, dict) else {"kernel": kernel}
    k.update(okw)
    return k


def run_verify(logits_dev, tok_off, draft_ids, V, tau, skip=None, guard=True, **okw):
    dev = logits_dev.device
    M, B = logits_dev.shape[0], len(tok_off) - 1
    o = H.opts(**okw)
    code = ssd.BF16 if logits_dev.dtype == torch.bfloat16 else ssd.F32
    ws = ssd.ssd_verify_workspace_bytes(B, M, V, code, o)
    if guard:
        g, out = H.guarded_verify_outputs(M, B, dev, ws)
    else:
        g, out = None, ssd.alloc_verify_outputs(M, B, dev, ws)
    out["token_logp"].fill_(float("nan"))
    skip_dev = None if skip is None else torch.as_tensor(skip, dtype=torch.uint8).to(dev)
    ssd.ssd_verify(logits_dev, tok_off.to(dev), draft_ids.to(dev), tau, skip=skip_dev, V=V,
                   out=out, opts=o)
    torch.cuda.synchronize()
    if g:
        g.check()
    return out


def check_verify(w, K, device, kernel, skip=None, require_all_margins=True, **okw):
    vb = synth.make_verify_batch(w, K, "cpu")
    out = run_verify(vb.logits.to(device), vb.tok_off, vb.draft_ids, w.V_llm, w.tau_slm,
                     skip=skip, **_kopts(kernel, okw))
    orc = ref.verify(H.storage_numpy(vb.logits), w.V_llm, vb.tok_off.numpy(),
                     vb.draft_ids.numpy(), float(np.float32(w.tau_slm)), skip=skip)
    H.compare_stage2(out, orc, vb.tok_off.numpy(), w.tau_slm, skip=skip,
                     require_all_margins=require_all_margins)
    return vb, out, orc


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
def test_config0_tiny_planted_reject(cuda_device, kernel):
    w = synth.CONFIGS[0]
    vb, out, orc = check_verify(w, [37], cuda_device, kernel)
    # anchored generator: the planted position is the first reject
    assert int(orc["accepted_len"][0]) == int(vb.planted_reject[0])


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
@pytest.mark.parametrize("variant", ["anchored", "literal"])
def test_config1_reduced_batch(cuda_device, kernel, variant):
    """Configuration 1's verify generator (V = 49,152 bf16) on 6 utterances of ragged length,
    one of them empty."""
    w = synth.scaled(synth.CONFIGS[1], B=6, variant=variant)
    K = [23, 0, 57, 1, 40, 12]
    vb, out, orc = check_verify(w, K, cuda_device, kernel,
                                require_all_margins=(variant == "anchored"))
    if variant == "anchored":
        want = [int(p) if p >= 0 else k for p, k in zip(vb.planted_reject.tolist(), K)]
        assert list(orc["accepted_len"]) == want
        assert len(set(orc["all_accepted"])) == 2      # both outcomes occur


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
def test_gate_skip_mask(cuda_device, kernel):
    """Utterances the gate accepted are not read: their token_logp stays untouched."""
    w = synth.scaled(synth.CONFIGS[2], B=5, V_llm=100352)
    K = [9, 14, 3, 20, 6]
    skip = np.array([1, 0, 1, 0, 0], np.uint8)
    vb, out, orc = check_verify(w, K, cuda_device, kernel, skip=skip)
    lp = out["token_logp"].cpu().numpy()
    assert np.isnan(lp[:9]).all() and np.isnan(lp[23:26]).all() and not np.isnan(lp[9:23]).any()


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 2, 5, 8, 17, 1000, 4099, 32000, 50001, 152064])
def test_vocabulary_sizes(cuda_device, kernel, dtype, V):
    w = synth.scaled(synth.CONFIGS[1], B=3, V_llm=V, dtype=dtype, seed=200 + V % 97,
                     variant="literal", tau_slm=0.1)
    check_verify(w, [5, 9, 2], cuda_device, kernel, require_all_margins=False)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("split", [1, 2, 3, 7, 64])
def test_column_spans(cuda_device, dtype, split):
    """Rows cut into column spans (used when there are few rows): same results."""
    w = synth.scaled(synth.CONFIGS[1], B=3, V_llm=49152 + 40, dtype=dtype, seed=31)
    check_verify(w, [4, 7, 2], cuda_device, 2, split=split)
    check_verify(w, [4, 7, 2], cuda_device, 1, split=split)


@pytest.mark.parametrize("warps,stages,stage_bytes,ctas", [(4, 2, 4096, 3), (16, 3, 65536, 148),
                                                            (8, 12, 16384, 7), (1, 16, 1024, 1)])
def test_pipeline_shapes(cuda_device, warps, stages, stage_bytes, ctas):
    w = synth.scaled(synth.CONFIGS[1], B=4, V_llm=32000, seed=17)
    for extra in (dict(finish=1), dict(finish=2, split=1)):
        check_verify(w, [11, 3, 8, 5], cuda_device, 2, warps=warps, stages=stages,
                     stage_bytes=stage_bytes, ctas=ctas, **extra)


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_padded_rows_and_misaligned_base(cuda_device, kernel, dtype):
    """ld > V with a row pitch that is not a multiple of 16 bytes and a base that is only
    element-aligned: rows start and end inside 16-byte chunks."""
    V, ld = 5003, 5011
    w = synth.scaled(synth.CONFIGS[1], B=3, V_llm=ld, dtype=dtype, seed=41, variant="literal")
    vb = synth.make_verify_batch(w, [6, 1, 9], "cpu")
    ids = (vb.draft_ids % V).to(torch.int32)
    wide = vb.logits.to(cuda_device)
    out = run_verify(wide[:, 5:5 + V], vb.tok_off, ids, V, 0.1, **kernel)
    orc = ref.verify(H.storage_numpy(vb.logits[:, 5:5 + V].contiguous()), V, vb.tok_off.numpy(),
                     ids.numpy(), float(np.float32(0.1)))
    H.compare_stage2(out, orc, vb.tok_off.numpy(), 0.1, require_all_margins=False)


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
def test_bad_draft_ids_nonfinite_rows_and_thresholds(cuda_device, kernel):
    V = 300
    g = torch.Generator().manual_seed(8)
    x = torch.randn((10, V), generator=g)
    ids = torch.randint(0, V, (10,), generator=g, dtype=torch.int32)
    for i in range(10):
        x[i, ids[i]] += 12.0
    off = torch.tensor([0, 3, 6, 10], dtype=torch.int64)
    bad = ids.clone()
    bad[4] = V          # utterance 1, position 1: out of range -> reject there, never read
    bad[7] = -1         # utterance 2, position 1
    x2 = x.clone()
    x2[0, 3] = float("nan")   # utterance 0, row 0
    x2[2, :10] = -float("inf")  # masked entries are fine
    out = run_verify(x2.to(cuda_device), off, bad, V, 0.1, **kernel)
    st = H.status_u32(out["utt_status"])
    assert st[0] == ssd.UTT_NONFINITE and st[1] == ssd.UTT_BAD_DRAFT_ID and st[2] == ssd.UTT_BAD_DRAFT_ID
    assert list(out["accepted_len"].cpu().numpy()) == [0, 1, 1]
    orc = ref.verify(x2.numpy(), V, off.numpy(), bad.numpy(), float(np.float32(0.1)))
    np.testing.assert_array_equal(orc["accepted_len"], [0, 1, 1])
    np.testing.assert_array_equal(st, orc["utt_status"] & 0xff)
    # tau <= 0 rejects nothing, tau >= 1 everything
    out0 = run_verify(x.to(cuda_device), off, ids, V, 0.0, **kernel)
    assert list(out0["accepted_len"].cpu().numpy()) == [3, 3, 4]
    out1 = run_verify(x.to(cuda_device), off, ids, V, 1.0, **kernel)
    assert list(out1["accepted_len"].cpu().numpy()) == [0, 0, 0]
    # a draft token so dominant that fp32 rounds its log-likelihood to 0 or just above: tau = 1
    # still rejects it (p <= 1)
    x40 = x.clone()
    for i in range(10):
        x40[i, ids[i]] += 40.0
    out40 = run_verify(x40.to(cuda_device), off, ids, V, 1.0, **kernel)
    assert list(out40["accepted_len"].cpu().numpy()) == [0, 0, 0]
    assert float(out40["token_logp"].abs().max()) < 1e-6


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
def test_exact_threshold_is_a_reject(cuda_device, kernel):
    """V = 2 with equal logits gives p = 0.5 exactly; with tau = 0.5 the position is rejected
    (p <= tau), with the next float below 0.5 it is accepted."""
    x = torch.zeros((3, 2), dtype=torch.float32)
    ids = torch.tensor([0, 1, 0], dtype=torch.int32)
    off = torch.tensor([0, 3], dtype=torch.int64)
    out = run_verify(x.to(cuda_device), off, ids, 2, 0.5, **kernel)
    assert int(out["accepted_len"].cpu()[0]) == 0 and int(out["all_accepted"].cpu()[0]) == 0
    below = float(np.nextafter(np.float32(0.5), np.float32(0)))
    out = run_verify(x.to(cuda_device), off, ids, 2, below, **kernel)
    assert int(out["accepted_len"].cpu()[0]) == 3 and int(out["all_accepted"].cpu()[0]) == 1


def test_empty_batch_and_malformed_offsets(cuda_device):
    dev = cuda_device
    x = torch.zeros((4, 9), dtype=torch.float32)
    ids = torch.zeros(4, dtype=torch.int32)
    out = run_verify(x[:0].to(dev), torch.zeros(1, dtype=torch.int64), ids[:0], 9, 0.1)
    assert out["accepted_len"].numel() == 0
    off = torch.tensor([0, 3, 2, 4], dtype=torch.int64)
    out = run_verify(x.to(dev), off, ids, 9, 0.05)
    st = H.status_u32(out["utt_status"])
    assert st[1] == ssd.UTT_BAD_OFFSETS and int(out["all_accepted"].cpu()[1]) == 0


@pytest.mark.parametrize("fill", [0x00, 0xff, 0x5a])
def test_workspace_left_dirty_by_anything(cuda_device, fill):
    """The words the streaming kernel keeps per utterance carry a per-call tag: whatever the
    workspace held before, and on a second call that finds the first call's words, the outputs
    are the oracle's."""
    dev = cuda_device
    w = synth.scaled(synth.CONFIGS[1], B=5, variant="literal", seed=71)
    K = [19, 0, 31, 7, 12]
    vb = synth.make_verify_batch(w, K, "cpu")
    x, off, ids = vb.logits.to(dev), vb.tok_off.to(dev), vb.draft_ids.to(dev)
    orc = ref.verify(H.storage_numpy(vb.logits), w.V_llm, vb.tok_off.numpy(), vb.draft_ids.numpy(),
                     float(np.float32(w.tau_slm)))
    out = ssd.alloc_verify_outputs(x.shape[0], 5, dev,
                                   ssd.ssd_verify_workspace_bytes(5, x.shape[0], w.V_llm, ssd.BF16,
                                                                  H.opts(finish=2, split=1)))
    out["workspace"].fill_(fill)
    for _ in range(2):
        ssd.ssd_verify(x, off, ids, w.tau_slm, out=out, opts=H.opts(finish=2, split=1))
        torch.cuda.synchronize()
        H.compare_stage2(out, orc, vb.tok_off.numpy(), w.tau_slm, require_all_margins=False)


def test_runs_are_bit_identical(cuda_device):
    w = synth.scaled(synth.CONFIGS[1], B=4, seed=3)
    vb = synth.make_verify_batch(w, [30, 11, 25, 8], "cpu")
    x = vb.logits.to(cuda_device)
    a = run_verify(x, vb.tok_off, vb.draft_ids, w.V_llm, 0.1, guard=False)
    b = run_verify(x, vb.tok_off, vb.draft_ids, w.V_llm, 0.1, guard=False)
    for k in ("token_logp", "row_lse", "accepted_len", "all_accepted"):
        assert torch.equal(a[k], b[k]), k


# ---- early exit --------------------------------------------------------------------------------

def check_early_exit(w, K, device, skip=None, **okw):
    """ssd_verify_early_exit against the oracle and against ssd_verify: identical decisions,
    log-likelihoods for every position up to the first reject, untouched or correct beyond."""
    vb = synth.make_verify_batch(w, K, "cpu")
    x, off, ids = vb.logits.to(device), vb.tok_off.to(device), vb.draft_ids.to(device)
    o = H.opts(**okw) if okw else None
    code = ssd.BF16 if x.dtype == torch.bfloat16 else ssd.F32
    out = ssd.alloc_early_exit_outputs(x.shape[0], len(K), w.V_llm, code, device, o)
    out["token_logp"].fill_(float("nan"))
    out["row_lse"].fill_(float("nan"))
    skip_dev = None if skip is None else torch.as_tensor(skip, dtype=torch.uint8).to(device)
    ssd.ssd_verify_early_exit(x, off, ids, w.tau_slm, skip=skip_dev, out=out, opts=o)
    torch.cuda.synchronize()
    orc = ref.verify(H.storage_numpy(vb.logits), w.V_llm, vb.tok_off.numpy(), vb.draft_ids.numpy(),
                     float(np.float32(w.tau_slm)), skip=skip)
    np.testing.assert_array_equal(out["accepted_len"].cpu().numpy(), orc["accepted_len"])
    np.testing.assert_array_equal(out["all_accepted"].cpu().numpy(), orc["all_accepted"])
    lp, lse = out["token_logp"].cpu().numpy(), out["row_lse"].cpu().numpy()
    rr = out["rows_read"].cpu().numpy()
    toff = vb.tok_off.numpy()
    for b in range(len(K)):
        if skip is not None and skip[b]:
            assert rr[b] in (0, -1) and np.isnan(lp[toff[b]:toff[b + 1]]).all()
            continue
        need = min(K[b], int(orc["accepted_len"][b]) + 1)
        seg, want = lp[toff[b]:toff[b + 1]].astype(np.float64), orc["token_logp"][toff[b]:toff[b + 1]]
        assert not np.isnan(seg[:need]).any(), "a position up to the first reject was not read"
        read = ~np.isnan(seg)
        assert np.abs(seg[read] - want[read]).max(initial=0.0) <= H.FLOAT_TOL
        ls = lse[toff[b]:toff[b + 1]].astype(np.float64)
        assert np.abs(ls[read] - orc["row_lse"][toff[b]:toff[b + 1]][read]).max(initial=0.0) <= H.FLOAT_TOL
        if rr[b] >= 0:
            assert rr[b] == read.sum() and need <= rr[b] <= K[b]
    return vb, out, orc, rr


def test_early_exit_reads_fewer_rows_and_decides_the_same(cuda_device):
    """Enough rows for the position-major kernel (>= 4 per CTA): planted rejects at all depths."""
    w = synth.scaled(synth.CONFIGS[3], B=24, V_llm=8192, seed=71)          # reject at f*K, f~U(0,1)
    K = [300 + 7 * (i % 11) for i in range(24)]        # ~50 rows per CTA: the lag of a few rows
                                                       # per CTA leaves most of the saving
    vb, out, orc, rr = check_early_exit(w, K, cuda_device)
    assert (rr >= 0).all()
    want = [int(p) if p >= 0 else k for p, k in zip(vb.planted_reject.tolist(), K)]
    assert list(orc["accepted_len"]) == want
    assert rr.sum() < 0.85 * sum(K), "rows after the first reject were not skipped"
    full = ssd.ssd_verify(vb.logits.to(cuda_device), vb.tok_off.to(cuda_device),
                          vb.draft_ids.to(cuda_device), w.tau_slm)
    torch.cuda.synchronize()
    assert torch.equal(full["accepted_len"], out["accepted_len"])
    assert torch.equal(full["utt_status"], out["utt_status"])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [17, 5003, 49152])
def test_early_exit_shapes_skip_and_ragged(cuda_device, dtype, V):
    w = synth.scaled(synth.CONFIGS[1], B=9, V_llm=V, dtype=dtype, seed=300 + V % 89)
    K = [70, 0, 91, 1, 66, 80, 75, 99, 120]
    skip = np.array([0, 0, 1, 0, 0, 0, 1, 0, 0], np.uint8)
    check_early_exit(w, K, cuda_device, skip=skip)
    check_early_exit(w, K, cuda_device, skip=None, warps=4, stages=3, stage_bytes=4096, ctas=7)


def test_early_exit_thousands_of_short_utterances(cuda_device):
    """More utterances than the kernel keeps offsets for in shared memory, rows so short that the
    warp that finishes rows is what limits the rate (its hand-back of row slots holds the
    producer), drafts of 0 to 4 tokens."""
    B = 2500
    w = synth.scaled(synth.CONFIGS[3], B=B, V_llm=96, seed=77)
    K = [(7 * i + i // 5) % 5 for i in range(B)]
    vb, out, orc, rr = check_early_exit(w, K, cuda_device, ctas=24)
    assert (rr >= 0).all()                                   # the position-major kernel ran
    assert int(rr.sum()) <= sum(K)


def test_early_exit_falls_back_on_small_batches(cuda_device):
    w = synth.scaled(synth.CONFIGS[1], B=3, V_llm=32000, seed=9)
    vb, out, orc, rr = check_early_exit(w, [12, 30, 7], cuda_device)
    assert (rr == -1).all()
    assert not np.isnan(out["token_logp"].cpu().numpy()).any()        # the full kernel read everything


def test_early_exit_bad_ids_nonfinite_and_thresholds(cuda_device):
    V, B, Kb = 300, 8, 90
    g = torch.Generator().manual_seed(12)
    x = torch.randn((B * Kb, V), generator=g)
    ids = torch.randint(0, V, (B * Kb,), generator=g, dtype=torch.int32)
    x[torch.arange(B * Kb), ids.long()] += 14.0
    off = torch.arange(0, B * Kb + 1, Kb, dtype=torch.int64)
    bad = ids.clone()
    bad[1 * Kb + 5] = V            # utterance 1: out-of-range id at position 5
    x2 = x.clone()
    x2[2 * Kb + 0, 3] = float("nan")   # utterance 2: NaN in its first row
    dev = cuda_device
    out = ssd.ssd_verify_early_exit(x2.to(dev), off.to(dev), bad.to(dev), 0.1)
    torch.cuda.synchronize()
    st = H.status_u32(out["utt_status"])
    assert st[1] & ssd.UTT_BAD_DRAFT_ID and st[2] & ssd.UTT_NONFINITE
    acc = out["accepted_len"].cpu().tolist()
    assert acc[1] == 5 and acc[2] == 0 and acc[0] == Kb and acc[3:] == [Kb] * 5
    none = ssd.ssd_verify_early_exit(x.to(dev), off.to(dev), ids.to(dev), 0.0)
    every = ssd.ssd_verify_early_exit(x.to(dev), off.to(dev), ids.to(dev), 1.0)
    torch.cuda.synchronize()
    assert none["accepted_len"].cpu().tolist() == [Kb] * B
    assert every["accepted_len"].cpu().tolist() == [0] * B
