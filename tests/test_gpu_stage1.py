"""GPU parity of stage 1 (ssd_ctc_draft + ssd_entropy_gate) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import helpers as H
from oracle import ref
from paper_2603_11243_b200 import binding as ssd
from paper_2603_11243_b200 import synth

pytestmark = pytest.mark.gpu

KERNELS = {"plain": 1, "tma": 2}


def run_stage1(logits_dev, frame_off, V, blank_id, cap, tau, kernel, guard=True, **okw):
    dev = logits_dev.device
    N = logits_dev.shape[0]
    B = len(frame_off) - 1
    off_dev = frame_off.to(dev)
    if guard:
        g, out = H.guarded_ctc_outputs(N, B, dev)
    else:
        g, out = None, ssd.alloc_ctc_outputs(N, B, dev)
    ssd.ssd_ctc_draft(logits_dev, off_dev, blank_id, cap, V=V, out=out,
                      opts=H.opts(kernel=kernel, **okw))
    gate = ssd.ssd_entropy_gate(out["frame_entropy"], off_dev, tau)
    torch.cuda.synchronize()
    if g:
        g.check()
    H.check_gate_from_maxima(out, gate, tau)
    return out, gate


def check_workload(w, device, kernel, lengths=None, **okw):
    cb = synth.make_ctc_batch(w, "cpu", lengths)
    x = cb.logits.to(device)
    out, gate = run_stage1(x, cb.frame_off, w.V_ctc, w.blank_id, w.max_draft_len, w.tau_ctc,
                           kernel, **okw)
    orc = H.oracle_stage1(H.storage_numpy(cb.logits), w.V_ctc, cb.frame_off.numpy(), w.blank_id,
                          w.max_draft_len, w.tau_ctc)
    stats = H.compare_stage1(out, gate, orc, cb.frame_off.numpy(), w.tau_ctc)
    return cb, out, gate, orc, stats


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
def test_config0_tiny(cuda_device, kernel):
    w = synth.CONFIGS[0]
    cb, out, gate, orc, _ = check_workload(w, cuda_device, kernel)
    # anchored generator: the boosted symbol is the greedy symbol (generator <-> oracle <-> GPU)
    np.testing.assert_array_equal(orc["frame_argmax"], cb.winners.numpy())
    assert 0 < orc["draft_len"][0] <= 50


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
@pytest.mark.parametrize("variant", ["anchored", "literal"])
def test_config1_reduced_batch(cuda_device, kernel, variant):
    """Configuration 1's generator on 6 ragged utterances (T in [250,750], V = 1025 bf16):
    several tiles per warp and a ragged last tile."""
    w = synth.scaled(synth.CONFIGS[1], B=6, variant=variant,
                     tau_ctc=0.7 if variant == "anchored" else 3.0)
    cb, out, gate, orc, _ = check_workload(w, cuda_device, kernel)
    if variant == "anchored":
        np.testing.assert_array_equal(orc["frame_argmax"], cb.winners.numpy())


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
def test_config2_mix_gate_branches(cuda_device, kernel):
    """Configuration 2's value mix on a reduced batch: all-confident utterances pass the gate,
    the others fail it."""
    w = synth.scaled(synth.CONFIGS[2], B=8, t_lo=120, t_hi=300)
    cb, out, gate, orc, _ = check_workload(w, cuda_device, kernel)
    acc = gate["gate_accept"].cpu().numpy().astype(bool)
    np.testing.assert_array_equal(acc, cb.confident.numpy())
    assert acc.any() and (~acc).any()


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
def test_config3_wide_rows_heavy_tail(cuda_device, kernel):
    w = synth.scaled(synth.CONFIGS[3], B=5)
    check_workload(w, cuda_device, kernel, lengths=[100, 333, 1, 0, 257])


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 2, 3, 7, 8, 9, 31, 33, 129, 348, 1000, 1025, 4097])
def test_odd_vocabulary_sizes(cuda_device, kernel, dtype, V):
    """Row lengths that are not multiples of the 16-byte chunk, down to V = 1; lengths 0 and 1."""
    w = synth.scaled(synth.CONFIGS[1], B=5, V_ctc=V, dtype=dtype, variant="literal",
                     tau_ctc=0.31, seed=100 + V, max_draft_len=7)
    cb = synth.make_ctc_batch(w, "cpu", [37, 1, 0, 64, 5])
    x = cb.logits.to(cuda_device)
    out, gate = run_stage1(x, cb.frame_off, V, 0, 7, 0.31, kernel)
    orc = H.oracle_stage1(H.storage_numpy(cb.logits), V, cb.frame_off.numpy(), 0, 7, 0.31)
    H.compare_stage1(out, gate, orc, cb.frame_off.numpy(), 0.31, require_all_margins=False)


@pytest.mark.parametrize("V,T", [(1, [4096, 4096, 1]), (3, [1360, 1360, 1]), (3, [2000, 720, 2]),
                                 (5, [816, 816, 816, 1])])
def test_last_tile_of_a_few_bytes(cuda_device, V, T):
    """Tiny vocabularies make tiles of thousands of rows; a matrix that ends with a tile of one
    or two rows (fewer than 16 bytes) has its second-to-last tile fetched with a shortened bulk
    copy plus plain loads.  (That no read leaves the matrix is checked on the host, in
    test_read_span.py; this checks the values.)"""
    w = synth.scaled(synth.CONFIGS[1], B=len(T), V_ctc=V, dtype="bf16", variant="literal",
                     tau_ctc=0.31, seed=300 + V, max_draft_len=50)
    cb = synth.make_ctc_batch(w, "cpu", T)
    x = cb.logits.to(cuda_device)
    out, gate = run_stage1(x, cb.frame_off, V, 0, 50, 0.31, KERNELS["tma"])
    orc = H.oracle_stage1(H.storage_numpy(cb.logits), V, cb.frame_off.numpy(), 0, 50, 0.31)
    H.compare_stage1(out, gate, orc, cb.frame_off.numpy(), 0.31, require_all_margins=False)


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_padded_rows_and_misaligned_base(cuda_device, kernel, dtype):
    """ld > V, and a base address that is only element-aligned (a column slice of a wider
    matrix starting at column 3)."""
    V, ld, T = 129, 200, [50, 13, 31]
    w = synth.scaled(synth.CONFIGS[0], B=3, V_ctc=ld, dtype=dtype, variant="literal", seed=77)
    cb = synth.make_ctc_batch(w, "cpu", T)
    wide = cb.logits.to(cuda_device)
    view_dev, view_cpu = wide[:, 3:3 + V], cb.logits[:, 3:3 + V]
    out, gate = run_stage1(view_dev, cb.frame_off, V, 0, 50, 2.0, kernel)
    orc = H.oracle_stage1(H.storage_numpy(view_cpu.contiguous()), V, cb.frame_off.numpy(), 0, 50, 2.0)
    H.compare_stage1(out, gate, orc, cb.frame_off.numpy(), 2.0, require_all_margins=False)


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
def test_ties_go_to_the_lowest_index(cuda_device, kernel):
    """bf16 rows with many exactly equal maxima, placed in different 16-byte chunks."""
    V, T = 1025, 64
    x = torch.zeros((T, V), dtype=torch.bfloat16)
    g = torch.Generator().manual_seed(5)
    x += torch.randn((T, V), generator=g).to(torch.bfloat16) * 0.25
    first = []
    for t in range(T):
        pos = torch.randint(0, V, (4,), generator=g)
        x[t, pos] = 7.0
        first.append(int(pos.min()))
    off = torch.tensor([0, T], dtype=torch.int64)
    out, gate = run_stage1(x.to(cuda_device), off, V, 0, T, 1.0, kernel)
    np.testing.assert_array_equal(out["frame_argmax"].cpu().numpy(), np.array(first, np.int32))
    orc = H.oracle_stage1(H.storage_numpy(x), V, off.numpy(), 0, T, 1.0)
    H.compare_stage1(out, gate, orc, off.numpy(), 1.0, require_all_margins=False)


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_masked_and_nonfinite_logits(cuda_device, kernel, dtype):
    """-inf entries are legal and contribute nothing; NaN, +inf or an all -inf row flag the
    utterance and never pass the gate."""
    V = 40
    x = torch.zeros((6, V), dtype=dtype)
    x[0, 5:] = -float("inf")             # uniform over 5 symbols: H = ln 5
    x[1, 7] = float("nan")
    x[2, :] = -float("inf")
    x[3, 2] = float("inf")
    x[4, 1] = 30.0                       # one-hot
    x[5, ::2] = -float("inf")            # uniform over 20
    off = torch.tensor([0, 1, 2, 3, 4, 5, 6], dtype=torch.int64)
    out, gate = run_stage1(x.to(cuda_device), off, V, 0, 4, 5.0, kernel)
    st = H.status_u32(out["utt_status"])
    assert list(st & ssd.UTT_NONFINITE) == [0, 1, 1, 1, 0, 0]
    Hh = out["frame_entropy"].cpu().numpy()
    assert abs(Hh[0] - np.log(5)) < 1e-5 and abs(Hh[5] - np.log(20)) < 1e-5 and Hh[4] < 1e-6
    assert list(gate["gate_accept"].cpu().numpy()) == [1, 0, 0, 0, 1, 1]
    orc = ref.ctc_draft(H.storage_numpy(x), V, off.numpy(), 0, 4)
    np.testing.assert_array_equal(st, orc["utt_status"])


@pytest.mark.parametrize("kernel", KERNELS.values(), ids=KERNELS.keys())
def test_dense_log_softmax_output(cuda_device, kernel):
    w = synth.scaled(synth.CONFIGS[0], B=2, seed=9)
    cb = synth.make_ctc_batch(w, "cpu", [40, 17])
    x = cb.logits.to(cuda_device)
    out = ssd.ssd_ctc_draft(x, cb.frame_off.to(cuda_device), 0, 50, want_logprob=True,
                            opts=H.opts(kernel=kernel))
    torch.cuda.synchronize()
    orc = ref.ctc_draft(H.storage_numpy(cb.logits), w.V_ctc, cb.frame_off.numpy(), 0, 50,
                        want_logprob=True)
    d = np.abs(out["frame_logprob"].cpu().numpy().astype(np.float64) - orc["frame_logprob"])
    assert d.max() <= H.FLOAT_TOL
    assert np.abs(np.exp(out["frame_logprob"].cpu().numpy().astype(np.float64)).sum(1) - 1).max() < 1e-4


def test_empty_batch_and_malformed_offsets(cuda_device):
    dev = cuda_device
    x = torch.zeros((4, 9), dtype=torch.float32, device=dev)
    # B = 0
    out = ssd.ssd_ctc_draft(x[:0], torch.zeros(1, dtype=torch.int64, device=dev), 0, 5, V=9)
    torch.cuda.synchronize()
    assert out["draft_len"].numel() == 0
    # utterance 1 runs backwards: flagged, treated as empty, never accepted, nothing followed
    off = torch.tensor([0, 3, 2, 4], dtype=torch.int64)
    out, gate = run_stage1(x, off, 9, 0, 5, 9.0, 2)
    st = H.status_u32(out["utt_status"])
    assert st[1] == ssd.UTT_BAD_OFFSETS and out["draft_len"].cpu()[1] == 0
    assert gate["gate_accept"].cpu()[1] == 0


def test_runs_are_bit_identical(cuda_device):
    w = synth.scaled(synth.CONFIGS[1], B=4, seed=3)
    cb = synth.make_ctc_batch(w, "cpu")
    x = cb.logits.to(cuda_device)
    a, _ = run_stage1(x, cb.frame_off, w.V_ctc, 0, 200, 0.7, 2, guard=False)
    b, _ = run_stage1(x, cb.frame_off, w.V_ctc, 0, 200, 0.7, 2, guard=False)
    for k in ("frame_entropy", "frame_lse", "frame_argmax", "draft_len", "utt_max_entropy"):
        assert torch.equal(a[k], b[k]), k


@pytest.mark.parametrize("warps,stages,rows", [(16, 2, 1), (8, 4, 3), (4, 3, 0), (1, 8, 5)])
def test_pipeline_shapes(cuda_device, warps, stages, rows):
    """Other ring shapes of the bulk-copy kernel give the same answers."""
    w = synth.scaled(synth.CONFIGS[1], B=3, seed=21)
    check_workload(w, cuda_device, 2, warps=warps, stages=stages, stage_bytes=rows, ctas=5)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 5, 17, 24, 129])
@pytest.mark.parametrize("shift", [-100.0, -200.0, 90.0])
def test_short_rows_far_from_zero(cuda_device, dtype, V, shift):
    """Rows with fewer 16-byte chunks than lanes share them, all logits moved by a constant
    (Eq. 2 / Eq. 3 do not change under it): lanes that hold no chunk of a row must add nothing,
    whatever the row maximum is."""
    w = synth.scaled(synth.CONFIGS[1], B=4, V_ctc=V, dtype=dtype, variant="literal",
                     tau_ctc=0.9, seed=500 + V, max_draft_len=30)
    cb = synth.make_ctc_batch(w, "cpu", [33, 2, 0, 50])
    x = (cb.logits.float() + shift).to(cb.logits.dtype)
    for G in (0, 2, 4, 8, 32):
        out, gate = run_stage1(x.to(cuda_device), cb.frame_off, V, 0, 30, 0.9, 2, split=G)
        st = H.status_u32(out["utt_status"])
        assert not (st & ssd.UTT_NONFINITE).any()
        orc = H.oracle_stage1(H.storage_numpy(x), V, cb.frame_off.numpy(), 0, 30, 0.9)
        H.compare_stage1(out, gate, orc, cb.frame_off.numpy(), 0.9, require_all_margins=False)


@pytest.mark.parametrize("V,shift", [(5000, -150.0), (4097, 90.0), (20000, -150.0)])
def test_one_logit_far_above_many_equal_ones(cuda_device, V, shift):
    """bf16 rows far from zero, where a step of the format is 1: the many small logits take three
    or four values, one logit stands 12 above them.  A lane's running sums then hold one term of
    2^17 and get thousands of equal small ones added, whose rounding errors all point the same
    way unless they are summed apart first.  With few lanes per row (long lanes) this was off
    by 1.4e-4; half the tolerance is asked for here."""
    g = torch.Generator().manual_seed(V)
    T = [130, 0, 75, 1]
    N = sum(T)
    x = torch.randn((N, V), generator=g) * 0.3 + shift
    win = torch.randint(0, V, (N,), generator=g)
    x[torch.arange(N), win] += 12.0
    x = x.to(torch.bfloat16)
    off = torch.tensor([0] + list(np.cumsum(T)), dtype=torch.int64)
    orc = H.oracle_stage1(H.storage_numpy(x), V, off.numpy(), 0, 50, 0.9)
    ran = 0
    for G in (0, 4, 8, 16, 32):
        try:
            out, gate = run_stage1(x.to(cuda_device), off, V, 0, 50, 0.9, 2, split=G)
        except ssd.SsdError as e:
            assert e.code == ssd.ERR_ARG and G != 0      # too many chunks per lane: refused
            continue
        ran += 1
        H.compare_stage1(out, gate, orc, off.numpy(), 0.9, require_all_margins=False)
        dH = np.abs(out["frame_entropy"].cpu().numpy().astype(np.float64) - orc["frame_entropy"])
        assert dH.max() <= 0.5 * H.FLOAT_TOL, (G, dH.max())
    assert ran >= 2


@pytest.mark.parametrize("V,dtype", [(1025, "bf16"), (348, "bf16"), (4097, "bf16"), (129, "f32"),
                                     (1025, "f32"), (2049, "bf16"), (64, "bf16"), (7, "bf16")])
def test_lanes_per_row_and_exponential_split(cuda_device, V, dtype):
    """Every number of lanes per row the kernel is built for, and the FMA-pipe exponential on
    one or two of a bf16 chunk's four pairs, give the oracle's answers."""
    w = synth.scaled(synth.CONFIGS[1], B=5, V_ctc=V, dtype=dtype, t_lo=37, t_hi=211, seed=40 + V)
    cb = synth.make_ctc_batch(w, "cpu")
    x = cb.logits.to(cuda_device)
    orc = H.oracle_stage1(H.storage_numpy(cb.logits), V, cb.frame_off.numpy(), w.blank_id,
                          w.max_draft_len, w.tau_ctc)
    variants = [dict(split=G) for G in (2, 4, 8, 16, 32)]
    if dtype == "bf16":
        variants += [dict(fma_exp=1), dict(fma_exp=2), dict(split=8, fma_exp=1)]
    ran = 0
    for kw in variants:
        try:
            out, gate = run_stage1(x, cb.frame_off, V, w.blank_id, w.max_draft_len, w.tau_ctc, 0, **kw)
        except ssd.SsdError as e:        # few lanes on a long row: refused for accuracy
            assert e.code == ssd.ERR_ARG and kw.get("split", 32) < 32
            continue
        ran += 1
        H.compare_stage1(out, gate, orc, cb.frame_off.numpy(), w.tau_ctc, require_all_margins=False)
    assert ran >= 3


def test_fma_exponential_range_guards(cuda_device):
    """The FMA-pipe exponential represents neither 2^t for t above 120 nor references beyond
    +-4096 (its lower clamp is a bf16 value): such rows must take the exact routine."""
    V, T = 1025, 24
    g = torch.Generator().manual_seed(8)
    x = torch.randn((T, V), generator=g)
    x[0:8, 700] += 200.0                 # far above the first chunk's reference
    x[8:16] += 6000.0                    # large reference
    x[16:24] -= 9000.0
    x[16:24, 3] += 150.0
    x = x.to(torch.bfloat16)
    off = torch.tensor([0, 8, 16, 24], dtype=torch.int64)
    orc = H.oracle_stage1(H.storage_numpy(x), V, off.numpy(), 0, T, 1.0)
    for f in (1, 2):
        out, gate = run_stage1(x.to(cuda_device), off, V, 0, T, 1.0, 2, fma_exp=f)
        np.testing.assert_array_equal(out["frame_argmax"].cpu().numpy(), orc["frame_argmax"])
        d = np.abs(out["frame_entropy"].cpu().numpy().astype(np.float64) - orc["frame_entropy"])
        assert d.max() <= H.FLOAT_TOL
        # lse is thousands here: one fp32 ulp at that size is beyond 1e-4 absolute
        lse, want = out["frame_lse"].cpu().numpy().astype(np.float64), orc["frame_lse"]
        assert (np.abs(lse - want) <= 1e-4 + 2 * np.spacing(np.abs(want).astype(np.float32))).all()


def test_many_short_utterances_per_tile(cuda_device):
    """Utterances of 0 to 3 frames, empty ones between them: a tile of frames spans dozens."""
    rng = np.random.default_rng(77)
    lens = rng.integers(0, 4, size=700).tolist()
    w = synth.scaled(synth.CONFIGS[1], B=len(lens), V_ctc=33, dtype="bf16", seed=9, tau_ctc=1.5)
    cb = synth.make_ctc_batch(w, "cpu", lens)
    x = cb.logits.to(cuda_device)
    out, gate = run_stage1(x, cb.frame_off, 33, 0, 2, 1.5, 2)
    orc = H.oracle_stage1(H.storage_numpy(cb.logits), 33, cb.frame_off.numpy(), 0, 2, 1.5)
    H.compare_stage1(out, gate, orc, cb.frame_off.numpy(), 1.5, require_all_margins=False)


def test_thousands_of_utterances(cuda_device):
    """A batch of 2,300 utterances of 0 to 8 frames."""
    rng = np.random.default_rng(78)
    lens = rng.integers(0, 9, size=2300).tolist()
    w = synth.scaled(synth.CONFIGS[1], B=len(lens), V_ctc=129, dtype="f32", seed=10, tau_ctc=1.5)
    cb = synth.make_ctc_batch(w, "cpu", lens)
    x = cb.logits.to(cuda_device)
    out, gate = run_stage1(x, cb.frame_off, 129, 0, 5, 1.5, 2)
    orc = H.oracle_stage1(H.storage_numpy(cb.logits), 129, cb.frame_off.numpy(), 0, 5, 1.5)
    H.compare_stage1(out, gate, orc, cb.frame_off.numpy(), 1.5, require_all_margins=False)


def test_workspace_left_dirty_by_anything(cuda_device):
    """The tile counter carries a per-call tag: whatever the workspace held before -- zeros, all
    ones, the word of an earlier call -- and with no workspace at all (tiles dealt out in a
    fixed order), the call gives the same outputs.  Few warps, so that most tiles are claimed
    from the counter."""
    dev = cuda_device
    w = synth.scaled(synth.CONFIGS[1], B=6, seed=31)
    cb = synth.make_ctc_batch(w, "cpu")
    x, off = cb.logits.to(dev), cb.frame_off.to(dev)
    ref_out = ssd.ssd_ctc_draft(x, off, 0, 200)
    torch.cuda.synchronize()
    few = H.opts(ctas=3, warps=2)
    for fill in (0x00, 0xff, 0x5a, None):
        out = ssd.alloc_ctc_outputs(x.shape[0], w.B, dev)
        if fill is None:
            del out["workspace"]
        else:
            out["workspace"].fill_(fill)
        for _ in range(2):               # the second call finds the first call's word
            ssd.ssd_ctc_draft(x, off, 0, 200, out=out, opts=few)
            torch.cuda.synchronize()
            for k in ("frame_entropy", "frame_argmax", "draft_len", "draft_full_len",
                      "utt_max_entropy", "utt_status"):
                assert torch.equal(out[k], ref_out[k]), (fill, k)
            n = int(out["draft_len"].sum())
            assert n > 0


def test_internal_error_marks_never_pass_the_gate(cuda_device):
    """The value a kernel leaves in a frame's entropy when one of its bounded waits ran out
    (a NaN with a fixed payload) makes the gate refuse the utterance and report
    SSD_UTT_INTERNAL; so does that status bit in the form that reads utterance maxima."""
    dev = cuda_device
    h = torch.full((10,), 0.01, dtype=torch.float32)
    h[7] = torch.tensor([0x7fc0dead], dtype=torch.int32).view(torch.float32)[0]
    off = torch.tensor([0, 5, 10], dtype=torch.int64)
    gate = ssd.ssd_entropy_gate(h.to(dev), off.to(dev), 5.0)
    assert gate["gate_accept"].cpu().tolist() == [1, 0]
    mx = torch.tensor([0.01, 0.01, 0.01], dtype=torch.float32, device=dev)
    st = torch.tensor([0, ssd.UTT_INTERNAL - (1 << 32), ssd.UTT_BAD_OFFSETS], dtype=torch.int32, device=dev)
    g2 = ssd.ssd_entropy_gate_from_maxima(mx, st, 5.0)
    assert g2["gate_accept"].cpu().tolist() == [1, 0, 0]
