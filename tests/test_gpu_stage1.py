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
