"""Parity at the full sizes of the benchmark configurations (and of sampled points of the
throughput sweep), in the launch configuration
bench.py times (default options, inputs generated on the device): every output of
configuration 1 against the oracle; for configurations 2 and 3 (10 and 46 GB of verify logits)
the GPU computes everything and the oracle recomputes a sample of utterances, chosen to include
the longest, the shortest and gate-accepted ones, plus properties that hold for all."""
import numpy as np
import pytest
import torch

import helpers as H
from oracle import ref
from paper_2603_11243_b200 import binding as ssd
from paper_2603_11243_b200 import synth

pytestmark = pytest.mark.gpu


def run_path(w, dev):
    cb = synth.make_ctc_batch(w, dev)
    off = cb.frame_off.to(dev)
    s1 = ssd.ssd_ctc_draft(cb.logits, off, w.blank_id, w.max_draft_len)
    gate = ssd.ssd_entropy_gate(s1["frame_entropy"], off, w.tau_ctc)
    torch.cuda.synchronize()
    K = s1["draft_len"].cpu().tolist()
    vb = synth.make_verify_batch(w, K, dev)
    s2 = ssd.ssd_verify(vb.logits, vb.tok_off.to(dev), vb.draft_ids.to(dev), w.tau_slm,
                        skip=gate["gate_accept"])
    torch.cuda.synchronize()
    return cb, vb, s1, gate, s2, K


def check_sample(w, cb, vb, s1, gate, s2, sample):
    """Oracle on the utterances in `sample`, fed with the bytes the GPU saw."""
    foff, toff = cb.frame_off.numpy(), vb.tok_off.numpy()
    H1 = s1["frame_entropy"].cpu().numpy()
    A1 = s1["frame_argmax"].cpu().numpy()
    L1 = s1["frame_lse"].cpu().numpy()
    tok = s1["draft_tokens"].cpu().numpy()
    dl, dfl = s1["draft_len"].cpu().numpy(), s1["draft_full_len"].cpu().numpy()
    ga = gate["gate_accept"].cpu().numpy()
    lp, al = s2["token_logp"].cpu().numpy(), s2["accepted_len"].cpu().numpy()
    aa = s2["all_accepted"].cpu().numpy()
    tau_c, tau_s = float(np.float32(w.tau_ctc)), float(np.float32(w.tau_slm))
    worst = 0.0
    for b in sample:
        f0, f1, k0, k1 = int(foff[b]), int(foff[b + 1]), int(toff[b]), int(toff[b + 1])
        x = H.storage_numpy(cb.logits[f0:f1])
        o = ref.ctc_draft(x, w.V_ctc, np.array([0, f1 - f0]), w.blank_id, w.max_draft_len)
        np.testing.assert_array_equal(A1[f0:f1], o["frame_argmax"])
        worst = max(worst, np.abs(H1[f0:f1] - o["frame_entropy"]).max(),
                    np.abs(L1[f0:f1] - o["frame_lse"]).max())
        assert dl[b] == o["draft_len"][0] and dfl[b] == o["draft_full_len"][0]
        n = int(dl[b])
        np.testing.assert_array_equal(tok[f0:f0 + n], o["draft_tokens"][:n])
        g = ref.entropy_gate(o["frame_entropy"], np.array([0, f1 - f0]), tau_c)
        assert abs(g["max_entropy"][0] - tau_c) > H.MARGIN
        assert ga[b] == g["gate_accept"][0]
        if ga[b]:
            assert al[b] == k1 - k0 and aa[b] == 1
            continue
        y = H.storage_numpy(vb.logits[k0:k1])
        v = ref.verify(y, w.V_llm, np.array([0, k1 - k0]), vb.draft_ids[k0:k1].numpy(), tau_s)
        if k1 > k0:
            worst = max(worst, np.abs(lp[k0:k1] - v["token_logp"]).max())
            assert (np.abs(v["token_logp"] - np.log(tau_s)) > H.MARGIN).all()
        assert al[b] == v["accepted_len"][0] and aa[b] == v["all_accepted"][0]
        want = int(vb.planted_reject[b]) if vb.planted_reject[b] >= 0 else k1 - k0
        assert al[b] == want                      # generator <-> oracle <-> GPU
    assert worst <= H.FLOAT_TOL, worst
    return worst


def global_properties(w, cb, vb, s1, gate, s2, K):
    B = w.B
    foff = cb.frame_off.numpy()
    T = np.diff(foff)
    dl = s1["draft_len"].cpu().numpy()
    assert (dl <= np.minimum(T, w.max_draft_len)).all() and (dl >= 0).all()
    assert (s1["draft_full_len"].cpu().numpy() >= dl).all()
    Hh = s1["frame_entropy"].cpu().numpy()
    assert np.isfinite(Hh).all() and Hh.min() >= 0 and Hh.max() <= np.log(w.V_ctc) + 1e-4
    np.testing.assert_array_equal(s1["frame_argmax"].cpu().numpy(), cb.winners.numpy())
    assert (H.status_u32(s1["utt_status"]) == 0).all() and (H.status_u32(s2["utt_status"]) == 0).all()
    ga = gate["gate_accept"].cpu().numpy().astype(bool)
    np.testing.assert_array_equal(ga, cb.confident.numpy())
    al = s2["accepted_len"].cpu().numpy()
    want = np.where(vb.planted_reject.numpy() >= 0, vb.planted_reject.numpy(), np.array(K))
    want = np.where(ga, np.array(K), want)
    np.testing.assert_array_equal(al, want)
    lp = s2["token_logp"].cpu().numpy()
    toff = vb.tok_off.numpy()
    rows = np.concatenate([np.arange(toff[b], toff[b + 1]) for b in range(B) if not ga[b]] or
                          [np.array([], np.int64)]).astype(np.int64)
    assert (lp[rows] <= 1e-5).all() and np.isfinite(lp[rows]).all()


def early_exit_agrees(w, vb, gate, s2, dev):
    """ssd_verify_early_exit on the same rows: the same decisions, log-likelihoods up to each
    first reject that agree with ssd_verify's, and no more rows read than there are."""
    off, ids = vb.tok_off.to(dev), vb.draft_ids.to(dev)
    M, B = vb.logits.shape[0], w.B
    code = ssd.BF16 if vb.logits.dtype == torch.bfloat16 else ssd.F32
    out = ssd.alloc_early_exit_outputs(M, B, w.V_llm, code, dev)
    out["token_logp"].fill_(float("nan"))
    ssd.ssd_verify_early_exit(vb.logits, off, ids, w.tau_slm, skip=gate["gate_accept"], out=out)
    torch.cuda.synchronize()
    for k in ("accepted_len", "all_accepted", "utt_status"):
        assert torch.equal(out[k], s2[k]), k
    rr = out["rows_read"].cpu().numpy()
    K = np.diff(vb.tok_off.numpy())
    ga = gate["gate_accept"].cpu().numpy().astype(bool)
    al = s2["accepted_len"].cpu().numpy()
    assert (rr >= 0).all(), "the position-major kernel did not run"
    assert (rr[ga] == 0).all() and (rr <= K).all()
    assert (rr[~ga] >= np.minimum(K, al + 1)[~ga]).all()
    lp_e, lp_f = out["token_logp"].cpu().numpy(), s2["token_logp"].cpu().numpy()
    read = ~np.isnan(lp_e)
    assert read.sum() == rr.sum()
    assert np.abs(lp_e[read] - lp_f[read]).max(initial=0.0) <= 1e-5
    # every position up to the first reject was read
    toff = vb.tok_off.numpy()
    for b in np.flatnonzero(~ga):
        need = min(int(K[b]), int(al[b]) + 1)
        assert read[toff[b]:toff[b] + need].all()
    return float(rr.sum()) / max(1, int(K[~ga].sum()))


def pick(T, ga, n):
    order = np.argsort(T)
    sample = {int(order[0]), int(order[-1]), int(order[len(order) // 2])}
    acc = np.flatnonzero(ga)
    if len(acc):
        sample.add(int(acc[0]))
    rng = np.random.default_rng(11)
    while len(sample) < n:
        sample.add(int(rng.integers(0, len(T))))
    return sorted(sample)


def test_configuration1_every_output(cuda_device):
    w = synth.CONFIGS[1]
    cb, vb, s1, gate, s2, K = run_path(w, cuda_device)
    global_properties(w, cb, vb, s1, gate, s2, K)
    check_sample(w, cb, vb, s1, gate, s2, range(w.B))
    assert early_exit_agrees(w, vb, gate, s2, cuda_device) < 0.9


@pytest.mark.parametrize("cfg,n_sample", [(2, 6), (3, 6)])
def test_configurations_2_and_3_sampled(cuda_device, cfg, n_sample):
    w = synth.CONFIGS[cfg]
    free, _ = torch.cuda.mem_get_info()
    cb, vb, s1, gate, s2, K = run_path(w, cuda_device)
    global_properties(w, cb, vb, s1, gate, s2, K)
    T = np.diff(cb.frame_off.numpy())
    sample = pick(T, gate["gate_accept"].cpu().numpy(), n_sample)
    check_sample(w, cb, vb, s1, gate, s2, sample)
    assert early_exit_agrees(w, vb, gate, s2, cuda_device) < 0.8
    del cb, vb, s1, gate, s2
    torch.cuda.empty_cache()


@pytest.mark.parametrize("cfg", [5, 6])
def test_paper_shape_batches(cuda_device, cfg):
    """The paper's own shape: 348 CTC symbols, length-sorted batches of at most 50,000 frames,
    at the high-accuracy (5) and the high-RTFx (6) operating point.  First and last batch."""
    w = synth.CONFIGS[cfg]
    batches = synth.length_sorted_batches(synth.draw_lengths(w))
    assert all(sum(b) <= synth.MAX_BATCH_TOKENS for b in batches) and sum(len(b) for b in batches) == w.B
    assert all(a >= b for bt in batches for a, b in zip(bt, bt[1:]))
    for lengths in (batches[0], batches[-1]):
        wb = synth.scaled(w, B=len(lengths))
        dev = cuda_device
        cb = synth.make_ctc_batch(wb, dev, lengths)
        off = cb.frame_off.to(dev)
        s1 = ssd.ssd_ctc_draft(cb.logits, off, wb.blank_id, wb.max_draft_len)
        gate = ssd.ssd_entropy_gate(s1["frame_entropy"], off, wb.tau_ctc)
        torch.cuda.synchronize()
        K = s1["draft_len"].cpu().tolist()
        vb = synth.make_verify_batch(wb, K, dev)
        s2 = ssd.ssd_verify(vb.logits, vb.tok_off.to(dev), vb.draft_ids.to(dev), wb.tau_slm,
                            skip=gate["gate_accept"])
        torch.cuda.synchronize()
        ga = gate["gate_accept"].cpu().numpy().astype(bool)
        if cfg == 6:
            assert ga.all()                       # "close to 100 % CTC gating"
        else:
            np.testing.assert_array_equal(ga, cb.confident.numpy())
        sample = pick(np.array(lengths), ga, min(5, len(lengths)))
        check_sample(wb, cb, vb, s1, gate, s2, sample)


@pytest.mark.parametrize("B,V,dtype", [(1, 100352, "bf16"), (8, 152064, "f32"), (64, 32000, "bf16"),
                                       (256, 49152, "f32")])
def test_sweep_points_sampled(cuda_device, B, V, dtype):
    """Points of the throughput sweep (configuration 4) at their full size, spanning its batch
    sizes, vocabularies and both dtypes; few rows (B = 1, 8) take the column-span path of
    ssd_verify.  The GPU computes everything, the oracle recomputes a sample of utterances."""
    w = synth.sweep_point(B, V, dtype)
    cb, vb, s1, gate, s2, K = run_path(w, cuda_device)
    global_properties(w, cb, vb, s1, gate, s2, K)
    sample = sorted({0, B - 1, B // 2})
    check_sample(w, cb, vb, s1, gate, s2, sample)
    del cb, vb, s1, gate, s2
    torch.cuda.empty_cache()
