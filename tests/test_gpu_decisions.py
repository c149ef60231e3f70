"""GPU parity of the calls that sit around the two verification stages: the operating-point
sweep (ssd_threshold_sweep), the final-hypothesis assembly (ssd_assemble, Eq. 7) and the
greedy auto-regressive step head (ssd_greedy_step, Eq. 6), each against the fp64 oracle."""
import math

import numpy as np
import pytest
import torch

import helpers as H
from oracle import ref
from paper_2603_11243_b200 import binding as ssd
from paper_2603_11243_b200 import synth

pytestmark = pytest.mark.gpu


# ---- threshold sweep -------------------------------------------------------------------------

def _sweep_inputs(seed, B, kmax):
    rng = np.random.default_rng(seed)
    K = rng.integers(0, kmax + 1, size=B)
    K[0] = 0
    off = np.concatenate([[0], np.cumsum(K)]).astype(np.int64)
    logp = np.log(rng.uniform(0.01, 0.99, size=int(off[-1]))).astype(np.float32)
    hmax = rng.uniform(0.0, 4.0, size=B).astype(np.float32)
    return hmax, logp, off


@pytest.mark.parametrize("P", [1, 7, 130, 300])
def test_sweep_matches_oracle(cuda_device, P):
    hmax, logp, off = _sweep_inputs(3, 37, 90)
    rng = np.random.default_rng(P)
    tc = rng.uniform(0.3, 3.5, size=P).astype(np.float32)
    ts = rng.uniform(0.0, 0.6, size=P).astype(np.float32)
    ts[0] = 0.0                                   # rejects nothing
    if P > 3:
        ts[3] = 1.5                               # rejects everything
    dev = cuda_device
    out = ssd.ssd_threshold_sweep(torch.from_numpy(hmax).to(dev), torch.from_numpy(logp).to(dev),
                                  torch.from_numpy(off).to(dev), tc.tolist(), ts.tolist())
    torch.cuda.synchronize()
    o = ref.threshold_sweep(hmax, logp, off, tc, ts)
    # decisions are compared where the value is clear of the threshold (fp32 vs fp64 compare)
    gate_safe = np.abs(hmax[None, :].astype(np.float64) - tc[:, None]) > 1e-6
    np.testing.assert_array_equal(out["gate_accept"].cpu().numpy()[gate_safe], o["gate_accept"][gate_safe])
    lt = np.where(ts > 0, np.log(np.maximum(ts.astype(np.float64), 1e-300)), -np.inf)
    al = out["accepted_len"].cpu().numpy()
    aa = out["all_accepted"].cpu().numpy()
    checked = 0
    for p in range(P):
        for b in range(len(off) - 1):
            seg = logp[off[b]:off[b + 1]].astype(np.float64)
            if ts[p] > 0 and (np.abs(seg - lt[p]) < 1e-5).any():
                continue
            assert al[p, b] == o["accepted_len"][p, b] and aa[p, b] == o["all_accepted"][p, b]
            checked += 1
    assert checked > 0.95 * P * (len(off) - 1)
    if gate_safe.all():
        np.testing.assert_array_equal(out["counts"].cpu().numpy().sum(1), np.full(P, len(off) - 1))


def test_sweep_reproduces_verify_and_gate_at_their_thresholds(cuda_device):
    """At the thresholds ssd_entropy_gate / ssd_verify were run with, the sweep returns their
    decisions bit for bit (same fp32 values, same compare)."""
    dev = cuda_device
    w = synth.scaled(synth.CONFIGS[1], B=6)
    cb = synth.make_ctc_batch(w, "cpu")
    off = cb.frame_off.to(dev)
    s1 = ssd.ssd_ctc_draft(cb.logits.to(dev), off, 0, w.max_draft_len)
    K = [9, 0, 31, 14, 22, 5]
    vb = synth.make_verify_batch(w, K, "cpu")
    tok_off = vb.tok_off.to(dev)
    pairs = [(0.7, 0.2), (3.0, 0.1), (5.0, 0.05), (0.1, 0.9)]
    sw = ssd.ssd_threshold_sweep(s1["utt_max_entropy"], torch.zeros(sum(K), device=dev), tok_off,
                                 [p[0] for p in pairs], [p[1] for p in pairs])
    for i, (tc, ts) in enumerate(pairs):
        g = ssd.ssd_entropy_gate(s1["frame_entropy"], off, tc)
        v = ssd.ssd_verify(vb.logits.to(dev), tok_off, vb.draft_ids.to(dev), ts)
        one = ssd.ssd_threshold_sweep(g["max_entropy"], v["token_logp"], tok_off, [tc], [ts])
        torch.cuda.synchronize()
        assert torch.equal(one["gate_accept"][0], g["gate_accept"])
        assert torch.equal(one["accepted_len"][0], v["accepted_len"])
        assert torch.equal(one["all_accepted"][0], v["all_accepted"])
        assert torch.equal(sw["gate_accept"][i], g["gate_accept"])


def test_sweep_edge_cases(cuda_device):
    dev = cuda_device
    off = torch.tensor([0, 2, 1, 3], dtype=torch.int64, device=dev)         # utterance 1 malformed
    logp = torch.tensor([-0.1, float("nan"), -0.2], device=dev)
    hmax = torch.tensor([0.5, float("nan"), 0.5], device=dev)
    out = ssd.ssd_threshold_sweep(hmax, logp, off, [1.0, 1.0], [0.1, 0.0])
    torch.cuda.synchronize()
    assert out["gate_accept"].cpu().tolist() == [[1, 0, 1], [1, 0, 1]]
    # utterance 0 = rows {0, 1}, utterance 2 = rows {1, 2}; row 1 is NaN: a reject unless tau <= 0
    assert out["accepted_len"].cpu().tolist() == [[1, 0, 0], [2, 0, 2]]
    assert out["all_accepted"].cpu().tolist() == [[0, 0, 0], [1, 0, 1]]
    empty = ssd.ssd_threshold_sweep(hmax[:0], logp[:0], off[:1], [0.5], [0.1])
    assert empty["gate_accept"].shape == (1, 0)


# ---- assembly (Eq. 7) ------------------------------------------------------------------------

@pytest.mark.parametrize("B", [1, 5, 300, 1500])
def test_assemble_matches_oracle(cuda_device, B):
    rng = np.random.default_rng(B)
    K = rng.integers(0, 40, size=B)
    off = np.concatenate([[0], np.cumsum(K)]).astype(np.int64)
    M = int(off[-1])
    tokens = rng.integers(0, 50000, size=M).astype(np.int32)
    gate = (rng.uniform(size=B) < 0.2).astype(np.uint8)
    acc = np.array([rng.integers(0, k + 1) for k in K], np.int32)
    alla = (acc == K).astype(np.uint8)
    acc[rng.uniform(size=B) < 0.05] = 1000                    # out-of-range lengths are clamped
    dev = cuda_device
    t = lambda a: torch.from_numpy(a).to(dev)
    out = ssd.ssd_assemble(t(tokens), t(off), t(gate), t(acc), t(alla))
    out["final_tokens"].fill_(-7)
    out = ssd.ssd_assemble(t(tokens), t(off), t(gate), t(acc), t(alla), out=out)
    torch.cuda.synchronize()
    o = ref.assemble(tokens, off, gate, acc, alla)
    np.testing.assert_array_equal(out["final_len"].cpu().numpy(), o["final_len"])
    np.testing.assert_array_equal(out["is_final"].cpu().numpy(), o["is_final"])
    n = int(out["ar_count"].cpu()[0])
    assert n == o["ar_count"]
    np.testing.assert_array_equal(out["ar_utt"].cpu().numpy()[:n], o["ar_utt"][:n])
    np.testing.assert_array_equal(out["ar_resume"].cpu().numpy()[:n], o["ar_resume"][:n])
    ft = out["final_tokens"].cpu().numpy()
    for b in range(B):
        L = int(o["final_len"][b])
        np.testing.assert_array_equal(ft[off[b]:off[b] + L], tokens[off[b]:off[b] + L])
        assert (ft[off[b] + L:off[b + 1]] == -7).all()          # nothing past the prefix is written


def test_assemble_after_the_whole_path(cuda_device):
    """ctc_draft -> gate -> verify -> assemble on configuration 2's value mix: gate-accepted and
    fully verified utterances are final, the others resume at the planted reject."""
    dev = cuda_device
    w = synth.scaled(synth.CONFIGS[2], B=12, t_lo=80, t_hi=160, V_llm=4096)
    cb = synth.make_ctc_batch(w, "cpu")
    off = cb.frame_off.to(dev)
    s1 = ssd.ssd_ctc_draft(cb.logits.to(dev), off, 0, w.max_draft_len)
    g = ssd.ssd_entropy_gate(s1["frame_entropy"], off, w.tau_ctc)
    K = s1["draft_len"].cpu().tolist()
    vb = synth.make_verify_batch(w, K, "cpu")
    tok_off, ids = vb.tok_off.to(dev), vb.draft_ids.to(dev)
    v = ssd.ssd_verify(vb.logits.to(dev), tok_off, ids, w.tau_slm, skip=g["gate_accept"])
    out = ssd.ssd_assemble(ids, tok_off, g["gate_accept"], v["accepted_len"], v["all_accepted"])
    torch.cuda.synchronize()
    conf = cb.confident.numpy()
    planted = vb.planted_reject.numpy()
    want_final = conf | (planted < 0)
    np.testing.assert_array_equal(out["is_final"].cpu().numpy().astype(bool), want_final)
    need = np.flatnonzero(~want_final)
    n = int(out["ar_count"].cpu()[0])
    np.testing.assert_array_equal(out["ar_utt"].cpu().numpy()[:n], need)
    np.testing.assert_array_equal(out["ar_resume"].cpu().numpy()[:n], planted[need])
    assert want_final.any() and (~want_final).any()


# ---- greedy step (Eq. 6) ---------------------------------------------------------------------

def _check_greedy(x_cpu, dev, V=None, **okw):
    V = x_cpu.shape[1] if V is None else V
    o = H.opts(**okw) if okw else None
    out = ssd.ssd_greedy_step(x_cpu.to(dev)[:, :V] if V != x_cpu.shape[1] else x_cpu.to(dev), V=V, opts=o)
    torch.cuda.synchronize()
    orc = ref.greedy_step(H.storage_numpy(x_cpu[:, :V].contiguous()), V)
    np.testing.assert_array_equal(out["next_token"].cpu().numpy(), orc["next_token"])
    d = np.abs(out["next_logp"].cpu().numpy().astype(np.float64) - orc["next_logp"])
    dl = np.abs(out["row_lse"].cpu().numpy().astype(np.float64) - orc["row_lse"])
    assert d.max() <= H.FLOAT_TOL and dl.max() <= H.FLOAT_TOL, (d.max(), dl.max())
    assert (H.status_u32(out["row_status"]) == 0).all()
    return out, orc


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V", [1, 2, 9, 1000, 4099, 32000, 50001, 152064])
def test_greedy_vocabulary_sizes(cuda_device, dtype, V):
    g = torch.Generator().manual_seed(V)
    x = (torch.randn((7, V), generator=g) * 2).to(dtype)
    _check_greedy(x, cuda_device)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("split", [1, 3, 16])
def test_greedy_column_spans_and_ties(cuda_device, dtype, split):
    """Equal maxima in different spans, warps and chunks: the lowest index wins."""
    V, R = 49152 + 24, 9
    g = torch.Generator().manual_seed(1)
    x = (torch.randn((R, V), generator=g) * 0.5).to(dtype)
    first = []
    for r in range(R):
        pos = torch.randint(0, V, (5,), generator=g)
        x[r, pos] = 6.0
        first.append(int(pos.min()))
    out, _ = _check_greedy(x, cuda_device, split=split)
    assert out["next_token"].cpu().tolist() == first


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_greedy_padded_rows_and_misaligned_base(cuda_device, dtype):
    g = torch.Generator().manual_seed(2)
    wide = (torch.randn((11, 5011), generator=g) * 3).to(dtype)
    dev = cuda_device
    V = 5003
    view = wide.to(dev)[:, 5:5 + V]
    out = ssd.ssd_greedy_step(view, V=V)
    torch.cuda.synchronize()
    orc = ref.greedy_step(H.storage_numpy(wide[:, 5:5 + V].contiguous()), V)
    np.testing.assert_array_equal(out["next_token"].cpu().numpy(), orc["next_token"])
    assert np.abs(out["next_logp"].cpu().numpy() - orc["next_logp"]).max() <= H.FLOAT_TOL


def test_greedy_many_rows_peaked(cuda_device):
    """Rows like an LLM's: one token far ahead; 700 rows, more than one per CTA."""
    w = synth.scaled(synth.CONFIGS[1], B=1, V_llm=32000, dtype="bf16", seed=5)
    vb = synth.make_verify_batch(w, [700], "cpu")
    out, orc = _check_greedy(vb.logits, cuda_device)
    # every row but the planted one votes for its boosted token
    agree = (orc["next_token"] == vb.draft_ids.numpy())
    assert agree.sum() == 699


def test_greedy_nonfinite_rows_and_empty(cuda_device):
    dev = cuda_device
    x = torch.zeros((4, 300))
    x[0, 17] = 5.0
    x[1, 3] = float("nan")
    x[2, :] = -float("inf")
    x[3, :100] = -float("inf")
    x[3, 250] = 1.0
    out = ssd.ssd_greedy_step(x.to(dev))
    torch.cuda.synchronize()
    st = H.status_u32(out["row_status"])
    assert list(st) == [0, ssd.UTT_NONFINITE, ssd.UTT_NONFINITE, 0]
    assert out["next_token"].cpu().tolist()[0] == 17 and out["next_token"].cpu().tolist()[3] == 250
    empty = ssd.ssd_greedy_step(x[:0].to(dev), V=300)
    assert empty["next_token"].numel() == 0
