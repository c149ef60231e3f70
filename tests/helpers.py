"""Shared pieces of the GPU parity tests: storage conversion, oracle calls on the bytes the
GPU saw, and the comparison rules (integers bit-exact, floats within 1e-4 absolute,
threshold decisions compared where the oracle's value is more than 1e-3 from the threshold)."""
import math

import numpy as np
import torch

from oracle import ref
from paper_2603_11243_b200 import binding as ssd

FLOAT_TOL = 1e-4      # absolute, fp32 outputs vs fp64 oracle
MARGIN = 1e-3         # distance from a threshold below which a decision is not compared


def storage_numpy(t: torch.Tensor) -> np.ndarray:
    """Host copy of a logits tensor in the form the oracle takes (float32, or uint16 bits)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def status_u32(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def oracle_stage1(logits_np, V, frame_off, blank_id, cap, tau_ctc, want_logprob=False):
    o = ref.ctc_draft(logits_np, V, frame_off, blank_id, cap, want_logprob=want_logprob)
    g = ref.entropy_gate(o["frame_entropy"], frame_off, float(np.float32(tau_ctc)))
    o.update(g)
    return o


def compare_stage1(gpu, gate, orc, frame_off, tau_ctc, require_all_margins=True):
    """gpu: outputs of ssd_ctc_draft; gate: outputs of ssd_entropy_gate; orc: oracle_stage1."""
    off = np.asarray(frame_off)
    B = len(off) - 1
    np.testing.assert_array_equal(gpu["frame_argmax"].cpu().numpy(), orc["frame_argmax"])
    dH = np.abs(gpu["frame_entropy"].cpu().numpy().astype(np.float64) - orc["frame_entropy"])
    assert dH.size == 0 or dH.max() <= FLOAT_TOL, "entropy off by %g" % dH.max()
    dL = np.abs(gpu["frame_lse"].cpu().numpy().astype(np.float64) - orc["frame_lse"])
    assert dL.size == 0 or dL.max() <= FLOAT_TOL, "lse off by %g" % dL.max()
    np.testing.assert_array_equal(gpu["draft_len"].cpu().numpy(), orc["draft_len"])
    np.testing.assert_array_equal(gpu["draft_full_len"].cpu().numpy(), orc["draft_full_len"])
    tok, frm = gpu["draft_tokens"].cpu().numpy(), gpu["draft_frames"].cpu().numpy()
    for b in range(B):
        n = int(orc["draft_len"][b])
        s = slice(int(off[b]), int(off[b]) + n)
        np.testing.assert_array_equal(tok[s], orc["draft_tokens"][s])
        np.testing.assert_array_equal(frm[s], orc["draft_frames"][s])
    dM = np.abs(gpu["utt_max_entropy"].cpu().numpy().astype(np.float64) - orc["utt_max_entropy"])
    assert dM.size == 0 or dM.max() <= FLOAT_TOL
    np.testing.assert_array_equal(status_u32(gpu["utt_status"]), orc["utt_status"])
    if gate is not None:
        dG = np.abs(gate["max_entropy"].cpu().numpy().astype(np.float64) - orc["max_entropy"])
        assert dG.size == 0 or dG.max() <= FLOAT_TOL
        # the frame of the maximum is unique only up to the float tolerance: the GPU's frame
        # must hold (in the oracle's entropies) a value within tolerance of the maximum, and
        # must be the oracle's frame when the runner-up is clearly lower
        af = gate["argmax_frame"].cpu().numpy()
        for b in range(B):
            T = int(off[b + 1] - off[b])
            if T <= 0 or orc["utt_status"][b] & 4:
                assert af[b] == -1
                continue
            h = orc["frame_entropy"][off[b]:off[b + 1]]
            if np.isnan(h).any():
                continue
            assert 0 <= af[b] < T and h[af[b]] >= h.max() - 2 * FLOAT_TOL
            if T == 1 or np.partition(h, -2)[-2] < h.max() - 2 * FLOAT_TOL:
                assert af[b] == orc["argmax_frame"][b]
        safe = np.abs(orc["max_entropy"] - float(np.float32(tau_ctc))) > MARGIN
        if require_all_margins:
            assert safe.all(), "generator put a max entropy within 1e-3 of tau_ctc"
        np.testing.assert_array_equal(gate["gate_accept"].cpu().numpy()[safe],
                                      orc["gate_accept"][safe])
    return dict(max_dH=float(dH.max()) if dH.size else 0.0,
                max_dlse=float(dL.max()) if dL.size else 0.0)


def check_gate_from_maxima(ctc_out, gate, tau_ctc):
    """ssd_entropy_gate's second form (from ssd_ctc_draft's utterance maxima and status words)
    against its first form (from the frame entropies): the same decisions and maxima, bit for
    bit; the first form is what compare_stage1 holds against the oracle."""
    g2 = ssd.ssd_entropy_gate_from_maxima(ctc_out["utt_max_entropy"], ctc_out["utt_status"], tau_ctc)
    torch.cuda.synchronize()
    assert torch.equal(g2["gate_accept"], gate["gate_accept"])
    assert torch.equal(g2["max_entropy"].view(torch.int32), gate["max_entropy"].view(torch.int32))


def compare_stage2(gpu, orc, tok_off, tau_slm, skip=None, require_all_margins=True):
    off = np.asarray(tok_off)
    B = len(off) - 1
    lp_g = gpu["token_logp"].cpu().numpy().astype(np.float64)
    lse_g = gpu["row_lse"].cpu().numpy().astype(np.float64)
    tau = float(np.float32(tau_slm))
    log_tau = math.log(tau) if tau > 0 else -math.inf
    worst = 0.0
    acc_g, all_g = gpu["accepted_len"].cpu().numpy(), gpu["all_accepted"].cpu().numpy()
    for b in range(B):
        s = slice(int(off[b]), int(off[b + 1]))
        if skip is not None and skip[b]:
            assert acc_g[b] == off[b + 1] - off[b] and all_g[b] == 1
            continue
        lp_o, lse_o = orc["token_logp"][s], orc["row_lse"][s]
        fin = np.isfinite(lp_o)
        d = np.abs(lp_g[s][fin] - lp_o[fin])
        if d.size:
            worst = max(worst, float(d.max()))
        assert d.size == 0 or d.max() <= FLOAT_TOL, "token_logp off by %g (utt %d)" % (d.max(), b)
        np.testing.assert_array_equal(lp_g[s][~fin], lp_o[~fin])     # -inf for bad ids
        dl = np.abs(lse_g[s] - lse_o)
        assert dl.size == 0 or dl.max() <= FLOAT_TOL, "row_lse off by %g" % dl.max()
        safe = (not fin.any()) or tau <= 0 or bool((np.abs(lp_o[fin] - log_tau) > MARGIN).all())
        if require_all_margins:
            assert safe, "generator put a likelihood within 1e-3 of tau_slm (utt %d)" % b
        if safe:
            assert acc_g[b] == orc["accepted_len"][b], (b, acc_g[b], orc["accepted_len"][b])
            assert all_g[b] == orc["all_accepted"][b]
    st = status_u32(gpu["utt_status"])
    np.testing.assert_array_equal(st, orc["utt_status"] & 0xff)
    assert not (orc["utt_status"] & ref.UTT_LOGP_P_DISAGREE).any()
    return dict(max_dlogp=worst)


class Guarded:
    """Output tensors carved out of one buffer with sentinel bands around each, so that a
    kernel writing outside its output is caught without a memory checker."""
    BAND = 64  # elements of 4 bytes

    def __init__(self, device):
        self.device = device
        self.bufs = []

    def alloc(self, n, dtype):
        itemsize = torch.empty((), dtype=dtype).element_size()
        band_b = self.BAND * 4
        raw = torch.full((band_b * 2 + n * itemsize + 16,), 0xA5, dtype=torch.uint8,
                         device=self.device)
        view = raw[band_b:band_b + n * itemsize].view(dtype)
        self.bufs.append((raw, band_b, n * itemsize))
        return view

    def check(self):
        for raw, band_b, nbytes in self.bufs:
            h = raw.cpu().numpy()
            assert (h[:band_b] == 0xA5).all(), "write before an output buffer"
            assert (h[band_b + nbytes:] == 0xA5).all(), "write past an output buffer"


def guarded_ctc_outputs(N, B, device):
    g = Guarded(device)
    out = dict(frame_entropy=g.alloc(N, torch.float32), frame_argmax=g.alloc(N, torch.int32),
               frame_lse=g.alloc(N, torch.float32), draft_tokens=g.alloc(N, torch.int32),
               draft_frames=g.alloc(N, torch.int32), draft_len=g.alloc(B, torch.int32),
               draft_full_len=g.alloc(B, torch.int32), utt_max_entropy=g.alloc(B, torch.float32),
               utt_status=g.alloc(B, torch.int32))
    ws = g.alloc(64 + 512, torch.int32)                      # 256-byte aligned slice of it
    shift = ((-ws.data_ptr()) % 256) // 4
    out["workspace"] = ws[shift:shift + 512].view(torch.uint8)
    return g, out


def guarded_verify_outputs(M, B, device, ws_bytes):
    g = Guarded(device)
    out = dict(token_logp=g.alloc(M, torch.float32), row_lse=g.alloc(M, torch.float32),
               accepted_len=g.alloc(B, torch.int32), all_accepted=g.alloc(B, torch.uint8),
               utt_status=g.alloc(B, torch.int32))
    ws = torch.empty((ws_bytes + 256,), dtype=torch.uint8, device=device)
    shift = (-ws.data_ptr()) % 256
    out["workspace"] = ws[shift:shift + max(ws_bytes, 256)]
    return g, out


def opts(**kw):
    o = ssd.LaunchOpts()
    for k, v in kw.items():
        setattr(o, k, v)
    return o
