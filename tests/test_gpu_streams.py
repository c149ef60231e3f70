"""Two batches decoded on two streams at the same time, each with its own outputs and workspace:
the calls share no state (no globals, no hidden scratch), so every result must be bit-identical
to the one the batch gives when it runs alone."""
import pytest
import torch

from paper_2603_11243_b200 import binding as ssd
from paper_2603_11243_b200 import synth

pytestmark = pytest.mark.gpu


def _make(seed, B, device):
    w = synth.scaled(synth.CONFIGS[1], B=B, seed=seed)
    cb = synth.make_ctc_batch(w, device)
    off = cb.frame_off.to(device)
    s1 = ssd.ssd_ctc_draft(cb.logits, off, w.blank_id, w.max_draft_len)
    torch.cuda.synchronize()
    K = s1["draft_len"].cpu().tolist()
    vb = synth.make_verify_batch(w, K, device)
    return dict(w=w, cb=cb, off=off, vb=vb, tok_off=vb.tok_off.to(device), ids=vb.draft_ids.to(device))


def _run(b, device):
    w = b["w"]
    N, B, M = b["cb"].logits.shape[0], w.B, b["vb"].logits.shape[0]
    s1 = ssd.alloc_ctc_outputs(N, B, device)
    for t in s1.values():
        t.zero_()
    ssd.ssd_ctc_draft(b["cb"].logits, b["off"], w.blank_id, w.max_draft_len, out=s1)
    gate = ssd.ssd_entropy_gate(s1["frame_entropy"], b["off"], w.tau_ctc)
    s2 = ssd.alloc_verify_outputs(M, B, device, ssd.ssd_verify_workspace_bytes(B, M, w.V_llm, ssd.BF16))
    s2["token_logp"].zero_()
    s2["row_lse"].zero_()
    ssd.ssd_verify(b["vb"].logits, b["tok_off"], b["ids"], w.tau_slm, skip=gate["gate_accept"], out=s2)
    return s1, gate, s2


def _same(a, b):
    for x, y in zip(a, b):
        for k in x:
            if k == "workspace":
                continue
            assert torch.equal(x[k].view(torch.uint8), y[k].view(torch.uint8)), k


def test_two_streams_do_not_interfere(cuda_device):
    dev = cuda_device
    a, b = _make(11, 7, dev), _make(12, 9, dev)
    alone_a, alone_b = _run(a, dev), _run(b, dev)
    torch.cuda.synchronize()
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    for _ in range(4):
        with torch.cuda.stream(sa):
            ra = _run(a, dev)
        with torch.cuda.stream(sb):
            rb = _run(b, dev)
        with torch.cuda.stream(sa):
            ra2 = _run(a, dev)
        torch.cuda.synchronize()
        _same(ra, alone_a)
        _same(ra2, alone_a)
        _same(rb, alone_b)
