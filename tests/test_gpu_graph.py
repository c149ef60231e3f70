"""The calls of a step captured into a CUDA graph and replayed with new contents in the same
buffers give what the same calls give when made one by one.  (The frame statistics kernel hands
out tiles from counter words that are told apart from leftovers by a per-launch tag; a replay
repeats the launch's parameters, so the tag must not come from them alone.)"""
import numpy as np
import pytest
import torch

from paper_2603_11243_b200 import binding as ssd
from paper_2603_11243_b200 import synth

pytestmark = pytest.mark.gpu


def _eager(cb, off, w, vb, tok_off, ids, dev, early_exit):
    s1 = ssd.ssd_ctc_draft(cb, off, w.blank_id, w.max_draft_len)
    gate = ssd.ssd_entropy_gate_from_maxima(s1["utt_max_entropy"], s1["utt_status"], w.tau_ctc)
    if early_exit:
        s2 = ssd.ssd_verify_early_exit(vb, tok_off, ids, w.tau_slm, skip=gate["gate_accept"])
    else:
        s2 = ssd.ssd_verify(vb, tok_off, ids, w.tau_slm, skip=gate["gate_accept"])
    torch.cuda.synchronize()
    return s1, gate, s2


@pytest.mark.parametrize("early_exit", [False, True])
def test_captured_step_replays_with_new_inputs(cuda_device, early_exit):
    dev = cuda_device
    # more tiles than warps in the grid, so that tiles are claimed from the counters
    B = 40
    lengths = [560 + 13 * (i % 9) for i in range(B)]
    K = [30 + (5 * i) % 23 for i in range(B)]
    base = synth.scaled(synth.CONFIGS[1], B=B, V_llm=8192)
    sets = []
    for seed in (11, 12, 13, 14):
        w = synth.scaled(base, seed=seed)
        cb = synth.make_ctc_batch(w, dev, lengths)
        vb = synth.make_verify_batch(w, K, dev)
        sets.append((w, cb, vb))
    w0, cb0, vb0 = sets[0]
    N, M = cb0.logits.shape[0], vb0.logits.shape[0]
    assert N > 8 * 148 * 16, "not enough frames for the tile counters to be used"
    # static buffers of the graph
    x_c, off_c = torch.empty_like(cb0.logits), cb0.frame_off.to(dev).clone()
    x_v, off_v, ids_v = torch.empty_like(vb0.logits), vb0.tok_off.to(dev).clone(), vb0.draft_ids.to(dev).clone()
    code = ssd.BF16 if x_v.dtype == torch.bfloat16 else ssd.F32
    s1 = ssd.alloc_ctc_outputs(N, B, dev)
    gate = ssd.alloc_gate_outputs(B, dev)
    if early_exit:
        s2 = ssd.alloc_early_exit_outputs(M, B, w0.V_llm, code, dev)
    else:
        s2 = ssd.alloc_verify_outputs(M, B, dev, ssd.ssd_verify_workspace_bytes(B, M, w0.V_llm, code))

    def step():
        ssd.ssd_ctc_draft(x_c, off_c, w0.blank_id, w0.max_draft_len, out=s1)
        ssd.ssd_entropy_gate_from_maxima(s1["utt_max_entropy"], s1["utt_status"], w0.tau_ctc, out=gate)
        if early_exit:
            ssd.ssd_verify_early_exit(x_v, off_v, ids_v, w0.tau_slm, skip=gate["gate_accept"], out=s2)
        else:
            ssd.ssd_verify(x_v, off_v, ids_v, w0.tau_slm, skip=gate["gate_accept"], out=s2)

    x_c.copy_(cb0.logits); x_v.copy_(vb0.logits)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                       # one call of each kind before capturing
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for w, cb, vb in sets[1:] + sets[:1] + sets[1:2]:       # five replays
        x_c.copy_(cb.logits); x_v.copy_(vb.logits)
        off_v.copy_(vb.tok_off.to(dev)); ids_v.copy_(vb.draft_ids.to(dev))
        graph.replay()
        torch.cuda.synchronize()
        e1, eg, e2 = _eager(cb.logits, cb.frame_off.to(dev), w, vb.logits, vb.tok_off.to(dev),
                            vb.draft_ids.to(dev), dev, early_exit)
        assert int(s1["utt_status"].max().item()) == 0 and int(s2["utt_status"].max().item()) == 0
        for k in ("frame_argmax", "draft_len", "draft_full_len", "utt_status"):
            assert torch.equal(s1[k], e1[k]), k
        # utterance b's draft sits at its first frame's index; what follows it is not written
        start = cb.frame_off.to(dev)[:-1]
        frame = torch.arange(N, device=dev)
        utt = torch.searchsorted(cb.frame_off.to(dev)[1:].contiguous(), frame, right=True)
        used = frame - start[utt] < s1["draft_len"].to(torch.int64)[utt]
        assert torch.equal(s1["draft_tokens"][used], e1["draft_tokens"][used])
        np.testing.assert_array_equal(s1["frame_entropy"].cpu().numpy(), e1["frame_entropy"].cpu().numpy())
        np.testing.assert_array_equal(s1["utt_max_entropy"].cpu().numpy(), e1["utt_max_entropy"].cpu().numpy())
        assert torch.equal(gate["gate_accept"], eg["gate_accept"])
        for k in ("accepted_len", "all_accepted", "utt_status"):
            assert torch.equal(s2[k], e2[k]), k
        if not early_exit:
            np.testing.assert_array_equal(s2["token_logp"].cpu().numpy(), e2["token_logp"].cpu().numpy())


@pytest.mark.filterwarnings("ignore:The CUDA Graph is empty")
def test_finish_inside_is_refused_while_capturing(cuda_device):
    dev = cuda_device
    w = synth.scaled(synth.CONFIGS[1], B=6, V_llm=4096, seed=5)
    vb = synth.make_verify_batch(w, [40, 50, 60, 70, 80, 90], dev)
    off, ids = vb.tok_off.to(dev), vb.draft_ids.to(dev)
    o = ssd.LaunchOpts()
    o.finish, o.split = 2, 1
    code = ssd.BF16 if vb.logits.dtype == torch.bfloat16 else ssd.F32
    M = vb.logits.shape[0]
    out = ssd.alloc_verify_outputs(M, 6, dev, ssd.ssd_verify_workspace_bytes(6, M, w.V_llm, code, o))
    ssd.ssd_verify(vb.logits, off, ids, w.tau_slm, out=out, opts=o)       # fine outside a capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with pytest.raises(ssd.SsdError) as err:
        with torch.cuda.graph(graph):
            ssd.ssd_verify(vb.logits, off, ids, w.tau_slm, out=out, opts=o)
    assert err.value.code == ssd.ERR_ARG
