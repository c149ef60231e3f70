"""Stage 2 over a vocabulary-parallel LLM head (ssd_verify_shard on every column slice, then
ssd_verify_combine on the stacked statistics), against the fp64 oracle on the whole matrix and
against ssd_verify.  The slices are views of one matrix on one GPU: the exchange between ranks
is a plain all-gather of [M, 3] tensors (tests/test_dist.py covers it with two gloo ranks)."""
import numpy as np
import pytest
import torch

import helpers as H
from oracle import ref
from paper_2603_11243_b200 import binding as ssd
from paper_2603_11243_b200 import synth

pytestmark = pytest.mark.gpu


def sharded_verify(x, cuts, tok_off, ids, tau, skip=None, **okw):
    """x [M, V] on the GPU; cuts = column boundaries (0 = c_0 < ... < c_R = V)."""
    dev = x.device
    M, V = x.shape
    o = H.opts(**okw)
    stats = []
    for c0, c1 in zip(cuts, cuts[1:]):
        st = torch.full((M, 3), float("nan"), dtype=torch.float32, device=dev)
        ssd.ssd_verify_shard(x[:, c0:c1], c0, tok_off, ids, skip=skip, stats=st, opts=o)
        stats.append(st)
    out = ssd.alloc_verify_outputs(M, tok_off.shape[0] - 1, dev, 0)
    out["token_logp"].fill_(float("nan"))
    out["row_lse"].fill_(float("nan"))
    ssd.ssd_verify_combine(torch.stack(stats).contiguous(), V, tok_off, ids, tau, skip=skip, out=out)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("cuts", [(0, 4099), (0, 2048, 4099), (0, 1367, 2733, 4099),
                                  (0, 3, 1000, 1001, 4090, 4099)])
def test_column_slices_against_the_oracle(cuda_device, dtype, cuts):
    """Uneven slices whose first column is not on a 16-byte boundary, down to 1 and 3 columns."""
    w = synth.scaled(synth.CONFIGS[1], B=6, V_llm=4099, dtype=dtype, seed=41)
    K = [37, 0, 120, 1, 64, 9]
    vb = synth.make_verify_batch(w, K, "cpu")
    x = vb.logits.to(cuda_device)
    tok_off, ids = vb.tok_off.to(cuda_device), vb.draft_ids.to(cuda_device)
    out = sharded_verify(x, cuts, tok_off, ids, w.tau_slm)
    orc = ref.verify(H.storage_numpy(vb.logits), w.V_llm, vb.tok_off.numpy(), vb.draft_ids.numpy(),
                     float(np.float32(w.tau_slm)))
    H.compare_stage2(out, orc, vb.tok_off.numpy(), w.tau_slm)
    full = ssd.ssd_verify(x, tok_off, ids, w.tau_slm)
    torch.cuda.synchronize()
    for k in ("accepted_len", "all_accepted", "utt_status"):
        assert torch.equal(out[k], full[k]), k


def test_full_width_rows_split_in_four(cuda_device):
    """Configuration 1's vocabulary (49,152 bf16) over four ranks' worth of columns, with the
    gate's skip mask: skipped utterances are neither read nor combined."""
    w = synth.scaled(synth.CONFIGS[1], B=5, seed=43)
    K = [150, 200, 33, 77, 5]
    vb = synth.make_verify_batch(w, K, "cpu")
    x = vb.logits.to(cuda_device)
    tok_off, ids = vb.tok_off.to(cuda_device), vb.draft_ids.to(cuda_device)
    skip = np.array([0, 1, 0, 0, 1], np.uint8)
    skip_dev = torch.as_tensor(skip).to(cuda_device)
    V = w.V_llm
    out = sharded_verify(x, (0, V // 4, V // 2, 3 * V // 4, V), tok_off, ids, w.tau_slm, skip=skip_dev)
    orc = ref.verify(H.storage_numpy(vb.logits), V, vb.tok_off.numpy(), vb.draft_ids.numpy(),
                     float(np.float32(w.tau_slm)), skip=skip)
    H.compare_stage2(out, orc, vb.tok_off.numpy(), w.tau_slm, skip=skip)
    lp = out["token_logp"].cpu().numpy()
    assert np.isnan(lp[int(vb.tok_off[1]):int(vb.tok_off[2])]).all()      # untouched


def test_bad_ids_masked_shards_and_nonfinite_logits(cuda_device):
    V, cuts = 600, (0, 200, 408, 600)
    g = torch.Generator().manual_seed(5)
    x = torch.randn((12, V), generator=g)
    tok_off = torch.tensor([0, 4, 8, 12], dtype=torch.int64)
    ids = torch.randint(0, V, (12,), generator=g, dtype=torch.int32)
    ids[5], ids[6] = 10, 100
    for i in range(12):
        x[i, ids[i]] += 12.0         # every draft token is accepted unless something below bites
    ids[1] = -1                      # utterance 0, position 1: below the vocabulary
    ids[3] = V                       # ... position 3: one past it
    x[5, 200:408] = float("-inf")    # a whole shard of row 5 masked out, the token lives elsewhere
    x[6, 0:200] = float("-inf")      # row 6: the draft token itself is masked: p = 0, rejected
    x[9, 500] = float("nan")         # utterance 2, position 1 sees a NaN
    out = sharded_verify(x.to(cuda_device), cuts, tok_off.to(cuda_device), ids.to(cuda_device), 0.1)
    orc = ref.verify(x.numpy(), V, tok_off.numpy(), ids.numpy(), float(np.float32(0.1)))
    np.testing.assert_array_equal(orc["accepted_len"], [1, 2, 1])
    np.testing.assert_array_equal(out["accepted_len"].cpu().numpy(), orc["accepted_len"])
    np.testing.assert_array_equal(out["all_accepted"].cpu().numpy(), orc["all_accepted"])
    st = H.status_u32(out["utt_status"])
    np.testing.assert_array_equal(st, orc["utt_status"] & 0xff)
    assert st[0] == ssd.UTT_BAD_DRAFT_ID and st[1] == 0 and st[2] == ssd.UTT_NONFINITE
    lp, lse = out["token_logp"].cpu().numpy(), out["row_lse"].cpu().numpy()
    fin = np.isfinite(orc["token_logp"])
    assert np.abs(lp[fin] - orc["token_logp"][fin]).max() <= H.FLOAT_TOL
    np.testing.assert_array_equal(lp[~fin], orc["token_logp"][~fin])     # -inf and NaN in place
    finl = np.isfinite(orc["row_lse"])
    assert np.abs(lse[finl] - orc["row_lse"][finl]).max() <= H.FLOAT_TOL
    assert np.isnan(lse[9]) and finl.sum() == 11


def test_one_shard_reproduces_ssd_verify_bit_for_bit(cuda_device):
    w = synth.scaled(synth.CONFIGS[1], B=4, V_llm=32000, seed=47)
    vb = synth.make_verify_batch(w, [50, 60, 0, 7], "cpu")
    x = vb.logits.to(cuda_device)
    tok_off, ids = vb.tok_off.to(cuda_device), vb.draft_ids.to(cuda_device)
    out = sharded_verify(x, (0, w.V_llm), tok_off, ids, w.tau_slm)
    full = ssd.ssd_verify(x, tok_off, ids, w.tau_slm)
    torch.cuda.synchronize()
    for k in ("accepted_len", "all_accepted", "utt_status"):
        assert torch.equal(out[k], full[k]), k
    assert torch.allclose(out["token_logp"], full["token_logp"], rtol=0, atol=2e-6)


def test_internal_error_mark_in_a_rank_statistics(cuda_device):
    """The value a rank leaves in place of a row maximum when one of its kernel's bounded waits
    ran out makes the combination report SSD_UTT_INTERNAL for that utterance."""
    dev = cuda_device
    M, R = 6, 2
    st = torch.zeros((R, M, 3), dtype=torch.float32)
    st[:, :, 0] = 1.0
    st[:, :, 1] = 2.0
    st[0, :, 2] = 1.0
    st[1, :, 2] = -float("inf")
    st[1, 4, 0] = torch.tensor([0x7fc0dead], dtype=torch.int32).view(torch.float32)[0]
    off = torch.tensor([0, 3, 6], dtype=torch.int64, device=dev)
    ids = torch.zeros(M, dtype=torch.int32, device=dev)
    out = ssd.ssd_verify_combine(st.to(dev), 100, off, ids, 0.1)
    torch.cuda.synchronize()
    status = out["utt_status"].cpu().numpy().view(np.uint32)
    assert status[0] == 0 and status[1] & ssd.UTT_INTERNAL
    assert int(out["all_accepted"].cpu()[1]) == 0
