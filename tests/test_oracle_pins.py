"""The oracle against what the paper and the mathematics fix (CPU only)."""
import numpy as np
import pytest

import oracle_pins
from oracle import ref
from oracle_impls import MUTANTS, ORACLES


@pytest.mark.parametrize("impl", ORACLES, ids=lambda i: i.name)
@pytest.mark.parametrize("pin", oracle_pins.ALL_PINS, ids=lambda p: p.__name__)
def test_pin_holds(impl, pin):
    pin(impl)


@pytest.mark.parametrize("mutant", MUTANTS, ids=lambda i: i.name)
def test_planted_mistake_is_caught(mutant):
    """A pin-suite that a plausible mistake slips through pins nothing: each broken
    variant must fail at least one pin."""
    failed = []
    for pin in oracle_pins.ALL_PINS:
        try:
            pin(mutant)
        except AssertionError:
            failed.append(pin.__name__)
        except Exception:  # a mistake may also crash a pin; that counts as caught
            failed.append(pin.__name__)
    assert failed, "no pin noticed: " + mutant.name


# ---- batch-level behaviour of the C oracle (ragged layout, caps, flags) --------------------

def _batch():
    rng = np.random.default_rng(0)
    T = [5, 0, 9, 1]
    off = np.concatenate([[0], np.cumsum(T)]).astype(np.int64)
    V = 6
    x = rng.normal(size=(int(off[-1]), V)).astype(np.float32) * 3
    return x, off, V, T


def test_batch_matches_per_row_calls():
    x, off, V, T = _batch()
    o = ref.ctc_draft(x, V, off, blank_id=0, max_draft_len=3, want_logprob=True)
    for r in range(x.shape[0]):
        lse, H, arg, _ = ref.row_stats(x[r])
        assert o["frame_lse"][r] == lse and o["frame_entropy"][r] == H
        assert o["frame_argmax"][r] == arg
        np.testing.assert_allclose(o["frame_logprob"][r], x[r].astype(np.float64) - lse,
                                   rtol=0, atol=1e-15)
    for b in range(len(T)):
        a = o["frame_argmax"][off[b]:off[b + 1]]
        toks, frames, U = ref.collapse(a, 0) if T[b] else (np.array([], np.int32),) * 2 + (0,)
        assert o["draft_full_len"][b] == U
        assert o["draft_len"][b] == min(U, 3)
        n = min(U, 3)
        np.testing.assert_array_equal(o["draft_tokens"][off[b]:off[b] + n], toks[:n])
        np.testing.assert_array_equal(o["draft_frames"][off[b]:off[b] + n], frames[:n])
        hm = o["frame_entropy"][off[b]:off[b + 1]].max() if T[b] else 0.0
        assert o["utt_max_entropy"][b] == hm
        # collapse never carries state across the ragged boundary
        for k in range(n):
            assert a[frames[k]] == toks[k]
    assert o["draft_len"][1] == 0 and o["utt_max_entropy"][1] == 0.0  # empty utterance


def test_gate_on_batch_and_empty_utterance():
    x, off, V, T = _batch()
    o = ref.ctc_draft(x, V, off, 0, 100)
    g = ref.entropy_gate(o["frame_entropy"], off, 0.7)
    for b in range(len(T)):
        h = o["frame_entropy"][off[b]:off[b + 1]]
        assert bool(g["gate_accept"][b]) == all(v < 0.7 for v in h)
        if T[b]:
            assert g["argmax_frame"][b] == int(np.argmax(h)) and g["max_entropy"][b] == h.max()
    assert g["gate_accept"][1] == 1 and g["argmax_frame"][1] == -1
    assert ref.entropy_gate(o["frame_entropy"], off, 0.0)["gate_accept"][1] == 0


def test_verify_skip_bad_id_and_flags():
    rng = np.random.default_rng(1)
    V, K = 11, [3, 2, 4]
    off = np.concatenate([[0], np.cumsum(K)]).astype(np.int64)
    x = rng.normal(size=(9, V)).astype(np.float32)
    ids = rng.integers(0, V, size=9).astype(np.int32)
    for i in range(9):
        x[i, ids[i]] += 9.0
    ids_bad = ids.copy()
    ids_bad[4] = V  # utterance 1, position 1
    o = ref.verify(x, V, off, ids_bad, 0.1, skip=np.array([0, 0, 1], np.uint8))
    assert list(o["accepted_len"]) == [3, 1, 4] and list(o["all_accepted"]) == [1, 0, 1]
    assert o["utt_status"][1] & ref.UTT_BAD_DRAFT_ID and o["utt_status"][0] == 0
    assert np.isnan(o["token_logp"][5:]).all()  # skipped rows untouched
    assert o["token_logp"][4] == -np.inf
    assert not (o["utt_status"] & ref.UTT_LOGP_P_DISAGREE).any()
    # tau <= 0 rejects nothing, tau >= 1 rejects everything
    assert list(ref.verify(x, V, off, ids, 0.0)["accepted_len"]) == K
    assert list(ref.verify(x, V, off, ids, 1.0)["accepted_len"]) == [0, 0, 0]


def test_nonfinite_rows_are_flagged_and_minus_inf_is_legal():
    x = np.zeros((4, 5), np.float32)
    x[1, 2] = np.nan
    x[2, :] = -np.inf
    x[3, 1] = -np.inf
    off = np.array([0, 1, 2, 3, 4], np.int64)
    o = ref.ctc_draft(x, 5, off, 0, 10)
    assert list(o["utt_status"] & ref.UTT_NONFINITE) == [0, 1, 1, 0]
    assert abs(o["frame_entropy"][3] - np.log(4)) < 1e-12


def test_padded_leading_dimension():
    rng = np.random.default_rng(4)
    x = rng.normal(size=(7, 10)).astype(np.float32)
    off = np.array([0, 7], np.int64)
    a = ref.ctc_draft(np.ascontiguousarray(x[:, :6]), 6, off, 0, 10)
    b = ref.ctc_draft(x, 6, off, 0, 10)  # ld = 10, V = 6
    np.testing.assert_array_equal(a["frame_entropy"], b["frame_entropy"])
    np.testing.assert_array_equal(a["draft_tokens"], b["draft_tokens"])


def test_malformed_offsets_are_flagged_not_followed():
    x = np.zeros((4, 3), np.float32)
    off = np.array([0, 3, 2, 4], np.int64)  # utterance 1 runs backwards
    o = ref.ctc_draft(x, 3, off, 0, 10)
    assert o["utt_status"][1] == ref.UTT_BAD_OFFSETS and o["draft_len"][1] == 0


# ---- the two writings of the definitions against each other, on random inputs ----------------

@pytest.mark.parametrize("seed", range(8))
def test_c_oracle_and_numpy_oracle_agree_on_random_batches(seed):
    """Two independently written statements of the same mathematics (sequential C with a
    two-pass softmax; NumPy through normalised probabilities and run-length groups) must agree
    on the whole path, bf16 and fp32, ragged batches, every threshold outcome."""
    from oracle import mini
    from oracle_impls import to_storage
    rng = np.random.default_rng(700 + seed)
    dtype = "bf16" if seed % 2 else "f32"
    V, B = int(rng.integers(2, 40)), int(rng.integers(1, 6))
    T = rng.integers(0, 25, size=B)
    off = np.concatenate([[0], np.cumsum(T)]).astype(np.int64)
    x = to_storage(rng.normal(size=(int(off[-1]), V)) * rng.choice([0.5, 3.0, 9.0]), dtype)
    blank, cap, tau_c = int(rng.integers(0, V)), int(rng.integers(1, 12)), float(rng.uniform(0.2, 3.0))
    o = ref.ctc_draft(x, V, off, blank, cap)
    g = ref.entropy_gate(o["frame_entropy"], off, tau_c)
    xw = mini.widen(x).reshape(-1, V)
    for b in range(B):
        rows = xw[off[b]:off[b + 1]]
        a = mini.greedy_alignment(rows) if len(rows) else np.zeros(0, np.int32)
        np.testing.assert_array_equal(o["frame_argmax"][off[b]:off[b + 1]], a)
        H = [mini.frame_entropy(r) for r in rows]
        np.testing.assert_allclose(o["frame_entropy"][off[b]:off[b + 1]], H, rtol=0, atol=1e-12)
        y = mini.collapse(a, blank)
        assert o["draft_full_len"][b] == len(y) and o["draft_len"][b] == min(len(y), cap)
        n = int(o["draft_len"][b])
        assert list(o["draft_tokens"][off[b]:off[b] + n]) == y[:n]
        if len(H) and abs(max(H) - tau_c) > 1e-9:
            assert bool(g["gate_accept"][b]) == mini.gate(H, tau_c)
    # stage 2 on its own ragged batch
    Vl = int(rng.integers(2, 60))
    K = rng.integers(0, 15, size=B)
    toff = np.concatenate([[0], np.cumsum(K)]).astype(np.int64)
    xl = to_storage(rng.normal(size=(int(toff[-1]), Vl)) * 4.0, dtype)
    ids = rng.integers(0, Vl, size=int(toff[-1])).astype(np.int32)
    tau_s = float(rng.choice([0.02, 0.1, 0.2, 0.5]))
    v = ref.verify(xl, Vl, toff, ids, tau_s)
    gr = ref.greedy_step(xl, Vl) if len(ids) else None
    xlw = mini.widen(xl).reshape(-1, Vl)
    for b in range(B):
        rows, d = xlw[toff[b]:toff[b + 1]], ids[toff[b]:toff[b + 1]]
        p = mini.token_likelihoods(rows, d)
        np.testing.assert_allclose(np.exp(v["token_logp"][toff[b]:toff[b + 1]]), p, rtol=1e-12, atol=0)
        if len(p) == 0 or np.abs(p - tau_s).min() > 1e-9:
            assert v["accepted_len"][b] == mini.accepted_prefix(p, tau_s)
        for i, r in enumerate(rows):
            tok, lp = mini.greedy_token(r)
            assert gr["next_token"][toff[b] + i] == tok
            assert abs(gr["next_logp"][toff[b] + i] - lp) < 1e-12
