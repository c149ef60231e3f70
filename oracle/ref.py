"""ctypes wrapper of the C fp64 oracle (oracle/ssd_oracle.c).  Test infrastructure only.

Arrays are NumPy and live on the host.  A bf16 matrix is passed as a uint16 array holding
the raw bit patterns; an fp32 matrix as float32.  Outputs are float64 / int32 / uint8.
"""
import ctypes as C

import numpy as np

from . import build as _build

F32, BF16 = 0, 1
UTT_NONFINITE, UTT_BAD_DRAFT_ID, UTT_BAD_OFFSETS, UTT_LOGP_P_DISAGREE = 1, 2, 4, 0x100

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.ssd_ref_row_stats.restype = C.c_int
        _lib.ssd_ref_collapse.restype = C.c_int32
        for name in ("ssd_ref_ctc_draft", "ssd_ref_entropy_gate", "ssd_ref_verify",
                     "ssd_ref_set_threads", "ssd_ref_threshold_sweep", "ssd_ref_assemble",
                     "ssd_ref_greedy_step"):
            getattr(_lib, name).restype = C.c_int32
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dtype_code(logits):
    if logits.dtype == np.float32:
        return F32
    if logits.dtype == np.uint16:
        return BF16
    raise TypeError("logits must be float32 or uint16 (bf16 bit patterns)")


def set_threads(n: int) -> int:
    return int(lib().ssd_ref_set_threads(C.c_int32(n)))


def row_stats(row, want_logprob=False):
    """(lse, entropy, argmax[, logprob]) of one row of logits (Eq. 2, Eq. 3)."""
    row = np.ascontiguousarray(row)
    V = row.shape[0]
    lse, H, arg = C.c_double(), C.c_double(), C.c_int32()
    lp = np.empty(V, np.float64) if want_logprob else None
    ok = lib().ssd_ref_row_stats(_p(row), C.c_int(_dtype_code(row)), C.c_int64(0), C.c_int32(V),
                                 C.byref(lse), C.byref(H), C.byref(arg), _p(lp))
    out = (lse.value, H.value, arg.value)
    return out + (lp,) if want_logprob else out + ((bool(ok)),)


def collapse(a, blank_id, cap=None):
    """B(a): merged runs with blanks dropped; returns (tokens[:min(U,cap)], frames, U)."""
    a = np.ascontiguousarray(a, np.int32)
    T = a.shape[0]
    cap = T if cap is None else cap
    out = np.full(max(T, 1), -1, np.int32)
    fr = np.full(max(T, 1), -1, np.int32)
    U = lib().ssd_ref_collapse(_p(a), C.c_int64(T), C.c_int32(blank_id), C.c_int32(cap),
                               _p(out), _p(fr))
    n = min(U, cap)
    return out[:n].copy(), fr[:n].copy(), int(U)


def ctc_draft(logits, V, frame_off, blank_id, max_draft_len, want_logprob=False):
    logits = np.ascontiguousarray(logits)
    N, ld = logits.shape
    frame_off = np.ascontiguousarray(frame_off, np.int64)
    B = frame_off.shape[0] - 1
    o = dict(
        frame_entropy=np.zeros(N, np.float64), frame_argmax=np.full(N, -1, np.int32),
        frame_lse=np.zeros(N, np.float64),
        frame_logprob=np.zeros((N, V), np.float64) if want_logprob else None,
        draft_tokens=np.full(N, -1, np.int32), draft_frames=np.full(N, -1, np.int32),
        draft_len=np.zeros(B, np.int32), draft_full_len=np.zeros(B, np.int32),
        utt_max_entropy=np.zeros(B, np.float64), utt_status=np.zeros(B, np.uint32))
    rc = lib().ssd_ref_ctc_draft(
        _p(logits), C.c_int32(_dtype_code(logits)), C.c_int32(V), C.c_int64(ld), _p(frame_off),
        C.c_int32(B), C.c_int64(N), C.c_int32(blank_id), C.c_int32(max_draft_len),
        _p(o["frame_entropy"]), _p(o["frame_argmax"]), _p(o["frame_lse"]), _p(o["frame_logprob"]),
        _p(o["draft_tokens"]), _p(o["draft_frames"]), _p(o["draft_len"]), _p(o["draft_full_len"]),
        _p(o["utt_max_entropy"]), _p(o["utt_status"]))
    if rc != 0:
        raise ValueError("ssd_ref_ctc_draft rejected its arguments (code %d)" % rc)
    return o


def entropy_gate(frame_entropy, frame_off, tau_ctc):
    frame_entropy = np.ascontiguousarray(frame_entropy, np.float64)
    frame_off = np.ascontiguousarray(frame_off, np.int64)
    B, N = frame_off.shape[0] - 1, frame_entropy.shape[0]
    o = dict(gate_accept=np.zeros(B, np.uint8), max_entropy=np.zeros(B, np.float64),
             argmax_frame=np.zeros(B, np.int32))
    rc = lib().ssd_ref_entropy_gate(_p(frame_entropy), _p(frame_off), C.c_int32(B), C.c_int64(N),
                                    C.c_double(tau_ctc), _p(o["gate_accept"]),
                                    _p(o["max_entropy"]), _p(o["argmax_frame"]))
    if rc != 0:
        raise ValueError("ssd_ref_entropy_gate rejected its arguments (code %d)" % rc)
    return o


def verify(logits, V, tok_off, draft_ids, tau_slm, skip=None):
    logits = np.ascontiguousarray(logits)
    M, ld = logits.shape
    tok_off = np.ascontiguousarray(tok_off, np.int64)
    draft_ids = np.ascontiguousarray(draft_ids, np.int32)
    skip = None if skip is None else np.ascontiguousarray(skip, np.uint8)
    B = tok_off.shape[0] - 1
    o = dict(token_logp=np.full(M, np.nan, np.float64), row_lse=np.full(M, np.nan, np.float64),
             accepted_len=np.zeros(B, np.int32), all_accepted=np.zeros(B, np.uint8),
             utt_status=np.zeros(B, np.uint32))
    rc = lib().ssd_ref_verify(
        _p(logits), C.c_int32(_dtype_code(logits)), C.c_int32(V), C.c_int64(ld), _p(tok_off),
        _p(draft_ids), C.c_int32(B), C.c_int64(M), C.c_double(tau_slm), _p(skip),
        _p(o["token_logp"]), _p(o["row_lse"]), _p(o["accepted_len"]), _p(o["all_accepted"]),
        _p(o["utt_status"]))
    if rc != 0:
        raise ValueError("ssd_ref_verify rejected its arguments (code %d)" % rc)
    return o


def threshold_sweep(utt_max_entropy, token_logp, tok_off, tau_ctc, tau_slm):
    """Gate and first reject for every (tau_ctc[p], tau_slm[p]) pair (Section 3.2's sweep)."""
    h = np.ascontiguousarray(utt_max_entropy, np.float64)
    lp = np.ascontiguousarray(token_logp, np.float64)
    tok_off = np.ascontiguousarray(tok_off, np.int64)
    tc = np.ascontiguousarray(tau_ctc, np.float64)
    ts = np.ascontiguousarray(tau_slm, np.float64)
    B, M, P = tok_off.shape[0] - 1, lp.shape[0], tc.shape[0]
    assert ts.shape[0] == P and h.shape[0] == B
    o = dict(gate_accept=np.zeros((P, B), np.uint8), accepted_len=np.zeros((P, B), np.int32),
             all_accepted=np.zeros((P, B), np.uint8), counts=np.zeros((P, 3), np.int32))
    rc = lib().ssd_ref_threshold_sweep(_p(h), _p(lp), _p(tok_off), C.c_int32(B), C.c_int64(M),
                                       _p(tc), _p(ts), C.c_int32(P), _p(o["gate_accept"]),
                                       _p(o["accepted_len"]), _p(o["all_accepted"]), _p(o["counts"]))
    if rc != 0:
        raise ValueError("ssd_ref_threshold_sweep rejected its arguments (code %d)" % rc)
    return o


def assemble(tokens, tok_off, gate_accept, accepted_len, all_accepted):
    """Eq. 7: final hypotheses and the list of utterances left to the AR pass."""
    tokens = np.ascontiguousarray(tokens, np.int32)
    tok_off = np.ascontiguousarray(tok_off, np.int64)
    B, M = tok_off.shape[0] - 1, tokens.shape[0]
    g = np.ascontiguousarray(gate_accept, np.uint8)
    a = np.ascontiguousarray(accepted_len, np.int32)
    aa = np.ascontiguousarray(all_accepted, np.uint8)
    o = dict(final_tokens=np.full(M, -1, np.int32), final_len=np.zeros(B, np.int32),
             is_final=np.zeros(B, np.uint8), ar_utt=np.full(B, -1, np.int32),
             ar_resume=np.full(B, -1, np.int32))
    n = C.c_int32(0)
    rc = lib().ssd_ref_assemble(_p(tokens), _p(tok_off), C.c_int32(B), C.c_int64(M), _p(g), _p(a),
                                _p(aa), _p(o["final_tokens"]), _p(o["final_len"]),
                                _p(o["is_final"]), C.byref(n), _p(o["ar_utt"]), _p(o["ar_resume"]))
    if rc != 0:
        raise ValueError("ssd_ref_assemble rejected its arguments (code %d)" % rc)
    o["ar_count"] = int(n.value)
    return o


def greedy_step(logits, V):
    """One greedy decoding step (Eq. 6) per row: most likely token and its log-likelihood."""
    logits = np.ascontiguousarray(logits)
    R, ld = logits.shape
    o = dict(next_token=np.zeros(R, np.int32), next_logp=np.zeros(R, np.float64),
             row_lse=np.zeros(R, np.float64), row_bad=np.zeros(R, np.uint8))
    rc = lib().ssd_ref_greedy_step(_p(logits), C.c_int32(_dtype_code(logits)), C.c_int32(V),
                                   C.c_int64(ld), C.c_int64(R), _p(o["next_token"]),
                                   _p(o["next_logp"]), _p(o["row_lse"]), _p(o["row_bad"]))
    if rc != 0:
        raise ValueError("ssd_ref_greedy_step rejected its arguments (code %d)" % rc)
    return o
