"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random numbers and places boosted entries; it contains none of the
method's arithmetic (no softmax, entropy, argmax, collapse or acceptance rule), so that the
CUDA library and the CPU oracle can both be fed from it without sharing anything else.

The paper measures on speech corpora with a trained CTC encoder and LLM (Section 3); neither
is available offline, so these generators stand in for them.  Shapes follow the paper where
it gives them: 50 CTC frames per second of audio (Section 3.1), bf16 logits and ragged,
length-varied batches (Section 3.2), a mix of gate-accepted, verify-accepted and rejected
utterances (the %C / %L columns of Table 1).

Two ways of placing the boosted ("winner") logit of a row over unit-normal noise:
  literal   winner = noise + boost;
  anchored  winner = ln(V) + 1/2 + boost, where ln(V) + 1/2 is the expected log-sum-exp of V
            unit-normal logits, so that `boost` is (up to sampling noise) the winner's log-odds
            against the rest of the row.  This variant makes the thresholds of Table 1 bite:
            confident frames pass the entropy gate, planted reject rows fail Eq. 5 and the
            others pass it.
Throughput does not depend on the values; decisions are always taken from the oracle.
"""
import math
from dataclasses import dataclass, replace
from typing import List, Optional, Tuple

import torch

_ROW_CHUNK_BYTES = 256 << 20  # fp32 scratch per generation chunk (fixed: part of the recipe)


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    t_dist: str                    # 'const' | 'uniform' | 'lognormal'
    t_lo: int
    t_hi: int
    V_ctc: int
    V_llm: int
    dtype: str                     # 'f32' | 'bf16'
    max_draft_len: int
    tau_ctc: float
    tau_slm: float = 0.1
    blank_id: int = 0
    p_blank: float = 0.6
    boost_lo: float = 2.0          # per-frame winner boost m ~ U(boost_lo, boost_hi)
    boost_hi: float = 12.0
    flat_frac: float = 0.0         # fraction of frames with a flattened boost m ~ U(0, 1)
    confident_frac: float = 0.0    # fraction of utterances whose frames all use m ~ U(8, 12)
    reject_mode: str = "one"       # 'one' | 'uniform_or_none' | 'fraction'
    p_no_reject: float = 0.0
    variant: str = "anchored"      # 'anchored' | 'literal'
    seed: int = 0
    t_mu: float = math.log(600.0)  # lognormal parameters (ln T ~ N(t_mu, t_sigma^2), clipped)
    t_sigma: float = 0.75


def _torch_dtype(name: str):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


# The five configurations of the benchmark definition, by index.
CONFIGS = {
    0: Workload("cfg0_tiny", B=1, t_dist="const", t_lo=200, t_hi=200, V_ctc=129, V_llm=32000,
                dtype="f32", max_draft_len=50, tau_ctc=0.5, reject_mode="one", seed=0),
    1: Workload("cfg1_b32", B=32, t_dist="uniform", t_lo=250, t_hi=750, V_ctc=1025, V_llm=49152,
                dtype="bf16", max_draft_len=200, tau_ctc=0.7, flat_frac=0.10,
                reject_mode="uniform_or_none", p_no_reject=0.30, seed=1),
    2: Workload("cfg2_b128", B=128, t_dist="uniform", t_lo=500, t_hi=1500, V_ctc=1025,
                V_llm=100352, dtype="bf16", max_draft_len=400, tau_ctc=0.7, flat_frac=0.05,
                confident_frac=0.5, reject_mode="uniform_or_none", p_no_reject=0.30, seed=2),
    3: Workload("cfg3_b512", B=512, t_dist="lognormal", t_lo=100, t_hi=3000, V_ctc=4097,
                V_llm=152064, dtype="bf16", max_draft_len=600, tau_ctc=0.7, flat_frac=0.10,
                reject_mode="fraction", seed=3),
}


# The paper's own shape (Section 3.1 / 3.2): a 348-symbol character CTC head, 50 frames per
# second of 5-30 s utterances, batches of length-sorted utterances under a 50,000-token budget,
# and the two operating points of Table 1.  The value mix follows the table's Open ASR averages:
# high accuracy (tau_CTC 0.7, tau_SLM 0.2) accepts about 14 % of the utterances at the gate and
# 47 % at verification; high RTFx (tau_CTC 3.0, tau_SLM 0.1) gates close to all of them.
CONFIGS[5] = Workload("paper_high_accuracy", B=512, t_dist="lognormal", t_lo=250, t_hi=1500,
                      V_ctc=348, V_llm=49152, dtype="bf16", max_draft_len=1500, tau_ctc=0.7,
                      tau_slm=0.2, flat_frac=0.05, confident_frac=0.14,
                      reject_mode="uniform_or_none", p_no_reject=0.547, seed=5)
CONFIGS[6] = Workload("paper_high_rtfx", B=512, t_dist="lognormal", t_lo=250, t_hi=1500,
                      V_ctc=348, V_llm=49152, dtype="bf16", max_draft_len=1500, tau_ctc=3.0,
                      tau_slm=0.1, boost_lo=3.0, flat_frac=0.0, confident_frac=0.0,
                      reject_mode="uniform_or_none", p_no_reject=0.3, seed=6)
MAX_BATCH_TOKENS = 50000


def length_sorted_batches(lengths: List[int], max_tokens: int = MAX_BATCH_TOKENS) -> List[List[int]]:
    """Section 3.2's batching: utterances sorted by length (longest first), packed in order
    into batches whose total frame count stays within the budget (a batch always takes at least
    one utterance).  Returns the lengths of each batch."""
    out, cur, tot = [], [], 0
    for t in sorted((int(v) for v in lengths), reverse=True):
        if cur and tot + t > max_tokens:
            out.append(cur)
            cur, tot = [], 0
        cur.append(t)
        tot += t
    if cur:
        out.append(cur)
    return out


def sweep_point(B: int, V_llm: int, dtype: str) -> Workload:
    """One point of the throughput sweep (configuration 4): T = 1000, V_ctc = 1025, 250 draft
    tokens per utterance, generators as configuration 1."""
    return Workload("cfg4_b%d_v%d_%s" % (B, V_llm, dtype), B=B, t_dist="const", t_lo=1000,
                    t_hi=1000, V_ctc=1025, V_llm=V_llm, dtype=dtype, max_draft_len=250,
                    tau_ctc=0.7, flat_frac=0.10, reject_mode="uniform_or_none",
                    p_no_reject=0.30, seed=4)


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (smaller batch, other variant ...)."""
    return replace(w, **kw)


@dataclass
class CtcBatch:
    logits: torch.Tensor           # [N, V_ctc], storage dtype, on `device`
    frame_off: torch.Tensor        # [B+1] int64, host
    winners: torch.Tensor          # [N] int32, host: the boosted symbol of every frame
    boosts: torch.Tensor           # [N] float32, host
    confident: torch.Tensor        # [B] bool, host: utterance drawn as all-confident


@dataclass
class VerifyBatch:
    logits: torch.Tensor           # [M, V_llm]
    tok_off: torch.Tensor          # [B+1] int64, host
    draft_ids: torch.Tensor        # [M] int32, host
    planted_reject: torch.Tensor   # [B] int64, host: position of the planted reject, -1 if none


def _host_gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return g


def draw_lengths(w: Workload) -> List[int]:
    g = _host_gen(w.seed * 7919 + 11)
    if w.t_dist == "const":
        return [w.t_lo] * w.B
    if w.t_dist == "uniform":
        return torch.randint(w.t_lo, w.t_hi + 1, (w.B,), generator=g).tolist()
    if w.t_dist == "lognormal":
        z = torch.randn((w.B,), generator=g, dtype=torch.float64)
        t = torch.exp(w.t_mu + w.t_sigma * z).round().clamp(w.t_lo, w.t_hi)
        return [int(v) for v in t.tolist()]
    raise ValueError(w.t_dist)


def _fill_rows(out: torch.Tensor, cols: torch.Tensor, vals: torch.Tensor, replace_entry: bool,
               gen: torch.Generator) -> None:
    """out[r, :] = N(0,1) noise, then entry cols[r] gets vals[r] (added to, or replacing, it)."""
    n_rows, V = out.shape
    step = max(1, _ROW_CHUNK_BYTES // (4 * V))
    dev = out.device
    for r0 in range(0, n_rows, step):
        r1 = min(n_rows, r0 + step)
        x = torch.randn((r1 - r0, V), generator=gen, device=dev, dtype=torch.float32)
        idx = cols[r0:r1].to(dev, torch.int64).unsqueeze(1)
        v = vals[r0:r1].to(dev, torch.float32).unsqueeze(1)
        if replace_entry:
            x.scatter_(1, idx, v)
        else:
            x.scatter_add_(1, idx, v)
        out[r0:r1] = x.to(out.dtype)


def make_ctc_batch(w: Workload, device, lengths: Optional[List[int]] = None) -> CtcBatch:
    """CTC head logits of a ragged batch: every frame has one boosted symbol, the blank with
    probability p_blank, otherwise a uniformly drawn token."""
    T = draw_lengths(w) if lengths is None else list(lengths)
    B = len(T)
    frame_off = torch.zeros(B + 1, dtype=torch.int64)
    frame_off[1:] = torch.cumsum(torch.tensor(T, dtype=torch.int64), 0)
    N = int(frame_off[-1])
    g = _host_gen(w.seed * 7919 + 23)
    is_blank = torch.rand((N,), generator=g) < w.p_blank
    tokens = torch.randint(0, max(w.V_ctc - 1, 1), (N,), generator=g, dtype=torch.int64)
    tokens = tokens + (tokens >= w.blank_id).to(torch.int64)   # skip over the blank id
    if w.V_ctc == 1:
        tokens.zero_()
    winners = torch.where(is_blank, torch.full_like(tokens, w.blank_id), tokens).to(torch.int32)
    boosts = w.boost_lo + (w.boost_hi - w.boost_lo) * torch.rand((N,), generator=g)
    flat = torch.rand((N,), generator=g) < w.flat_frac
    flat_boost = torch.rand((N,), generator=g)
    boosts = torch.where(flat, flat_boost, boosts)
    confident = torch.rand((B,), generator=g) < w.confident_frac
    conf_boost = 8.0 + 4.0 * torch.rand((N,), generator=g)
    utt_of_frame = torch.repeat_interleave(torch.arange(B), torch.tensor(T, dtype=torch.int64))
    if N:
        boosts = torch.where(confident[utt_of_frame], conf_boost, boosts)
    boosts = boosts.to(torch.float32)
    dev = torch.device(device)
    dg = torch.Generator(device=dev)
    dg.manual_seed(w.seed * 7919 + 37)
    logits = torch.empty((N, w.V_ctc), dtype=_torch_dtype(w.dtype), device=dev)
    anchored = w.variant == "anchored"
    vals = boosts + (math.log(w.V_ctc) + 0.5) if anchored else boosts
    _fill_rows(logits, winners, vals, anchored, dg)
    return CtcBatch(logits, frame_off, winners, boosts, confident)


def make_verify_batch(w: Workload, draft_len: List[int], device) -> VerifyBatch:
    """LLM logits at the draft positions of each utterance: row i of an utterance boosts its
    draft token, except at one planted position where another token is boosted instead."""
    K = [int(k) for k in draft_len]
    B = len(K)
    tok_off = torch.zeros(B + 1, dtype=torch.int64)
    tok_off[1:] = torch.cumsum(torch.tensor(K, dtype=torch.int64), 0)
    M = int(tok_off[-1])
    g = _host_gen(w.seed * 7919 + 41)
    V = w.V_llm
    draft_ids = torch.randint(0, V, (M,), generator=g, dtype=torch.int64)
    u = torch.rand((B,), generator=g, dtype=torch.float64)
    none = torch.rand((B,), generator=g) < w.p_no_reject
    planted = torch.full((B,), -1, dtype=torch.int64)
    for b in range(B):
        if K[b] == 0:
            continue
        if w.reject_mode == "one":
            planted[b] = min(int(u[b] * K[b]), K[b] - 1)
        elif w.reject_mode == "uniform_or_none":
            planted[b] = -1 if bool(none[b]) else min(int(u[b] * K[b]), K[b] - 1)
        elif w.reject_mode == "fraction":
            pos = int(math.floor(float(u[b]) * K[b]))
            planted[b] = pos if pos < K[b] else -1
        else:
            raise ValueError(w.reject_mode)
    boosted = draft_ids.clone()
    other = (draft_ids + 1 + torch.randint(0, max(V - 1, 1), (M,), generator=g)) % V
    for b in range(B):
        if planted[b] >= 0:
            r = int(tok_off[b] + planted[b])
            boosted[r] = other[r]
    boosts = (3.0 + 7.0 * torch.rand((M,), generator=g)).to(torch.float32)
    dev = torch.device(device)
    dg = torch.Generator(device=dev)
    dg.manual_seed(w.seed * 7919 + 53)
    logits = torch.empty((M, V), dtype=_torch_dtype(w.dtype), device=dev)
    anchored = w.variant == "anchored"
    if anchored:
        tau = min(max(w.tau_slm, 1e-6), 1.0 - 1e-6)
        vals = boosts + (math.log(V) + 0.5 + math.log(tau / (1.0 - tau)))
    else:
        vals = boosts
    _fill_rows(logits, boosted, vals, anchored, dg)
    return VerifyBatch(logits, tok_off, draft_ids.to(torch.int32), planted)


def logits_bytes(w: Workload, N: int, M: int) -> Tuple[int, int]:
    """Bytes of CTC and of LLM logits a batch with N frames and M draft positions holds."""
    s = 4 if w.dtype == "f32" else 2
    return N * w.V_ctc * s, M * w.V_llm * s
