"""NumPy fp64 mini-oracle: a second, independent writing of the paper's definitions.

Test infrastructure only.  Used on tiny inputs to cross-check the C oracle (two separate
statements of the same mathematics must agree) and inside brute-force pins.  It is
vectorised per row and written differently on purpose: log-softmax through probabilities
normalised by their sum, collapse through run-length groups.
"""
import itertools

import numpy as np


def widen(logits):
    """float64 view of an fp32 array or of bf16 bit patterns held in uint16."""
    logits = np.asarray(logits)
    if logits.dtype == np.uint16:
        return (logits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return logits.astype(np.float64)


def log_softmax(x):
    """log p(a | h_t) for one row: the softmax of the CTC / LLM head (Section 2.1, Eq. 5)."""
    x = np.asarray(x, np.float64)
    top = np.max(x)
    e = np.exp(x - top)
    p = e / e.sum()
    with np.errstate(divide="ignore"):
        return np.log(p), p


def frame_entropy(x):
    """Eq. 3, left-hand side, in nats; the 0 log 0 terms are dropped."""
    logp, p = log_softmax(x)
    keep = p > 0
    return float(-(p[keep] * logp[keep]).sum())


def greedy_alignment(x2d):
    """Eq. 2: per-frame argmax (np.argmax returns the first maximiser)."""
    return np.argmax(np.asarray(x2d, np.float64), axis=1).astype(np.int32)


def collapse(a, blank_id):
    """B of Section 2.1: run-length groups first, then blank groups removed."""
    groups = [sym for sym, _ in itertools.groupby(int(v) for v in a)]
    return [g for g in groups if g != blank_id]


def gate(entropies, tau_ctc):
    """Eq. 3 as a decision: every frame strictly below the threshold."""
    return all(h < tau_ctc for h in entropies)


def token_likelihoods(x2d, draft):
    """p(y_i | y_<i, g) of Eq. 5: entry draft[i] of the softmax of row i."""
    return np.array([log_softmax(x2d[i])[1][draft[i]] for i in range(len(draft))], np.float64)


def accepted_prefix(likelihoods, tau_slm):
    """Section 2.3: j = min{i : p_i <= tau} (1-based); returns j-1, or len if no such i."""
    bad = [i for i, p in enumerate(likelihoods) if p <= tau_slm]
    return min(bad) if bad else len(likelihoods)


def sweep(max_entropy, likelihoods, pairs):
    """Section 3.2's operating-point sweep for one utterance: for every (tau_ctc, tau_slm)
    pair, whether the gate passes and how long the verified prefix is."""
    return [(max_entropy < tc, accepted_prefix(likelihoods, ts)) for tc, ts in pairs]


def final_hypothesis(draft, gate_ok, likelihoods, tau_slm):
    """Eq. 7 for one utterance: (tokens that are final so far, needs the AR pass?)."""
    j = accepted_prefix(likelihoods, tau_slm)
    if gate_ok or j == len(draft):
        return list(draft), False
    return list(draft[:j]), True


def greedy_token(x):
    """Eq. 6, one step: the most likely token (first maximiser) and its log-likelihood."""
    logp, p = log_softmax(x)
    v = int(np.argmax(p))
    return v, float(logp[v])
