"""Adapters that expose the C oracle, the NumPy mini-oracle and deliberately broken
variants of the latter behind one small interface, so that every pin can be run against
each of them: the two oracles must pass all pins, each planted mistake must fail one."""
import math

import numpy as np

from oracle import mini, ref


def to_storage(x, dtype):
    """fp64/fp32 values -> the storage array an oracle consumes ('f32' or 'bf16')."""
    x = np.asarray(x, np.float32)
    if dtype == "f32":
        return x
    # round-to-nearest-even truncation to the top 16 bits (values here are finite or -inf)
    u = x.view(np.uint32).astype(np.uint64)
    rounded = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    return rounded


class COracle:
    name = "c-oracle"

    def row(self, x):
        lse, H, arg, _ok = ref.row_stats(x)
        return lse, H, arg

    def logprob(self, x):
        return ref.row_stats(x, want_logprob=True)[3]

    def collapse(self, a, blank):
        return list(ref.collapse(np.asarray(a, np.int32), blank)[0]) if len(a) else []

    def gate(self, entropies, tau):
        h = np.asarray(entropies, np.float64)
        off = np.array([0, len(h)], np.int64)
        return bool(ref.entropy_gate(h, off, tau)["gate_accept"][0])

    def verify(self, x2d, draft, tau):
        x2d = np.ascontiguousarray(x2d)
        K = len(draft)
        if K == 0:
            x2d = x2d.reshape(0, max(x2d.shape[1] if x2d.ndim == 2 else 1, 1))
        o = ref.verify(x2d, x2d.shape[1], np.array([0, K], np.int64),
                       np.asarray(draft, np.int32), tau)
        return o["token_logp"], int(o["accepted_len"][0]), bool(o["all_accepted"][0])


    def sweep(self, max_entropy, logp, pairs):
        K = len(logp)
        o = ref.threshold_sweep([max_entropy], np.asarray(logp, np.float64), [0, K],
                                [p[0] for p in pairs], [p[1] for p in pairs])
        for i in range(len(pairs)):
            assert o["counts"][i].sum() == 1
            assert bool(o["all_accepted"][i, 0]) == (o["accepted_len"][i, 0] == K)
        return [(bool(o["gate_accept"][i, 0]), int(o["accepted_len"][i, 0]))
                for i in range(len(pairs))]

    def assemble(self, draft, gate_ok, logp, tau):
        K = len(draft)
        sw = ref.threshold_sweep([0.0], np.asarray(logp, np.float64), [0, K], [1.0], [tau])
        o = ref.assemble(np.asarray(draft, np.int32), [0, K], [1 if gate_ok else 0],
                         sw["accepted_len"][0], sw["all_accepted"][0])
        n = int(o["final_len"][0])
        needs_ar = o["ar_count"] == 1
        assert needs_ar == (not o["is_final"][0])
        if needs_ar:
            assert o["ar_utt"][0] == 0 and o["ar_resume"][0] == n
        return [int(v) for v in o["final_tokens"][:n]], bool(needs_ar)

    def greedy(self, x):
        x = np.ascontiguousarray(x)
        o = ref.greedy_step(x.reshape(1, -1), x.shape[0])
        return int(o["next_token"][0]), float(o["next_logp"][0])


class MiniOracle:
    name = "numpy-mini-oracle"

    def sweep(self, max_entropy, logp, pairs):
        with np.errstate(over="ignore"):
            return [(bool(g), int(n)) for g, n in mini.sweep(max_entropy, np.exp(np.asarray(logp, np.float64)), pairs)]

    def assemble(self, draft, gate_ok, logp, tau):
        return mini.final_hypothesis(draft, gate_ok, np.exp(np.asarray(logp, np.float64)), tau)

    def greedy(self, x):
        return mini.greedy_token(mini.widen(x))

    def row(self, x):
        x = mini.widen(x)
        logp, p = mini.log_softmax(x)
        lse = float(x[np.argmax(x)] - logp[np.argmax(x)])
        return lse, mini.frame_entropy(x), int(np.argmax(x))

    def logprob(self, x):
        return mini.log_softmax(mini.widen(x))[0]

    def collapse(self, a, blank):
        return mini.collapse(a, blank)

    def gate(self, entropies, tau):
        return mini.gate(entropies, tau)

    def verify(self, x2d, draft, tau):
        x = mini.widen(x2d)
        p = mini.token_likelihoods(x, draft)
        with np.errstate(divide="ignore"):
            logp = np.log(p)
        n = mini.accepted_prefix(p, tau)
        return logp, n, n == len(draft)


# ---- planted mistakes (each must be caught by at least one pin) -------------------------

class _Mutant(MiniOracle):
    pass


class EntropyWrongSign(_Mutant):
    name = "mutant: entropy with the sign dropped"

    def row(self, x):
        lse, H, a = super().row(x)
        return lse, -H, a


class EntropyBase2(_Mutant):
    name = "mutant: entropy in bits"

    def row(self, x):
        lse, H, a = super().row(x)
        return lse, H / math.log(2.0), a


class EntropyDropsLseTerm(_Mutant):
    name = "mutant: entropy uses unnormalised log (x - max) instead of log p"

    def row(self, x):
        xx = mini.widen(x)
        lse, _, a = super().row(x)
        _, p = mini.log_softmax(xx)
        keep = p > 0
        return lse, float(-(p[keep] * (xx[keep] - xx.max())).sum()), a


class LseWithoutMax(_Mutant):
    name = "mutant: lse forgets to add the max back"

    def row(self, x):
        xx = mini.widen(x)
        _, H, a = super().row(x)
        return float(np.log(np.exp(xx - xx.max()).sum())), H, a

    def logprob(self, x):
        xx = mini.widen(x)
        return xx - np.log(np.exp(xx - xx.max()).sum())

    def verify(self, x2d, draft, tau):
        x = mini.widen(x2d)
        logp = np.array([self.logprob(x[i])[draft[i]] for i in range(len(draft))])
        n = mini.accepted_prefix(np.exp(logp), tau)
        return logp, n, n == len(draft)


class ArgmaxLastOnTies(_Mutant):
    name = "mutant: argmax returns the last maximiser"

    def row(self, x):
        lse, H, _ = super().row(x)
        xx = mini.widen(x)
        return lse, H, int(len(xx) - 1 - np.argmax(xx[::-1]))


class ArgminInsteadOfArgmax(_Mutant):
    name = "mutant: argmin"

    def row(self, x):
        lse, H, _ = super().row(x)
        return lse, H, int(np.argmin(mini.widen(x)))


class CollapseBlanksFirst(_Mutant):
    name = "mutant: collapse drops blanks before merging duplicates"

    def collapse(self, a, blank):
        no_blank = [int(v) for v in a if v != blank]
        out = []
        for v in no_blank:
            if not out or out[-1] != v:
                out.append(v)
        return out


class CollapseKeepsBlanks(_Mutant):
    name = "mutant: collapse merges runs but keeps blanks"

    def collapse(self, a, blank):
        out = []
        for v in a:
            if not out or out[-1] != v:
                out.append(int(v))
        return out


class CollapseNoMerge(_Mutant):
    name = "mutant: collapse only drops blanks"

    def collapse(self, a, blank):
        return [int(v) for v in a if v != blank]


class GateNonStrict(_Mutant):
    name = "mutant: gate uses <="

    def gate(self, entropies, tau):
        return all(h <= tau for h in entropies)


class GateMean(_Mutant):
    name = "mutant: gate compares the mean entropy"

    def gate(self, entropies, tau):
        return (sum(entropies) / max(len(entropies), 1)) < tau


class GateAny(_Mutant):
    name = "mutant: gate accepts if any frame is below"

    def gate(self, entropies, tau):
        return any(h < tau for h in entropies) or len(entropies) == 0


class VerifyStrictReject(_Mutant):
    name = "mutant: reject uses p < tau"

    def verify(self, x2d, draft, tau):
        logp, _, _ = super().verify(x2d, draft, tau)
        bad = [i for i, lp in enumerate(logp) if math.exp(lp) < tau]
        n = min(bad) if bad else len(draft)
        return logp, n, n == len(draft)


class VerifyOneBased(_Mutant):
    name = "mutant: accepted length off by one (returns the paper's 1-based j)"

    def verify(self, x2d, draft, tau):
        logp, n, ok = super().verify(x2d, draft, tau)
        return logp, (n if ok else n + 1), ok


class VerifyLastReject(_Mutant):
    name = "mutant: takes the last rejected position"

    def verify(self, x2d, draft, tau):
        logp, _, _ = super().verify(x2d, draft, tau)
        bad = [i for i, lp in enumerate(logp) if math.exp(lp) <= tau]
        n = max(bad) if bad else len(draft)
        return logp, n, n == len(draft)


class VerifyTransposedGather(_Mutant):
    name = "mutant: gathers x[draft_i, i] (transposed operand)"

    def verify(self, x2d, draft, tau):
        x = mini.widen(x2d)
        K = len(draft)
        p = []
        for i in range(K):
            r, c = (draft[i] % x.shape[0], i % x.shape[1])
            p.append(mini.log_softmax(x[r])[1][c])
        n = mini.accepted_prefix(p, tau)
        with np.errstate(divide="ignore"):
            return np.log(np.array(p)), n, n == K


class VerifyShiftedRow(_Mutant):
    name = "mutant: scores draft token i with row i-1"

    def verify(self, x2d, draft, tau):
        x = mini.widen(x2d)
        K = len(draft)
        p = [mini.log_softmax(x[max(i - 1, 0)])[1][draft[i]] for i in range(K)]
        n = mini.accepted_prefix(p, tau)
        with np.errstate(divide="ignore"):
            return np.log(np.array(p)), n, n == K


class SweepNonStrictGate(_Mutant):
    name = "mutant: sweep gate uses <="

    def sweep(self, max_entropy, logp, pairs):
        return [(max_entropy <= tc, n) for (tc, _), (_, n) in zip(pairs, super().sweep(max_entropy, logp, pairs))]


class SweepIgnoresPairIndex(_Mutant):
    name = "mutant: sweep evaluates every pair with the first pair's thresholds"

    def sweep(self, max_entropy, logp, pairs):
        return super().sweep(max_entropy, logp, [pairs[0]] * len(pairs))


class SweepComparesLogpWithTau(_Mutant):
    name = "mutant: sweep compares the log-likelihood with tau itself"

    def sweep(self, max_entropy, logp, pairs):
        out = []
        for tc, ts in pairs:
            bad = [i for i, lp in enumerate(logp) if lp <= ts]
            out.append((max_entropy < tc, min(bad) if bad else len(logp)))
        return out


class AssembleKeepsRejectedToken(_Mutant):
    name = "mutant: assembled prefix includes the rejected token"

    def assemble(self, draft, gate_ok, logp, tau):
        toks, ar = super().assemble(draft, gate_ok, logp, tau)
        return (list(draft[:len(toks) + 1]), ar) if ar else (toks, ar)


class AssembleIgnoresGate(_Mutant):
    name = "mutant: a gate-accepted draft that fails verification is sent to the AR pass"

    def assemble(self, draft, gate_ok, logp, tau):
        return super().assemble(draft, False, logp, tau)


class AssembleRequiresBoth(_Mutant):
    name = "mutant: final only if gate AND verification hold"

    def assemble(self, draft, gate_ok, logp, tau):
        toks, ar = super().assemble(draft, False, logp, tau)
        if not gate_ok and not ar:
            return toks, True
        return toks, ar


class GreedyArgmin(_Mutant):
    name = "mutant: greedy step takes the least likely token"

    def greedy(self, x):
        xx = mini.widen(x)
        logp, _ = mini.log_softmax(xx)
        v = int(np.argmin(xx))
        return v, float(logp[v])


class GreedyUnnormalised(_Mutant):
    name = "mutant: greedy step returns the raw logit as log-likelihood"

    def greedy(self, x):
        xx = mini.widen(x)
        v = int(np.argmax(xx))
        return v, float(xx[v])


class GreedyLastOnTies(_Mutant):
    name = "mutant: greedy step returns the last maximiser"

    def greedy(self, x):
        xx = mini.widen(x)
        v = int(len(xx) - 1 - np.argmax(xx[::-1]))
        return v, mini.greedy_token(xx)[1]


ORACLES = [COracle(), MiniOracle()]
MUTANTS = [EntropyWrongSign(), EntropyBase2(), EntropyDropsLseTerm(), LseWithoutMax(),
           ArgmaxLastOnTies(), ArgminInsteadOfArgmax(), CollapseBlanksFirst(),
           CollapseKeepsBlanks(), CollapseNoMerge(), GateNonStrict(), GateMean(), GateAny(),
           VerifyStrictReject(), VerifyOneBased(), VerifyLastReject(), VerifyTransposedGather(),
           VerifyShiftedRow(), SweepNonStrictGate(), SweepIgnoresPairIndex(),
           SweepComparesLogpWithTau(), AssembleKeepsRejectedToken(), AssembleIgnoresGate(),
           AssembleRequiresBoth(), GreedyArgmin(), GreedyUnnormalised(), GreedyLastOnTies()]
