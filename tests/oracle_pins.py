"""Pins for the oracle: facts the paper and the mathematics fix, none of them produced by
the oracle itself.  Every function takes an implementation adapter (tests/oracle_impls.py)
and raises AssertionError when the implementation disagrees with the pinned fact."""
import itertools
import math
import os

import numpy as np
import scipy.special
import scipy.stats

from oracle_impls import to_storage

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _rows(path):
    for line in open(os.path.join(GOLDEN, path)):
        line = line.strip()
        if line and not line.startswith("#"):
            yield [f.strip() for f in line.split(";")]


def _close(a, b, tol, what):
    assert abs(a - b) <= tol, "%s: got %r, expected %r (tol %g)" % (what, a, b, tol)


# ---- Eq. 3 left-hand side: entropy; softmax normalisation ---------------------------------

def pin_uniform_entropy(impl):
    """A uniform frame has entropy ln V (values from tests/golden/uniform_entropy.txt)."""
    for V, lnv in _rows("uniform_entropy.txt"):
        V, lnv = int(V), float(lnv)
        for c in (0.0, -3.5, 11.0):
            for dt in ("f32", "bf16"):
                lse, H, arg = impl.row(to_storage(np.full(V, c), dt))
                _close(H, lnv, 1e-12 * max(1, lnv) + 1e-13, "uniform entropy V=%d" % V)
                _close(lse, c + lnv, 1e-12 * (abs(c) + lnv) + 1e-13, "uniform lse V=%d" % V)
                assert arg == 0, "argmax of an all-equal row must be index 0"


def pin_one_hot(impl):
    """A frame with one entry 60 above the rest has entropy ~0 and lse = that entry."""
    for V in (2, 129, 1025):
        x = np.zeros(V)
        x[V // 3] = 60.0
        lse, H, arg = impl.row(to_storage(x, "f32"))
        assert 0.0 <= H < 1e-20, H
        _close(lse, 60.0, 1e-12, "one-hot lse")
        assert arg == V // 3


def pin_k_of_v(impl):
    """Uniform over k entries, the others -inf: entropy ln k, masked entries add nothing."""
    for V, k in ((8, 3), (129, 7), (1025, 64)):
        x = np.full(V, -np.inf)
        idx = np.arange(V)[:: V // k][:k]
        x[idx] = 2.25
        for dt in ("f32", "bf16"):
            lse, H, arg = impl.row(to_storage(x, dt))
            _close(H, math.log(k), 1e-12, "k-of-V entropy")
            _close(lse, 2.25 + math.log(k), 1e-12, "k-of-V lse")
            assert arg == idx[0]


def pin_two_class(impl):
    """Two classes: p = sigmoid(d); entropy is the binary entropy, lse = softplus."""
    for d in (0.0, 0.5, 1.0, 3.0, -2.0, 8.0):
        x = to_storage(np.array([d, 0.0]), "f32")
        dd = float(x[0])
        p = 1.0 / (1.0 + math.exp(-dd))
        hb = -(p * math.log(p) + (1 - p) * math.log(1 - p))
        lse, H, arg = impl.row(x)
        _close(H, hb, 1e-13, "binary entropy d=%g" % d)
        _close(lse, math.log1p(math.exp(dd)) if dd < 30 else dd, 1e-13, "softplus")
        _close(impl.logprob(x)[1], -math.log1p(math.exp(dd)), 1e-13, "-softplus")
        assert arg == (0 if dd >= 0 else 1)


def _planted_row(rng, V, c):
    q = rng.dirichlet(np.full(V, 0.3)) + 1e-9
    q /= q.sum()
    return q, np.log(q) + c


def pin_planted_distribution(impl):
    """Logits x = ln q + c give back log p = ln q, lse = c and entropy -sum q ln q; the
    expected entropy comes from scipy.stats.entropy on q, not from the implementation."""
    rng = np.random.default_rng(11)
    for V in (3, 17, 348):
        for c in (0.0, 4.0, -7.0):
            q, x = _planted_row(rng, V, c)
            xs = to_storage(x, "f32")
            qq = np.exp(xs.astype(np.float64) - c)  # what fp32 storage really holds
            s = qq.sum()
            lse, H, arg = impl.row(xs)
            _close(lse, c + math.log(s), 1e-12, "planted lse")
            _close(H, float(scipy.stats.entropy(qq / s)), 1e-12, "planted entropy")
            np.testing.assert_allclose(impl.logprob(xs), np.log(qq / s), rtol=0, atol=1e-12)
            assert arg == int(np.argmax(qq))
            _close(float(np.exp(impl.logprob(xs)).sum()), 1.0, 1e-12, "sum of p")


def pin_shift_invariance(impl):
    """Adding a constant to a row moves lse by it and leaves entropy and argmax alone.
    Shifts are powers of two times small integers so that fp32 storage stays exact."""
    rng = np.random.default_rng(5)
    x = np.round(rng.normal(size=257) * 64) / 64  # exactly representable
    lse0, H0, a0 = impl.row(to_storage(x, "f32"))
    for c in (8.0, -16.0, 0.5):
        lse, H, a = impl.row(to_storage(x + c, "f32"))
        _close(lse, lse0 + c, 1e-12, "shift lse")
        _close(H, H0, 1e-12, "shift entropy")
        assert a == a0


def pin_entropy_bounds(impl):
    rng = np.random.default_rng(6)
    for V in (1, 2, 31, 33, 129):
        for scale in (0.1, 1.0, 10.0):
            xs = to_storage(rng.normal(size=V) * scale, "bf16")
            _, H, _ = impl.row(xs)
            assert -1e-15 <= H <= math.log(V) + 1e-12


def pin_scipy_special_case(impl):
    """On ordinary finite rows the definitions reduce to scipy's logsumexp / log_softmax /
    entropy (library routines as a special-case check, not as the oracle)."""
    rng = np.random.default_rng(7)
    for V, dt in ((129, "f32"), (1025, "bf16"), (4097, "bf16"), (1000, "f32")):
        xs = to_storage(rng.normal(size=V) * 2.0, dt)
        x64 = (xs.astype(np.uint32) << 16).view(np.float32).astype(np.float64) \
            if dt == "bf16" else xs.astype(np.float64)
        lse, H, arg = impl.row(xs)
        _close(lse, float(scipy.special.logsumexp(x64)), 1e-12, "logsumexp")
        lp = scipy.special.log_softmax(x64)
        np.testing.assert_allclose(impl.logprob(xs), lp, rtol=0, atol=1e-12)
        _close(H, float(scipy.stats.entropy(np.exp(lp))), 1e-11, "entropy")
        assert arg == int(np.argmax(x64))


# ---- Eq. 2: greedy alignment --------------------------------------------------------------

def pin_argmax_ties(impl):
    """Lowest index wins among equal maxima (a choice; both sides take the same)."""
    x = np.array([1.0, 3.0, 3.0, -1.0, 3.0])
    for dt in ("f32", "bf16"):
        assert impl.row(to_storage(x, dt))[2] == 1
    assert impl.row(to_storage(np.array([2.0, 2.0]), "f32"))[2] == 0


def pin_greedy_is_best_alignment(impl):
    """Brute force: among all V^T alignments the one maximising prod_t p(a_t|h_t), Eq. 1's
    summand, is the per-frame argmax path of Eq. 2."""
    rng = np.random.default_rng(3)
    for V, T in ((2, 6), (3, 5), (4, 4)):
        x = rng.normal(size=(T, V)) * 2
        xs = [to_storage(x[t], "f32") for t in range(T)]
        p = [scipy.special.softmax(r.astype(np.float64)) for r in xs]
        best = max(itertools.product(range(V), repeat=T),
                   key=lambda a: math.prod(p[t][a[t]] for t in range(T)))
        assert tuple(impl.row(r)[2] for r in xs) == best


# ---- the mapping B ------------------------------------------------------------------------

def _two_step_collapse(a, blank):
    """The sentence of Section 2.1 taken literally, as two separate passes."""
    merged = [a[i] for i in range(len(a)) if i == 0 or a[i] != a[i - 1]]
    return [s for s in merged if s != blank]


def pin_collapse_hand_cases(impl):
    for align, expect, why in _rows("collapse_cases.txt"):
        a = [int(s) for s in align.split()]
        e = [int(s) for s in expect.split()]
        assert [int(v) for v in impl.collapse(a, 0)] == e, (a, why)


def pin_collapse_brute_force(impl):
    """All sequences over 3 symbols up to length 7, against the two-pass reading; plus the
    invariants U <= T and no blank in the output."""
    for blank in (0, 2):
        for T in range(1, 8):
            for a in itertools.product(range(3), repeat=T):
                got = [int(v) for v in impl.collapse(list(a), blank)]
                assert got == _two_step_collapse(list(a), blank), (a, blank)
                assert len(got) <= T and blank not in got


def pin_collapse_reexpansion(impl):
    """B is idempotent on its own output once a blank is re-inserted between neighbours."""
    rng = np.random.default_rng(9)
    for _ in range(50):
        a = rng.integers(0, 5, size=int(rng.integers(1, 40))).tolist()
        y = [int(v) for v in impl.collapse(a, 0)]
        spaced = []
        for s in y:
            spaced += [s, 0]
        assert [int(v) for v in impl.collapse(spaced, 0)] == y


# ---- Eq. 3 as a decision -------------------------------------------------------------------

def pin_gate(impl):
    ln129 = math.log(129)
    assert impl.gate([0.0, 0.0, 0.0], 0.5) is True          # all one-hot frames
    assert impl.gate([0.0, ln129, 0.0], 3.0) is False        # one uniform frame
    assert impl.gate([0.0, ln129, 0.0], ln129) is False      # strict <: equality fails
    assert impl.gate([0.0, ln129, 0.0], math.nextafter(ln129, 10)) is True
    assert impl.gate([0.0], 0.0) is False                    # H = 0 against tau = 0
    assert impl.gate([0.1, 0.2, 0.69], 0.7) is True
    assert impl.gate([0.1, 0.2, 0.71], 0.7) is False         # max, not mean
    assert impl.gate([2.9] + [0.0] * 99, 0.7) is False       # one bad frame among many
    assert impl.gate([0.8, 0.1], 0.7) is False               # all frames, not any


# ---- Eq. 5 and the first-reject rule -------------------------------------------------------

def _planted_verify(V, K, draft, probs, c=1.5):
    """Rows x_i = ln q_i + c with q_i[draft_i] = probs[i], the rest spread evenly."""
    x = np.empty((K, V))
    for i in range(K):
        q = np.full(V, (1.0 - probs[i]) / (V - 1))
        q[draft[i]] = probs[i]
        x[i] = np.log(q) + c
    return x


def pin_verify_planted(impl):
    V, K, tau = 50, 9, 0.1
    rng = np.random.default_rng(2)
    draft = rng.integers(0, V, size=K).tolist()
    for plants in ([], [0], [4], [8], [3, 6], [6, 3, 7]):
        probs = [0.6 + 0.03 * i for i in range(K)]
        for r in plants:
            probs[r] = 0.02
        xs = to_storage(_planted_verify(V, K, draft, probs), "f32")
        logp, n, ok = impl.verify(xs, draft, tau)
        want = min(plants) if plants else K
        assert n == want and ok == (not plants), (plants, n, ok)
        np.testing.assert_allclose(logp, np.log(probs), rtol=0, atol=1e-6)


def pin_verify_boundary(impl):
    """p exactly equal to tau is a reject ('<=' in Section 2.3; '>' in Eq. 5): V = 2 with
    equal logits gives p = 0.5 exactly."""
    xs = to_storage(np.zeros((3, 2)), "f32")
    _, n, ok = impl.verify(xs, [0, 1, 0], 0.5)
    assert n == 0 and ok is False
    _, n, ok = impl.verify(xs, [0, 1, 0], math.nextafter(0.5, 0))
    assert n == 3 and ok is True
    # boundary at a later position only: rows 0,1 confident, row 2 on the boundary
    x = np.zeros((3, 2))
    x[0, 0] = x[1, 1] = 9.0
    _, n, ok = impl.verify(to_storage(x, "f32"), [0, 1, 0], 0.5)
    assert n == 2 and ok is False


def pin_verify_empty(impl):
    """An empty draft satisfies Eq. 5 vacuously."""
    _, n, ok = impl.verify(np.zeros((0, 4), np.float32), [], 0.1)
    assert n == 0 and ok is True


def pin_verify_rows_and_columns(impl):
    """Each draft token is scored by its own row and its own column: a matrix whose rows
    carry different planted tokens catches a shifted row or a transposed gather."""
    V, K = 7, 5
    draft = [3, 1, 6, 0, 2]
    x = np.zeros((K, V))
    for i in range(K):
        x[i, draft[i]] = 5.0 + i
    xs = to_storage(x, "f32")
    logp, n, ok = impl.verify(xs, draft, 0.5)
    for i in range(K):
        want = (5.0 + i) - math.log(math.exp(5.0 + i) + (V - 1))
        _close(float(logp[i]), want, 1e-12, "row %d" % i)
    assert n == K and ok is True
    # make row 2 vote for another token: first reject at 2
    x[2, draft[2]] = 0.0
    x[2, 4] = 9.0
    _, n, ok = impl.verify(to_storage(x, "f32"), draft, 0.5)
    assert n == 2 and ok is False


# ---- operating points from one pass (Section 3.2, Table 1 caption) ---------------------------

def pin_sweep_planted(impl):
    """Likelihoods worked by hand: for each tau_SLM the first position with p <= tau."""
    q = [0.9, 0.5, 0.3, 0.15, 0.6, 0.05]
    logp = [math.log(v) for v in q]
    by_tau = {0.0: 6, 0.01: 6, 0.06: 5, 0.1: 5, 0.16: 3, 0.2: 3, 0.31: 2, 0.4: 2, 0.51: 1, 0.7: 1,
              0.91: 0, 0.95: 0}      # thresholds sit strictly between the likelihoods
    h = 1.2
    gates = {0.7: False, 1.2: False, math.nextafter(1.2, 2): True, 3.0: True}
    pairs = [(tc, ts) for tc in gates for ts in by_tau]
    got = impl.sweep(h, logp, pairs)
    assert len(got) == len(pairs)
    for (tc, ts), (g, n) in zip(pairs, got):
        assert g is gates[tc] and n == by_tau[ts], (tc, ts, g, n)
    # the paper's two operating points on this utterance
    assert impl.sweep(h, logp, [(0.7, 0.2), (3.0, 0.1)]) == [(False, 3), (True, 5)]


def pin_sweep_monotone_and_empty(impl):
    rng = np.random.default_rng(5)
    logp = np.log(rng.uniform(0.02, 0.98, size=40)).tolist()
    taus = sorted(rng.uniform(0, 1, size=25).tolist())
    got = impl.sweep(0.5, logp, [(t * 3, t) for t in taus])
    lens = [n for _, n in got]
    assert all(a >= b for a, b in zip(lens, lens[1:]))       # a larger tau_SLM rejects earlier
    gates = [g for g, _ in got]
    assert gates == sorted(gates)                            # a larger tau_CTC accepts more
    for t, (_, n) in zip(taus, got):                         # definition, position by position
        assert all(math.exp(v) > t for v in logp[:n]) and (n == 40 or math.exp(logp[n]) <= t)
    assert impl.sweep(0.0, [], [(0.0, 0.5), (0.1, 0.5)]) == [(False, 0), (True, 0)]


# ---- Eq. 7 -----------------------------------------------------------------------------------

def pin_assemble_cases(impl):
    draft = [7, 8, 9, 10]
    ok = [math.log(0.8)] * 4
    bad2 = [math.log(0.8), math.log(0.7), math.log(0.01), math.log(0.9)]
    bad0 = [math.log(0.05)] + ok[1:]
    assert impl.assemble(draft, True, bad2, 0.1) == (draft, False)      # Eq. 3 holds
    assert impl.assemble(draft, False, ok, 0.1) == (draft, False)       # Eq. 5 holds
    assert impl.assemble(draft, True, ok, 0.1) == (draft, False)
    assert impl.assemble(draft, False, bad2, 0.1) == ([7, 8], True)     # prefix before j
    assert impl.assemble(draft, False, bad0, 0.1) == ([], True)
    assert impl.assemble([], False, [], 0.1) == ([], False)             # vacuous Eq. 5
    last = ok[:3] + [math.log(0.0999)]                                  # only the last token fails
    assert impl.assemble(draft, False, last, 0.1) == ([7, 8, 9], True)


# ---- Eq. 6, one step -------------------------------------------------------------------------

def pin_greedy_planted(impl):
    rng = np.random.default_rng(9)
    for V in (1, 2, 17, 300):
        q = rng.dirichlet(np.ones(V))
        x = to_storage(np.log(q) + 2.5, "f32")
        v, lp = impl.greedy(x)
        assert v == int(np.argmax(q))
        _close(lp, math.log(q.max()), 1e-6, "greedy logp V=%d" % V)
    x = np.zeros(9, np.float32)
    x[[2, 5, 7]] = 4.0                                      # three equal maxima
    v, lp = impl.greedy(x)
    assert v == 2
    _close(lp, 4.0 - math.log(3 * math.exp(4.0) + 6), 1e-12, "tie logp")
    v, lp = impl.greedy(np.array([3.25], np.float32))
    assert v == 0 and abs(lp) < 1e-15
    v, lp = impl.greedy(to_storage(np.array([-1.0, 2.0, 0.5]), "bf16"))
    assert v == 1
    _close(lp, 2.0 - math.log(math.exp(-1.0) + math.exp(2.0) + math.exp(0.5)), 1e-12, "bf16 row")


ALL_PINS = [v for k, v in sorted(globals().items()) if k.startswith("pin_")]
