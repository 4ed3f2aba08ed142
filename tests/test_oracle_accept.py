"""Pins for the accept/resample oracle: range, special cases, exact enumeration on a tiny
vocabulary with rational arithmetic, acceptance probabilities and the lossless property
(Section 2 "Speculative decoding": verification is lossless) by Monte Carlo."""
from fractions import Fraction
from itertools import product

import numpy as np
import pytest

import oracle
import tts_inputs as ti


def test_accepted_len_in_range_and_token_valid():
    for gamma in (0, 1, 3, 5):
        c = ti.make_accept_case(64, gamma, 257, 2.0, seed=gamma)
        acc, nxt, _ = oracle.accept(c.p_target, c.q_draft, c.draft_tokens, c.uniforms)
        assert ((acc >= 0) & (acc <= gamma)).all()
        assert ((nxt >= 0) & (nxt < 257)).all()
        # the emitted token always has positive residual / target mass
        for b in range(64):
            k = acc[b]
            if k < gamma:
                assert c.p_target[b, k, nxt[b]] > c.q_draft[b, k, nxt[b]]
            else:
                assert c.p_target[b, gamma, nxt[b]] > 0


def test_identical_distributions_always_accept():
    c = ti.make_accept_case(200, 4, 64, 2.0, seed=3)
    c.q_draft[:] = c.p_target[:, :4]
    c.uniforms[:, :4] = np.float32(1.0 - 2.0**-24)          # the hardest uniforms
    acc, nxt, _ = oracle.accept(c.p_target, c.q_draft, c.draft_tokens, c.uniforms)
    assert (acc == 4).all()
    # bonus token = inverse CDF of p_gamma at u_gamma
    for b in range(200):
        cdf = np.cumsum(c.p_target[b, 4].astype(np.float64))
        t = float(c.uniforms[b, 4]) * cdf[-1]
        assert nxt[b] == np.searchsorted(cdf, t, side="right")


def test_zero_target_probability_rejects_and_is_never_resampled():
    V, N = 32, 50
    c = ti.make_accept_case(N, 2, V, 2.0, seed=5)
    for b in range(N):
        x = int(c.draft_tokens[b, 0])
        c.q_draft[b, 0] = 0.0; c.q_draft[b, 0, x] = 1.0       # draft is certain of x
        c.p_target[b, 0, x] = 0.0                             # target says impossible
        c.uniforms[b, 0] = 0.0                                # even u = 0 must not accept
    acc, nxt, _ = oracle.accept(c.p_target, c.q_draft, c.draft_tokens, c.uniforms)
    assert (acc == 0).all()
    assert (nxt != c.draft_tokens[:, 0]).all()


def test_zero_draft_probability_with_positive_target_accepts():
    c = ti.make_accept_case(8, 1, 16, 2.0, seed=6)
    for b in range(8):
        c.q_draft[b, 0, c.draft_tokens[b, 0]] = 0.0
        c.uniforms[b, 0] = np.float32(1.0 - 2.0**-24)
    acc, _, _ = oracle.accept(c.p_target, c.q_draft, c.draft_tokens, c.uniforms)
    assert (acc == 1).all()


def test_residual_all_zero_falls_back_to_target():
    """p == q at the rejected position can only reject through p(x) = 0; then r = p_k."""
    V = 8
    p = np.array([0.0, 0.5, 0.25, 0.25, 0, 0, 0, 0], np.float32)
    P = np.stack([p, p])[None]                  # gamma = 1
    Q = p[None, None].copy()
    toks = np.array([[0]], np.int32)            # p(0) = 0 -> reject, residual identically 0
    for u_last, want in ((0.0, 1), (0.49, 1), (0.5, 2), (0.76, 3)):
        U = np.array([[0.3, u_last]], np.float32)
        acc, nxt, _ = oracle.accept(P, Q, toks, U)
        assert acc[0] == 0 and nxt[0] == want


def _exact_rule(p, q, toks, u):
    """The rule in exact rational arithmetic on dyadic inputs (no rounding anywhere)."""
    gamma = len(toks)
    k = gamma
    for i in range(gamma):
        pi, qi = Fraction(float(p[i][toks[i]])), Fraction(float(q[i][toks[i]]))
        if not (pi > 0 and Fraction(float(u[i])) * qi <= pi):
            k = i
            break
    if k < gamma:
        r = [max(Fraction(0), Fraction(float(a)) - Fraction(float(b))) for a, b in zip(p[k], q[k])]
        if sum(r) == 0:
            r = [Fraction(float(a)) for a in p[k]]
    else:
        r = [Fraction(float(a)) for a in p[gamma]]
    t = Fraction(float(u[gamma])) * sum(r)
    c = Fraction(0)
    for x, rx in enumerate(r):
        c += rx
        if c > t:
            return k, x
    raise AssertionError("u < 1 always leaves a token")


def test_exhaustive_grid_against_exact_rational_rule():
    """vocab 4, gamma 2, probabilities on a 1/64 grid, every uniform on a 1/16 grid and every
    draft-token pair: all quantities are exact in fp32, so the oracle must agree exactly."""
    rng = np.random.default_rng(8)
    def dist():
        cuts = np.sort(rng.integers(0, 65, size=3))
        parts = np.diff(np.concatenate([[0], cuts, [64]]))
        return (parts / 64.0).astype(np.float32)
    for _ in range(6):
        p = np.stack([dist() for _ in range(3)])
        q = np.stack([dist() for _ in range(2)])
        cases = [(x0, x1, a, b, c) for x0, x1 in product(range(4), repeat=2)
                 for a, b, c in product(range(16), repeat=3)]
        n = len(cases)
        P = np.broadcast_to(p, (n, 3, 4)).copy()
        Q = np.broadcast_to(q, (n, 2, 4)).copy()
        T = np.array([[c[0], c[1]] for c in cases], np.int32)
        U = np.array([[c[2] / 16, c[3] / 16, c[4] / 16] for c in cases], np.float32)
        acc, nxt, _ = oracle.accept(P, Q, T, U)
        for j in range(0, n, 7):
            k, x = _exact_rule(p, q, T[j], U[j])
            assert (acc[j], nxt[j]) == (k, x), (p, q, T[j], U[j])


def _chi2(counts, probs):
    n = counts.sum()
    e = probs * n
    return float(((counts - e) ** 2 / e).sum())


def test_lossless_chi_square_vocab16():
    """With x ~ q, the token emitted at position 0 (the draft token if accepted, else the
    resampled one) follows p_0; the bonus token given full acceptance follows p_gamma.
    10^6 trials, 15 degrees of freedom, threshold 37.7 (p = 0.001)."""
    V, n = 16, 1_000_000
    rng = np.random.Generator(np.random.Philox(key=[77, 0]))
    base = ti.make_accept_case(1, 1, V, 1.0, seed=41)
    p = base.p_target[0]                      # [2][V]
    q = base.q_draft[0]                       # [1][V]
    P = np.broadcast_to(p, (n, 2, V)).copy()
    Q = np.broadcast_to(q, (n, 1, V)).copy()
    toks = ti.sample_from_rows(rng, np.broadcast_to(q[0], (n, V))).reshape(n, 1)
    U = ti.uniforms24(rng, (n, 2))
    acc, nxt, _ = oracle.accept(P, Q, toks, U)
    first = np.where(acc >= 1, toks[:, 0], nxt)
    c0 = np.bincount(first, minlength=V).astype(np.float64)
    assert _chi2(c0, p[0].astype(np.float64) / p[0].sum()) < 37.7
    full = acc == 1
    cb = np.bincount(nxt[full], minlength=V).astype(np.float64)
    assert full.sum() > 1e5
    assert _chi2(cb, p[1].astype(np.float64) / p[1].sum()) < 37.7
    # a rule that skipped the residual (resampling from p instead) must fail the same test
    wrong = np.where(acc >= 1, toks[:, 0], ti.sample_from_rows(rng, np.broadcast_to(p[0], (n, V))))
    assert _chi2(np.bincount(wrong, minlength=V).astype(np.float64), p[0].astype(np.float64)) > 37.7


def test_acceptance_probabilities_match_closed_form():
    """P(accept at i) = sum_x min(p_i, q_i) and P(accepted_len >= k) = prod_{i<k} beta_i."""
    V, gamma, n = 16, 3, 400_000
    rng = np.random.Generator(np.random.Philox(key=[78, 0]))
    base = ti.make_accept_case(1, gamma, V, 1.0, seed=43)
    p, q = base.p_target[0], base.q_draft[0]
    P = np.broadcast_to(p, (n, gamma + 1, V)).copy()
    Q = np.broadcast_to(q, (n, gamma, V)).copy()
    toks = np.stack([ti.sample_from_rows(rng, np.broadcast_to(q[i], (n, V))) for i in range(gamma)], 1)
    U = ti.uniforms24(rng, (n, gamma + 1))
    acc, _, _ = oracle.accept(P, Q, toks, U)
    beta = np.minimum(p[:gamma].astype(np.float64), q.astype(np.float64)).sum(axis=1)
    surv = 1.0
    for k in range(1, gamma + 1):
        surv *= beta[k - 1]
        got = (acc >= k).mean()
        sigma = np.sqrt(surv * (1 - surv) / n)
        assert abs(got - surv) < 4 * sigma, (k, got, surv)


def test_near_threshold_flags():
    V = 8
    p = np.full((1, 2, V), 0.125, np.float32)
    q = np.full((1, 1, V), 0.25, np.float32); q[0, 0, 4:] = 0.0
    toks = np.array([[1]], np.int32)
    # u*q == p exactly at u = 0.5: accepted (<=) and flagged
    acc, nxt, near = oracle.accept(p, q, toks, np.array([[0.5, 0.3]], np.float32))
    assert acc[0] == 1 and near[0] & 1
    acc, _, near = oracle.accept(p, q, toks, np.array([[0.5 + 2.0**-20, 0.3]], np.float32))
    assert acc[0] == 0 and near[0] & 1
    acc, _, near = oracle.accept(p, q, toks, np.array([[0.75, 0.3]], np.float32))
    assert acc[0] == 0 and not (near[0] & 1)
    # bonus draw exactly on a CDF boundary (u = 0.25 -> t = C_1): strict > picks token 2, flagged
    acc, nxt, near = oracle.accept(p, q, toks, np.array([[0.1, 0.25]], np.float32))
    assert acc[0] == 1 and nxt[0] == 2 and near[0] & 2
