"""Pins for the oracle's logits -> probabilities step (`oracle.softmax_rows`) and for the accept rule fed
with logits (`oracle.accept_logits`): the exact softmax within the error the stated fp32 arithmetic allows,
invariants, special cases, and the lossless property (Section 2, "Speculative decoding") by Monte Carlo
against the EXACT softmax of the target logits."""
import numpy as np
import scipy.special

import oracle
import tts_inputs as ti


def _exact(logits):
    return scipy.special.softmax(np.asarray(logits, dtype=np.float64), axis=-1)


def test_matches_the_exact_softmax():
    """The largest error is the one rounded fp32 multiply of d = l - max by log2(e): half an ulp of the
    product, about 2^-24 |d| log2(e), i.e. a relative error of 2^-24 |d| in exp(d); the polynomial, the other
    roundings and the normaliser add a few 1e-7.  A dropped or wrong coefficient, a missing maximum or a sign
    error shows at 1e-4 or worse."""
    rng = np.random.default_rng(0)
    for sigma, vocab in ((2.0, 1024), (3.0, 151936), (0.01, 64), (8.0, 4100)):
        l = (rng.standard_normal((3, vocab)) * sigma).astype(np.float32)
        p, ex = oracle.softmax_rows(l), _exact(l)
        big = ex > 1e-30
        d = l.max(-1, keepdims=True).astype(np.float64) - l
        assert (np.abs(p / np.maximum(ex, 1e-300) - 1.0)[big] <= (2.0 ** -23 * d + 4e-7)[big]).all()
        assert (np.abs(p.astype(np.float64).sum(-1) - 1.0) <= 2e-6).all()
        assert np.array_equal(p.argmax(-1), ex.argmax(-1))


def test_special_rows():
    # one finite logit: probability exactly 1; -inf: exactly 0
    l = np.full((1, 16), -np.inf, np.float32); l[0, 5] = 3.25
    p = oracle.softmax_rows(l)
    assert p[0, 5] == 1.0 and (np.delete(p[0], 5) == 0).all()
    # equal logits: uniform, exactly 1/V for a power-of-two V
    assert (oracle.softmax_rows(np.full((2, 64), -7.5, np.float32)) == np.float32(1 / 64)).all()
    # two logits ln 2 apart (in fp32 terms: the closed form 2/3, 1/3 within the stated error)
    p = oracle.softmax_rows(np.array([[np.log(2.0), 0.0]], np.float32))
    assert abs(p[0, 0] - 2 / 3) < 1e-6 and abs(p[0, 1] - 1 / 3) < 1e-6
    # far below the maximum: underflows to exactly 0, never negative or NaN
    p = oracle.softmax_rows(np.array([[0.0, -80.0, -100.0, -3000.0]], np.float32))
    assert p[0, 0] == 1.0 and p[0, 3] == 0.0 and (p >= 0).all() and np.isfinite(p).all()
    assert abs(p[0, 1] / np.exp(-80.0) - 1) < 1e-5


def test_shift_invariance_is_exact():
    """Only differences to the row maximum enter: adding a constant that keeps every logit exactly
    representable leaves the probabilities bit-identical."""
    rng = np.random.default_rng(1)
    l = (rng.integers(-4096, 4096, size=(4, 512)) / 256.0).astype(np.float32)        # multiples of 2^-8
    base = oracle.softmax_rows(l)
    for c in (16.0, -32.0, 1024.0):
        assert np.array_equal(oracle.softmax_rows(l + np.float32(c)), base)


def test_bf16_bits_are_widened_exactly():
    rng = np.random.default_rng(2)
    bits = ti.f32_to_bf16_bits((rng.standard_normal((2, 300)) * 3).astype(np.float32))
    assert np.array_equal(oracle.softmax_rows(bits), oracle.softmax_rows(ti.bf16_bits_to_f32(bits)))


def test_accept_logits_range_and_consistency():
    c = ti.make_accept_logits_case(64, 3, 1000, 2.0, seed=3, draft_noise=0.5)
    acc, nxt, _ = oracle.accept_logits(c.target_logits, c.draft_logits, c.draft_tokens, c.uniforms)
    assert ((acc >= 0) & (acc <= 3)).all() and ((nxt >= 0) & (nxt < 1000)).all()
    assert (acc == 3).any() and (acc < 3).any()
    p = oracle.softmax_rows(c.target_logits)
    q = oracle.softmax_rows(c.draft_logits)
    for b in range(64):                        # the emitted token has positive residual / target mass
        k = acc[b]
        assert (p[b, k, nxt[b]] > q[b, k, nxt[b]]) if k < 3 else (p[b, 3, nxt[b]] > 0)
    # identical target and draft logits: everything is accepted, whatever the uniforms
    c.draft_logits[:] = c.target_logits[:, :3]
    c.uniforms[:, :3] = np.float32(1 - 2.0 ** -24)
    assert (oracle.accept_logits(c.target_logits, c.draft_logits, c.draft_tokens, c.uniforms)[0] == 3).all()


def test_lossless_against_the_exact_softmax_chi_square():
    """Draft tokens drawn from the exact softmax of the draft logits; the token emitted at position 0
    (the draft if accepted, else the resampled one) must follow the EXACT softmax of the target logits:
    chi-square on vocab 16, 400 000 trials, 15 degrees of freedom, threshold 37.7 (p = 0.001)."""
    V, n = 16, 400_000
    rng = np.random.Generator(np.random.Philox(key=[91, 0]))
    tl = (rng.standard_normal((2, V)) * 1.5).astype(np.float32)
    dl = (tl[:1] + rng.standard_normal((1, V)).astype(np.float32)).astype(np.float32)
    p0, q0 = _exact(tl[0]), _exact(dl[0])
    toks = ti.sample_from_rows(rng, np.broadcast_to(q0, (n, V))).reshape(n, 1)
    acc, nxt, _ = oracle.accept_logits(np.broadcast_to(tl, (n, 2, V)).copy(), np.broadcast_to(dl, (n, 1, V)).copy(),
                                       toks, ti.uniforms24(rng, (n, 2)))
    emitted = np.where(acc >= 1, toks[:, 0], nxt)
    counts = np.bincount(emitted, minlength=V)
    e = p0 * n
    assert float(((counts - e) ** 2 / e).sum()) < 37.7
    # acceptance probability = sum_x min(p, q) within 4 sigma
    beta = np.minimum(p0, q0).sum()
    assert abs((acc >= 1).mean() - beta) < 4 * np.sqrt(beta * (1 - beta) / n)
