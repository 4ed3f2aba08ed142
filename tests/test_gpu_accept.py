"""Parity of the CUDA accept/resample kernel against the CPU oracle: accepted_len and next_token
bit-exact on the same fp32 probabilities and uniforms, outside the draws the oracle flags as
within 1e-6 of the p/q threshold or 1e-9 Z of a CDF boundary (counted and printed)."""
import numpy as np
import pytest

import oracle
import tts_inputs as ti
from gpu_harness import run_accept

pytestmark = pytest.mark.gpu


def check(case, what, designed_near=False):
    acc_o, nxt_o, near = oracle.accept(case.p_target, case.q_draft, case.draft_tokens, case.uniforms)
    acc_g, nxt_g = run_accept(case)
    clean = near == 0
    n_near = int((~clean).sum())
    print(f"{what}: {case.n_branches} branches, {n_near} near-threshold draws excluded")
    if designed_near:
        # inputs placed on the threshold on purpose: the accept test is one fp32 multiply on both
        # sides, so accepted_len must agree even there
        assert np.array_equal(acc_g, acc_o), what
        clean = (near & 2) == 0
    else:
        assert n_near <= max(2, case.n_branches // 100)
    assert np.array_equal(acc_g[clean], acc_o[clean]), what
    assert np.array_equal(nxt_g[clean], nxt_o[clean]), what
    # flagged draws must still be valid: same accepted_len unless flag bit 0, token adjacent in CDF order
    assert ((acc_g >= 0) & (acc_g <= case.gamma)).all()
    assert ((nxt_g >= 0) & (nxt_g < case.vocab)).all()
    return acc_g, nxt_g


def test_tiny_config():
    check(ti.make_accept_case(4, 3, 1024, 2.0, seed=0x5EED), "tiny")


def test_3b_config():
    check(ti.make_accept_case(8, 4, 151936, 3.0, seed=0x5EED + 1), "3b")


def test_32b_config():
    check(ti.make_accept_case(16, 3, 152064, 3.0, seed=0x5EED + 2), "32b")


def test_high_acceptance_inputs():
    """Draft = target + noise: acceptance in the range the paper reports (Appendix A.1), so both the
    residual and the bonus branch of the final draw are exercised."""
    case = ti.make_accept_case(64, 5, 32768, 3.0, seed=5, draft_noise=0.5)
    acc, _ = check(case, "alpha-matched")
    assert (acc == 5).any() and (acc < 5).any()


@pytest.mark.parametrize("gamma", [0, 1, 2, 7])
@pytest.mark.parametrize("vocab", [4, 16, 132, 1024, 4100])
def test_shapes(gamma, vocab):
    check(ti.make_accept_case(37, gamma, vocab, 2.0, seed=gamma * 100 + vocab, draft_noise=0.7), f"g{gamma}_v{vocab}")


def test_special_cases():
    c = ti.make_accept_case(50, 4, 64, 2.0, seed=3)
    c.q_draft[:] = c.p_target[:, :4]                         # p == q: always accept
    c.uniforms[:, :4] = np.float32(1.0 - 2.0**-24)
    acc, _ = check(c, "p==q", designed_near=True)
    assert (acc == 4).all()
    c = ti.make_accept_case(50, 2, 32, 2.0, seed=5)          # p(x) = 0: reject even at u = 0
    for b in range(50):
        x = int(c.draft_tokens[b, 0])
        c.q_draft[b, 0] = 0.0; c.q_draft[b, 0, x] = 1.0
        c.p_target[b, 0, x] = 0.0
        c.uniforms[b, 0] = 0.0
    acc, nxt = check(c, "p(x)=0", designed_near=True)
    assert (acc == 0).all() and (nxt != c.draft_tokens[:, 0]).all()
    # residual identically zero -> falls back to p_k
    p = np.array([0.0, 0.5, 0.25, 0.25, 0, 0, 0, 0], np.float32)
    for u_last in (0.0, 0.49, 0.51, 0.76):
        cc = ti.AcceptCase(p_target=np.stack([p, p])[None].copy(), q_draft=p[None, None].copy(),
                           draft_tokens=np.array([[0]], np.int32), uniforms=np.array([[0.3, u_last]], np.float32),
                           n_branches=1, gamma=1, vocab=8)
        check(cc, f"zero residual u={u_last}", designed_near=True)


def test_draw_exactly_on_a_boundary_of_the_scan(capsys):
    """Dyadic weights (every sum exact in any order) and a uniform that puts u * Z exactly on the end of the
    vocabulary range that one lane of the scanning warp sums, followed by tokens of zero weight: the draw is the
    first token with weight after that boundary (running sum strictly above u * Z), in the bonus draw and in
    the residual draw alike."""
    V = 152064
    per_lane = -(-(-(-V // 128)) // 32) * 128            # tokens per lane of the 32-lane scan over 128-token tiles
    for lanes in (1, 2, 17):
        edge = lanes * per_lane
        w = np.zeros(V, np.float64)
        w[5:edge:37] = 1.0                                # mass before the boundary
        w[edge + 7::53] = 1.0                             # none in [edge, edge + 7)
        w[w > 0] *= 2.0 ** -18
        before = w[:edge].sum()
        w[0] = 1.0 - w.sum()                              # total mass exactly 1, still dyadic
        u = np.float32(w[:edge].sum())
        assert float(u) == w[:edge].sum() and w.sum() == 1.0 and before > 0
        p = w.astype(np.float32)
        assert (p.astype(np.float64) == w).all()
        # bonus draw (gamma = 0) from p
        bonus = ti.AcceptCase(p_target=p[None, None].copy(), q_draft=np.zeros((1, 0, V), np.float32),
                              draft_tokens=np.zeros((1, 0), np.int32), uniforms=np.array([[u]], np.float32),
                              n_branches=1, gamma=0, vocab=V)
        # residual draw: q takes the draft token's mass away from p, the rest of p - q is w scaled by 1/2
        q = np.zeros(V, np.float32); q[3] = 1.0
        pr = (w / 2).astype(np.float32); pr[3] = 0.0
        resid = ti.AcceptCase(p_target=np.stack([pr, pr])[None].copy(), q_draft=q[None, None].copy(),
                              draft_tokens=np.array([[3]], np.int32), uniforms=np.array([[0.5, u]], np.float32),
                              n_branches=1, gamma=1, vocab=V)
        for case, what in ((bonus, "bonus"), (resid, "residual")):
            acc_o, nxt_o, _ = oracle.accept(case.p_target, case.q_draft, case.draft_tokens, case.uniforms)
            acc_g, nxt_g = run_accept(case)
            assert int(nxt_o[0]) == edge + 7, what       # the oracle's strict crossing
            assert np.array_equal(acc_g, acc_o) and np.array_equal(nxt_g, nxt_o), what


def test_lossless_chi_square_on_gpu():
    """The chi-square pin of the oracle, run through the CUDA kernel: 65536 branches per call."""
    V, per_call, calls = 16, 65536, 8
    rng = np.random.Generator(np.random.Philox(key=[177, 0]))
    base = ti.make_accept_case(1, 1, V, 1.0, seed=41)
    p, q = base.p_target[0], base.q_draft[0]
    counts = np.zeros(V)
    for _ in range(calls):
        toks = ti.sample_from_rows(rng, np.broadcast_to(q[0], (per_call, V))).reshape(per_call, 1)
        case = ti.AcceptCase(p_target=np.broadcast_to(p, (per_call, 2, V)).copy(),
                             q_draft=np.broadcast_to(q, (per_call, 1, V)).copy(), draft_tokens=toks,
                             uniforms=ti.uniforms24(rng, (per_call, 2)), n_branches=per_call, gamma=1, vocab=V)
        acc, nxt = run_accept(case)
        counts += np.bincount(np.where(acc >= 1, toks[:, 0], nxt), minlength=V)
    e = p[0].astype(np.float64) / p[0].sum() * counts.sum()
    assert float(((counts - e) ** 2 / e).sum()) < 37.7
