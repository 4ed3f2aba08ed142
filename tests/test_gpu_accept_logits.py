"""Parity of tts_accept_logits (the accept rule fed with logits) against the oracle: the probabilities
are formed by the same step-by-step fp32 arithmetic on both sides, so accepted_len and next_token must be
bit-exact outside the draws the oracle flags as near a threshold (counted and printed)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2505_19634_b200 as tts
import tts_inputs as ti
from gpu_harness import dev

pytestmark = pytest.mark.gpu


def run_logits(case, ctx=None):
    own = ctx is None
    if own:
        ctx = tts.TtsContext(8, 2, 1, 1, 4, 4)          # tts_accept_logits takes its sizes per call
    as_dev = (lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()) if case.bf16 else dev
    acc = torch.full((case.n_branches,), -7, dtype=torch.int32, device="cuda")
    nxt = torch.full((case.n_branches,), -7, dtype=torch.int32, device="cuda")
    g = case.gamma
    ctx.tts_accept_logits(as_dev(case.target_logits), as_dev(case.draft_logits) if g else None,
                          tts.LOGITS_BF16 if case.bf16 else tts.LOGITS_FP32, dev(case.draft_tokens) if g else None,
                          dev(case.uniforms), case.n_branches, g, case.vocab, acc, nxt)
    torch.cuda.synchronize()
    assert ctx.tts_last_status() == 0
    if own:
        ctx.close()
    return acc.cpu().numpy(), nxt.cpu().numpy()


def check(case, what, designed_near=False):
    acc_o, nxt_o, near = oracle.accept_logits(case.target_logits, case.draft_logits, case.draft_tokens, case.uniforms)
    acc_g, nxt_g = run_logits(case)
    clean = near == 0
    print(f"{what}: {case.n_branches} branches, {int((~clean).sum())} near-threshold draws excluded")
    if designed_near:
        # inputs placed on the threshold on purpose: both sides form the same fp32 probabilities and take the
        # test with one fp32 multiply, so accepted_len must agree even there
        assert np.array_equal(acc_g, acc_o), what
        clean = (near & 2) == 0
    else:
        assert (~clean).sum() <= max(2, case.n_branches // 50)
    assert np.array_equal(acc_g[clean], acc_o[clean]), what
    assert np.array_equal(nxt_g[clean], nxt_o[clean]), what
    assert ((acc_g >= 0) & (acc_g <= case.gamma)).all() and ((nxt_g >= 0) & (nxt_g < case.vocab)).all()
    return acc_g, nxt_g


@pytest.mark.parametrize("bf16", [False, True], ids=["fp32", "bf16"])
def test_workload_shapes(bf16):
    check(ti.make_accept_logits_case(4, 3, 1024, 2.0, seed=0x5EED, bf16=bf16), "tiny")
    check(ti.make_accept_logits_case(8, 4, 151936, 3.0, seed=0x5EED + 1, bf16=bf16), "3b")
    acc, _ = check(ti.make_accept_logits_case(16, 3, 152064, 3.0, seed=0x5EED + 2, draft_noise=0.5, bf16=bf16), "32b, draft = target + noise")
    assert (acc == 3).any() and (acc < 3).any()           # bonus draws and residual draws both occur


@pytest.mark.parametrize("gamma", [0, 1, 2, 7])
@pytest.mark.parametrize("vocab", [4, 16, 132, 1024, 4100])
def test_shapes(gamma, vocab):
    check(ti.make_accept_logits_case(37, gamma, vocab, 2.0, seed=gamma * 100 + vocab, draft_noise=0.7), f"g{gamma}_v{vocab}")
    check(ti.make_accept_logits_case(5, gamma, vocab, 2.0, seed=gamma * 100 + vocab + 1, draft_noise=0.7, bf16=True), f"g{gamma}_v{vocab}_bf16")


def test_ruled_out_tokens_and_identical_logits():
    c = ti.make_accept_logits_case(40, 3, 256, 2.0, seed=7, draft_noise=0.5)
    c.target_logits[:, :, ::3] = -np.inf                       # every third token is ruled out by the target
    acc, nxt = check(c, "-inf logits")
    assert (nxt % 3 != 0).all()                                # never emitted
    for b in range(40):                                        # a draft token the target rules out is rejected
        k = acc[b]
        assert (c.draft_tokens[b, :k] % 3 != 0).all()
    c = ti.make_accept_logits_case(40, 3, 256, 2.0, seed=8)
    c.draft_logits[:] = c.target_logits[:, :3]
    c.uniforms[:, :3] = np.float32(1 - 2.0 ** -24)
    acc, _ = check(c, "p == q", designed_near=True)
    assert (acc == 3).all()


def test_lossless_chi_square_on_gpu():
    """The emitted token at position 0 follows the exact softmax of the target logits: 8 x 65536 branches
    through the kernel, vocab 16, 15 degrees of freedom, threshold 37.7 (p = 0.001)."""
    import scipy.special
    V, per_call, calls = 16, 65536, 8
    rng = np.random.Generator(np.random.Philox(key=[178, 0]))
    tl = (rng.standard_normal((2, V)) * 1.5).astype(np.float32)
    dl = (tl[:1] + rng.standard_normal((1, V)).astype(np.float32)).astype(np.float32)
    p0 = scipy.special.softmax(tl[0].astype(np.float64))
    q0 = scipy.special.softmax(dl[0].astype(np.float64))
    counts = np.zeros(V)
    for _ in range(calls):
        toks = ti.sample_from_rows(rng, np.broadcast_to(q0, (per_call, V))).reshape(per_call, 1)
        case = ti.AcceptLogitsCase(target_logits=np.broadcast_to(tl, (per_call, 2, V)).copy(),
                                   draft_logits=np.broadcast_to(dl, (per_call, 1, V)).copy(), draft_tokens=toks,
                                   uniforms=ti.uniforms24(rng, (per_call, 2)), n_branches=per_call, gamma=1, vocab=V,
                                   bf16=False)
        acc, nxt = run_logits(case)
        counts += np.bincount(np.where(acc >= 1, toks[:, 0], nxt), minlength=V)
    e = p0 * counts.sum()
    assert float(((counts - e) ** 2 / e).sum()) < 37.7


def test_argument_errors():
    ctx = tts.TtsContext(8, 2, 1, 1, 4, 4)
    z = torch.zeros(64, device="cuda", dtype=torch.int32)
    for kw, want in ((dict(dtype=5), -2), (dict(vocab=6), -1), (dict(gamma=-1), -1), (dict(n=0), -1)):
        a = dict(dtype=0, vocab=8, gamma=1, n=1); a.update(kw)
        with pytest.raises(tts.TtsError) as ei:
            ctx.tts_accept_logits(z, z, a["dtype"], z, z, a["n"], a["gamma"], a["vocab"], z, z)
        assert ei.value.status == want, kw
    ctx.close()
