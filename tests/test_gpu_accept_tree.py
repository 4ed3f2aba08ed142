"""Parity of tts_accept_tree against the oracle's tree-path rule: accepted_len, last_node and next_token
bit-exact outside the draws the oracle flags as near a threshold; a chain must equal tts_accept; malformed
trees are reported through the device status."""
import numpy as np
import pytest
import torch

import oracle
import paper_2505_19634_b200 as tts
import tts_inputs as ti
from gpu_harness import dev, run_accept

pytestmark = pytest.mark.gpu


def run_tree(case, parents, check_status=True):
    n = case.gamma
    N = case.n_branches
    ctx = tts.TtsContext(8, 2, 1, 1, 4, 4)           # tts_accept_tree takes its sizes per call
    acc = torch.full((N,), -7, dtype=torch.int32, device="cuda")
    last = torch.full((N,), -7, dtype=torch.int32, device="cuda")
    nxt = torch.full((N,), -7, dtype=torch.int32, device="cuda")
    ctx.tts_accept_tree(dev(case.p_target), dev(case.q_draft) if n else None, dev(case.draft_tokens) if n else None,
                        dev(parents) if n else None, dev(case.uniforms), N, n, case.vocab, acc, last, nxt)
    torch.cuda.synchronize()
    st = ctx.tts_last_status()
    ctx.close()
    if check_status:
        assert st == 0
    return acc.cpu().numpy(), last.cpu().numpy(), nxt.cpu().numpy(), st


@pytest.mark.parametrize("n,depth,vocab,seed,N", [(6, 3, 64, 1, 37), (12, 5, 1024, 2, 37), (30, 8, 4100, 3, 37),
                                                    (60, 10, 32768, 4, 37), (64, 64, 132, 5, 37),
                                                    (60, 6, 152064, 6, 8)])        # the tree workload's own shape
def test_trees_match_oracle(n, depth, vocab, seed, N):
    case = ti.make_accept_case(N, n, vocab, 2.0, seed=seed, draft_noise=0.6)
    parents = ti.make_tree_parents(N, n, depth, seed + 100)
    acc_o, last_o, nxt_o, near = oracle.accept_tree(case.p_target, case.q_draft, case.draft_tokens, parents, case.uniforms)
    acc_g, last_g, nxt_g, _ = run_tree(case, parents)
    clean = near == 0
    print(f"tree n={n}: {int((~clean).sum())} near-threshold draws excluded")
    assert (~clean).sum() <= max(2, N // 10)
    assert np.array_equal(acc_g[clean], acc_o[clean])
    assert np.array_equal(last_g[clean], last_o[clean])
    assert np.array_equal(nxt_g[clean], nxt_o[clean])
    assert ((nxt_g >= 0) & (nxt_g < vocab)).all()
    assert acc_o.max() > 0                                  # the case does accept something


@pytest.mark.parametrize("gamma", [0, 1, 3, 7])
def test_chain_equals_tts_accept(gamma):
    case = ti.make_accept_case(33, gamma, 2048, 2.0, seed=gamma + 9, draft_noise=0.5)
    parents = np.tile(np.arange(-1, gamma - 1, dtype=np.int32), (33, 1))
    acc_c, nxt_c = run_accept(case)
    acc_t, last_t, nxt_t, _ = run_tree(case, parents)
    assert np.array_equal(acc_c, acc_t) and np.array_equal(nxt_c, nxt_t)
    assert np.array_equal(last_t, acc_c - 1)


def test_malformed_tree_is_reported():
    case = ti.make_accept_case(4, 6, 64, 2.0, seed=3)
    parents = ti.make_tree_parents(4, 6, 3, 5)
    parents[2, 4] = 5                                       # a parent that comes later
    _, _, nxt, st = run_tree(case, parents, check_status=False)
    assert st == -4                                         # TTS_ERR_DEVICE_BOUNDS
    assert ((nxt >= 0) & (nxt < 64)).all()
