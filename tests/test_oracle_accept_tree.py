"""Pins of the oracle's tree-path accept rule: a chain must reproduce the (separately pinned) chain
oracle; on small trees every pattern of passing and failing nodes is enumerated and compared with the
rule evaluated by hand-written path lists; structural invariants.  The distribution of the emitted token
under the path-selection rule is parity unpinned (stated in the oracle)."""
import itertools

import numpy as np
import pytest

import oracle
import tts_inputs as ti


def chain_case(n_branches, gamma, vocab, seed):
    return ti.make_accept_case(n_branches, gamma, vocab, 2.0, seed)


@pytest.mark.parametrize("gamma,vocab,seed", [(1, 64, 1), (3, 256, 2), (5, 1024, 3), (8, 128, 4)])
def test_chain_tree_is_the_chain_rule(gamma, vocab, seed):
    c = chain_case(32, gamma, vocab, seed)
    parents = np.tile(np.arange(-1, gamma - 1, dtype=np.int32), (32, 1))
    a0, n0, f0 = oracle.accept(c.p_target, c.q_draft, c.draft_tokens, c.uniforms)
    a1, l1, n1, f1 = oracle.accept_tree(c.p_target, c.q_draft, c.draft_tokens, parents, c.uniforms)
    assert np.array_equal(a0, a1) and np.array_equal(n0, n1)
    assert np.array_equal(l1, a0 - 1)
    assert np.array_equal(f0 & 1, f1 & 1)                 # the same tests were near the threshold


# a fixed 6-node tree:      -1 -> 0 -> 1 -> 3
#                                  |    `-> 4
#                                  `-> 2 -> 5
TREE = np.array([-1, 0, 0, 1, 1, 2], np.int32)
PATHS = {3: [0, 1, 3], 4: [0, 1, 4], 5: [0, 2, 5]}       # leaf -> nodes from the root side


def controlled_case(pattern, vocab=8):
    """p, q such that node i passes iff pattern[i]: every node's token has q = 0.5 and p = 0.25, u = 0.25
    passes (0.125 <= 0.25) and u = 0.75 fails (0.375 > 0.25)."""
    n = len(TREE)
    p = np.full((1, n + 1, vocab), 0.75 / (vocab - 1), np.float32)
    q = np.full((1, n, vocab), 0.5 / (vocab - 1), np.float32)
    x = np.array([[i % vocab for i in range(n)]], np.int32)
    for i in range(n):
        par = TREE[i]
        p[0, par + 1, x[0, i]] = 0.25
        q[0, i, x[0, i]] = 0.5
    u = np.array([[0.25 if ok else 0.75 for ok in pattern] + [0.5]], np.float32)
    return p, q, x, u


def test_every_pass_pattern_of_a_small_tree():
    for pattern in itertools.product([False, True], repeat=len(TREE)):
        p, q, x, u = controlled_case(pattern)
        acc, last, nxt, _ = oracle.accept_tree(p, q, x, TREE[None, :], u)
        counts = {}
        for leaf, path in PATHS.items():
            c = 0
            for node in path:
                if not pattern[node]:
                    break
                c += 1
            counts[leaf] = c
        best = max(counts.values())
        leaf = min(l for l, c in counts.items() if c == best)
        assert acc[0] == best
        assert last[0] == (PATHS[leaf][best - 1] if best else -1)
        # the draw: residual of the first failing node of that path, or the leaf's own row
        if best < len(PATHS[leaf]):
            k = PATHS[leaf][best]
            r = np.maximum(p[0, TREE[k] + 1] - q[0, k], 0).astype(np.float64)
        else:
            r = p[0, leaf + 1].astype(np.float64)
        cdf = np.cumsum(r)
        assert nxt[0] == int(np.nonzero(cdf > 0.5 * cdf[-1])[0][0])


def test_structure():
    rng = np.random.default_rng(7)
    n, vocab, N = 12, 64, 16
    parents = ti.make_tree_parents(N, n, 5, 9)
    c = ti.make_accept_case(N, n, vocab, 2.0, 5)           # rows reused as per-node distributions
    acc, last, nxt, _ = oracle.accept_tree(c.p_target, c.q_draft, c.draft_tokens, parents, c.uniforms)
    for b in range(N):
        depth = np.zeros(n, int)
        for i in range(n):
            depth[i] = 1 + (depth[parents[b, i]] if parents[b, i] >= 0 else 0)
        assert 0 <= acc[b] <= depth.max()
        assert (last[b] == -1) == (acc[b] == 0)
        if acc[b]:
            assert depth[last[b]] == acc[b]
        assert 0 <= nxt[b] < vocab
    # u = 0 everywhere: every node with p > 0 passes, so the deepest leaf (lowest index among equals) wins
    u0 = np.zeros_like(c.uniforms)
    p_pos = np.maximum(c.p_target, 1e-6).astype(np.float32)
    acc, last, _, _ = oracle.accept_tree(p_pos, c.q_draft, c.draft_tokens, parents, u0)
    for b in range(N):
        depth = np.zeros(n, int)
        for i in range(n):
            depth[i] = 1 + (depth[parents[b, i]] if parents[b, i] >= 0 else 0)
        has_child = np.zeros(n, bool)
        has_child[parents[b][parents[b] >= 0]] = True
        leaves = [i for i in range(n) if not has_child[i]]
        deepest = max(depth[l] for l in leaves)
        assert acc[b] == deepest and last[b] == min(l for l in leaves if depth[l] == deepest)
    with pytest.raises(ValueError):
        bad = parents.copy(); bad[0, 3] = 7
        oracle.accept_tree(c.p_target, c.q_draft, c.draft_tokens, bad, c.uniforms)
