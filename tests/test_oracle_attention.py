"""Pins for the attention oracle: things the mathematics fixes, checked with code that does
not share the oracle's paged loop (dense numpy matrices, scipy's softmax, closed forms)."""
from dataclasses import replace
from pathlib import Path

import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax

import oracle
import tts_inputs as ti

GOLDEN = Path(__file__).parent / "golden"


def small_shape(**kw):
    base = ti.AttnShape("small", n_q_heads=4, n_kv_heads=2, prefix_len=32, n_branches=3, gamma=2,
                        branch_lens=(19, 3, 40), permute_pages=True, extra_pages=3)
    return replace(base, **kw)


def dense_reference(case, mask_kind=0, tree_parents=None):
    """Brute force: gather each branch into contiguous K, V, build the whole score matrix and
    an explicit 0/-inf mask matrix, dense softmax, dense P @ V.  fp64 numpy."""
    s = case.shape
    R, G, D, ps = s.rows_per_branch, s.group, s.head_dim, s.page_size
    qf = ti.bf16_bits_to_f32(case.q).astype(np.float64)
    kf = ti.bf16_bits_to_f32(case.k_pages).astype(np.float64)
    vf = ti.bf16_bits_to_f32(case.v_pages).astype(np.float64)
    out = np.zeros((s.n_branches, R, s.n_q_heads, D))
    P = case.prefix_len
    for b in range(s.n_branches):
        L = int(case.branch_lens[b])
        T = P + L
        pages = case.block_table[b, :(T + ps - 1) // ps]
        mask = np.full((R, T), -np.inf)
        mask[:, :P] = 0.0
        for i in range(R):
            if mask_kind == 0:
                mask[i, P:P + L - R + i + 1] = 0.0
            else:
                mask[i, P:P + L - R] = 0.0
                a = i
                while a >= 0:
                    mask[i, P + L - R + a] = 0.0
                    a = int(tree_parents[b, a])
        for h in range(s.n_q_heads):
            kvh = h // G
            K = kf[pages, kvh].reshape(-1, D)[:T]
            V = vf[pages, kvh].reshape(-1, D)[:T]
            S = qf[b, :, h, :] @ K.T / np.sqrt(D) + mask
            W = np.exp(S - S.max(axis=1, keepdims=True))
            W /= W.sum(axis=1, keepdims=True)
            out[b, :, h, :] = W @ V
    return out


def run(case, **kw):
    return oracle.verify_attn(case.q, case.k_pages, case.v_pages, case.block_table,
                              case.prefix_len, case.branch_lens, case.shape.gamma, **kw)


@pytest.mark.parametrize("seed", [1, 2, 3])
@pytest.mark.parametrize("kw", [dict(), dict(prefix_len=0), dict(gamma=0, branch_lens=(1, 16, 17)),
                                dict(n_branches=1, branch_lens=(33,), gamma=4),
                                dict(n_q_heads=6, n_kv_heads=1, gamma=3, branch_lens=(4, 5, 64))])
def test_matches_dense_brute_force(seed, kw):
    case = ti.make_attn_case(small_shape(**kw), seed)
    ti.poison_unused_slots(case)          # NaN in every slot no query may read
    got = run(case)
    want = dense_reference(case)
    assert np.isfinite(got).all()
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-13)


def test_softmax_weights_sum_to_one():
    case = ti.make_attn_case(small_shape(), 5)
    _, wsum = run(case, return_weight_sums=True)
    assert np.abs(wsum - 1.0).max() < 1e-12


def test_page_permutation_leaves_result_bit_identical():
    shp = small_shape(permute_pages=False, extra_pages=0)
    a = ti.make_attn_case(shp, 11)
    perm = np.random.default_rng(0).permutation(a.num_pages)
    inv = np.argsort(perm)
    b = ti.make_attn_case(shp, 11)
    b.k_pages = a.k_pages[perm]           # physical page j now holds old page perm[j]
    b.v_pages = a.v_pages[perm]
    b.block_table = np.where(a.block_table >= 0, inv[np.maximum(a.block_table, 0)], -1).astype(np.int32)
    assert np.array_equal(run(a), run(b))


def test_constant_values_give_constant_output():
    case = ti.make_attn_case(small_shape(), 7)
    c = ti.f32_to_bf16_bits(np.array([0.75], np.float32))[0]
    case.v_pages[:] = c
    np.testing.assert_allclose(run(case), 0.75, rtol=0, atol=1e-12)


def test_dominant_key_selects_its_value_row():
    shp = small_shape(n_branches=1, branch_lens=(24,), gamma=0, n_q_heads=2, n_kv_heads=2)
    case = ti.make_attn_case(shp, 9)
    # query head 0 = 8 * e_0 ; key of logical token 37 (private token 5) = 64 * e_0: score
    # 8*64/sqrt(128) = 45.3 above every other key (others are ~N(0, 8^2/128)).
    q = np.zeros((1, 1, 2, 128), np.float32); q[0, 0, :, 0] = 8.0
    case.q = ti.f32_to_bf16_bits(q)
    kf = ti.bf16_bits_to_f32(case.k_pages); kf[..., 0] = 0.0
    page, slot = ti.token_slot(case, 0, 37)
    kf[page, :, slot, 0] = 64.0
    case.k_pages = ti.f32_to_bf16_bits(kf)
    got = run(case)
    vf = ti.bf16_bits_to_f32(case.v_pages).astype(np.float64)
    for h in range(2):
        np.testing.assert_allclose(got[0, 0, h], vf[page, h, slot], atol=1e-12)


def test_reduces_to_textbook_decode_attention():
    """gamma = 0, one branch, no prefix: softmax(q K^T / sqrt(D)) V with a library softmax."""
    shp = small_shape(n_branches=1, prefix_len=0, gamma=0, branch_lens=(50,), n_q_heads=4,
                      n_kv_heads=4, permute_pages=False, extra_pages=0)
    case = ti.make_attn_case(shp, 13)
    got = run(case)
    qf = ti.bf16_bits_to_f32(case.q).astype(np.float64)[0, 0]                   # [H][D]
    K = ti.bf16_bits_to_f32(case.k_pages).astype(np.float64).transpose(1, 0, 2, 3).reshape(4, -1, 128)[:, :50]
    V = ti.bf16_bits_to_f32(case.v_pages).astype(np.float64).transpose(1, 0, 2, 3).reshape(4, -1, 128)[:, :50]
    for h in range(4):
        w = scipy_softmax(K[h] @ qf[h] / np.sqrt(128.0))
        np.testing.assert_allclose(got[0, 0, h], w @ V[h], rtol=1e-11, atol=1e-13)


def test_causal_rows_equal_truncated_single_row_problems():
    """Row i < gamma of a branch equals the gamma' = 0 result for the same query with the
    branch cut to L - (gamma - i) private tokens."""
    shp = small_shape()
    case = ti.make_attn_case(shp, 17)
    full = run(case)
    g = shp.gamma
    for i in range(g + 1):
        sub = ti.make_attn_case(shp, 17)
        sub.shape = replace(shp, gamma=0)
        sub.q = np.ascontiguousarray(case.q[:, i:i + 1])
        sub.branch_lens = (case.branch_lens - (g - i)).astype(np.int32)
        got = oracle.verify_attn(sub.q, sub.k_pages, sub.v_pages, sub.block_table, sub.prefix_len,
                                 sub.branch_lens, 0)
        np.testing.assert_allclose(got[:, 0], full[:, i], rtol=1e-12, atol=1e-14)


def test_sentinel_in_masked_positions_has_no_effect():
    """Huge K/V in the positions a row must not see leave that row unchanged."""
    shp = small_shape()
    a = ti.make_attn_case(shp, 19)
    ref = run(a)
    b = ti.make_attn_case(shp, 19)
    big = ti.f32_to_bf16_bits(np.array([1.0e4], np.float32))[0]
    g = shp.gamma
    for br in range(shp.n_branches):
        L = int(b.branch_lens[br])
        page, slot = ti.token_slot(b, br, b.prefix_len + L - 1)   # last token: only row gamma sees it
        b.k_pages[page, :, slot, :] = big
        b.v_pages[page, :, slot, :] = big
    got = run(b)
    assert np.array_equal(got[:, :g], ref[:, :g])
    assert np.abs(got[:, g] - ref[:, g]).max() > 1.0


def test_tree_mask_chain_equals_causal_and_tree_matches_brute_force():
    shp = small_shape(gamma=5, branch_lens=(19, 6, 40))
    case = ti.make_attn_case(shp, 23)
    chain = np.tile(np.arange(-1, 5, dtype=np.int32), (3, 1))
    assert np.array_equal(run(case), run(case, mask_kind=1, tree_parents=chain))
    parents = ti.make_tree_parents(3, 6, 3, seed=4)
    assert (parents < np.arange(6)).all() and (parents >= -1).all()
    got = run(case, mask_kind=1, tree_parents=parents)
    want = dense_reference(case, mask_kind=1, tree_parents=parents)
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-13)
    assert np.abs(got - run(case)).max() > 1e-3      # a real tree differs from the chain


def test_row_selection_matches_full_result():
    case = ti.make_attn_case(small_shape(), 29)
    full = run(case)
    sel = np.array([[0, 0, 0], [2, 2, 3], [1, 1, 2]], np.int32)
    got = run(case, row_sel=sel)
    for r, (b, i, h) in enumerate(sel):
        assert np.array_equal(got[r], full[b, i, h])


def test_rejects_branch_shorter_than_query_rows():
    shp = small_shape(branch_lens=(19, 2, 40))       # 2 < gamma + 1 = 3
    case = ti.make_attn_case(replace(shp, branch_lens=(19, 3, 40)), 1)
    case.branch_lens[1] = 2
    with pytest.raises(ValueError):
        run(case)


def test_kv_byte_accounting_matches_the_paper():
    """Appendix A.1: 0.25 GB of KV per branch at 1024 tokens for the 32B shape."""
    kv = dict(line.split() for line in (GOLDEN / "kv_bytes_32b.txt").read_text().splitlines()
              if line and not line.startswith("#"))
    shp = ti.CONFIGS["32b"]
    assert shp.n_layers == int(kv["layers"]) and shp.n_kv_heads == int(kv["kv_heads"])
    one = replace(shp, n_branches=1, prefix_len=0, private_len=int(kv["tokens"]))
    total = one.unique_kv_bytes() * shp.n_layers
    assert total == float(kv["gigabytes"]) * 2**30
    # unique K+V bytes of the three shape configs (prefix counted once)
    assert ti.CONFIGS["tiny"].unique_kv_bytes() == 1310720
    assert ti.CONFIGS["3b"].unique_kv_bytes() == 17301504
    assert ti.CONFIGS["32b"].unique_kv_bytes() == 270532608


# ---- several prefix groups per call (multi-request setting of the paper's appendix) ----
def _group_case(seed=4, **kw):
    args = dict(n_q_heads=4, n_kv_heads=2, gamma=2, group_sizes=(2, 1, 3), group_prefix_lens=(32, 0, 48),
                branch_lens=(19, 3, 40, 7, 33, 16), seed=seed, extra_pages=3)
    args.update(kw)
    return ti.make_group_case(**args)


def _run_groups(c):
    return oracle.verify_attn_groups(c.q, c.k_pages, c.v_pages, c.block_table, c.group_sizes, c.group_prefix_lens,
                                     c.branch_lens, c.gamma)


def test_groups_match_dense_brute_force_per_branch():
    """Every branch against the dense reference run on that branch alone with ITS group's prefix length
    (explicit mask matrix, dense softmax: code that knows nothing about groups)."""
    c = _group_case()
    ti.poison_unused_slots_groups(c)
    got = _run_groups(c)
    assert np.isfinite(got).all()
    group = c.group_of_branch()
    for b in range(c.n_branches):
        one = ti.AttnCase(shape=ti.AttnShape("one", n_q_heads=4, n_kv_heads=2, prefix_len=int(c.group_prefix_lens[group[b]]),
                                             n_branches=1, gamma=2, branch_lens=(int(c.branch_lens[b]),)),
                          q=c.q[b:b + 1], k_pages=c.k_pages, v_pages=c.v_pages, block_table=c.block_table[b:b + 1],
                          branch_lens=c.branch_lens[b:b + 1], prefix_len=int(c.group_prefix_lens[group[b]]),
                          num_pages=c.num_pages, max_blocks=c.max_blocks)
        np.testing.assert_allclose(got[b:b + 1], dense_reference(one), rtol=1e-11, atol=1e-13)


def test_one_group_is_the_single_question_call_bit_for_bit():
    case = ti.make_attn_case(small_shape(), 6)
    want = run(case)
    got = oracle.verify_attn_groups(case.q, case.k_pages, case.v_pages, case.block_table, [3], [case.prefix_len],
                                    case.branch_lens, case.shape.gamma)
    assert np.array_equal(got, want)


def test_groups_do_not_interact():
    """Overwriting the prefix keys and values of group 0 changes the rows of group 0 and leaves every other
    group's rows bit-identical; the block table really shares the prefix pages inside a group only."""
    c = _group_case()
    base = _run_groups(c)
    n_pre0 = int(c.group_prefix_lens[0]) // 16
    shared = c.block_table[0, :n_pre0]
    assert np.array_equal(c.block_table[1, :n_pre0], shared)                       # shared inside group 0
    assert not np.isin(c.block_table[2:], shared).any()                            # and nowhere else
    c.k_pages[shared] = ti.f32_to_bf16_bits(np.full(c.k_pages[shared].shape, 0.5, np.float32))
    c.v_pages[shared] = ti.f32_to_bf16_bits(np.full(c.v_pages[shared].shape, -2.0, np.float32))
    moved = _run_groups(c)
    assert np.array_equal(moved[2:], base[2:])
    assert np.abs(moved[:2] - base[:2]).max() > 1e-3
