"""Pins of the oracle's KV-cache bookkeeping (append before the verify step, rollback after the accept
test) against facts that do not come from it: reading the appended tokens back through an independent
page-table walk, the untouched remainder of the pools, and the attention oracle itself (a cache built by
appending the newest rows must give the attention of the cache that was generated whole)."""
from dataclasses import replace

import numpy as np
import pytest

import oracle
import tts_inputs as ti

SHAPE = ti.AttnShape("kv", n_q_heads=8, n_kv_heads=2, prefix_len=32, n_branches=4, gamma=3,
                     branch_lens=(4, 17, 33, 50), permute_pages=True, extra_pages=3)


def newest_rows(case, rows):
    """[N][rows][Hkv][D] bits of the last `rows` private tokens of every branch, read slot by slot."""
    s = case.shape
    k = np.zeros((s.n_branches, rows, s.n_kv_heads, 128), np.uint16)
    v = np.zeros_like(k)
    for b in range(s.n_branches):
        for i in range(rows):
            page, slot = ti.token_slot(case, b, case.prefix_len + int(case.branch_lens[b]) - rows + i)
            k[b, i] = case.k_pages[page, :, slot, :]
            v[b, i] = case.v_pages[page, :, slot, :]
    return k, v


def test_append_restores_a_cache_whose_newest_rows_were_wiped():
    case = ti.make_attn_case(SHAPE, 3)
    rows = SHAPE.gamma + 1
    k_new, v_new = newest_rows(case, rows)
    wiped_k, wiped_v = case.k_pages.copy(), case.v_pages.copy()
    for b in range(SHAPE.n_branches):
        for i in range(rows):
            page, slot = ti.token_slot(case, b, case.prefix_len + int(case.branch_lens[b]) - rows + i)
            wiped_k[page, :, slot, :] = 0x7FC0
            wiped_v[page, :, slot, :] = 0x7FC0
    assert not np.array_equal(wiped_k, case.k_pages)
    k2, v2 = oracle.kv_append(wiped_k, wiped_v, k_new, v_new, case.block_table, case.prefix_len, case.branch_lens)
    assert np.array_equal(k2, case.k_pages) and np.array_equal(v2, case.v_pages)      # every other byte untouched
    # and the attention over the rebuilt cache is the attention over the original one
    a = oracle.verify_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.prefix_len, case.branch_lens, SHAPE.gamma)
    b = oracle.verify_attn(case.q, k2, v2, case.block_table, case.prefix_len, case.branch_lens, SHAPE.gamma)
    assert np.array_equal(a, b)


def test_append_writes_exactly_the_causal_tail_of_the_attention():
    """Changing an appended row changes the attention output of the rows that may see it and of no other:
    row i of a branch sees appended rows 0..i (the positions the attention masks causally)."""
    case = ti.make_attn_case(replace(SHAPE, branch_lens=(20, 21, 22, 23)), 5)
    rows = SHAPE.gamma + 1
    k_new, v_new = newest_rows(case, rows)
    base = oracle.verify_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.prefix_len, case.branch_lens, SHAPE.gamma)
    for j in range(rows):
        v_mod = v_new.copy()
        v_mod[1, j] ^= 0x0100                                     # another value for appended row j of branch 1
        k2, v2 = oracle.kv_append(case.k_pages, case.v_pages, k_new, v_mod, case.block_table, case.prefix_len, case.branch_lens)
        out = oracle.verify_attn(case.q, k2, v2, case.block_table, case.prefix_len, case.branch_lens, SHAPE.gamma)
        changed = np.any(out != base, axis=(2, 3))                # [N][R]
        want = np.zeros_like(changed)
        want[1, j:] = True
        assert np.array_equal(changed, want), j


def test_append_across_a_page_edge_and_short_branch():
    case = ti.make_attn_case(replace(SHAPE, branch_lens=(4, 18, 32, 49)), 7)   # tails straddle slots 15 | 0
    rows = 4
    rng = np.random.default_rng(1)
    k_new = rng.integers(0, 1 << 15, size=(4, rows, 2, 128), dtype=np.uint16)
    v_new = rng.integers(0, 1 << 15, size=(4, rows, 2, 128), dtype=np.uint16)
    k2, v2 = oracle.kv_append(case.k_pages, case.v_pages, k_new, v_new, case.block_table, case.prefix_len, case.branch_lens)
    case2 = replace(case, k_pages=k2, v_pages=v2)
    kk, vv = newest_rows(case2, rows)
    assert np.array_equal(kk, k_new) and np.array_equal(vv, v_new)
    changed = np.any(k2 != case.k_pages, axis=(1, 3))             # [page][slot]
    assert changed.sum() <= 4 * rows
    with pytest.raises(ValueError):
        oracle.kv_append(case.k_pages, case.v_pages, k_new, v_new, case.block_table, case.prefix_len, np.array([3, 18, 32, 49]))


def test_rollback_keeps_what_was_accepted():
    lens = np.array([10, 20, 30, 40], np.int32)
    gamma = 3
    assert np.array_equal(oracle.kv_rollback(lens, [3, 3, 3, 3], gamma), lens)             # all accepted: nothing leaves
    assert np.array_equal(oracle.kv_rollback(lens, [0, 0, 0, 0], gamma), lens - gamma)     # none: all drafts leave
    assert np.array_equal(oracle.kv_rollback(lens, [0, 1, 2, 3], gamma), [7, 18, 29, 40])
    # a step nets accepted_len + 1 tokens per branch: the committed token and the accepted drafts stay
    before = lens - (gamma + 1)
    assert np.array_equal(oracle.kv_rollback(lens, [0, 1, 2, 3], gamma) - before, [1, 2, 3, 4])
    with pytest.raises(ValueError):
        oracle.kv_rollback(lens, [0, 4, 0, 0], gamma)
