"""KV-cache bookkeeping on the GPU (tts_kv_append, tts_kv_rollback) against the oracle: byte-exact pools
and lengths, page edges, and the error statuses of the bounds checks."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import paper_2505_19634_b200 as tts
import tts_inputs as ti
from gpu_harness import dev, dev_bf16, make_ctx

pytestmark = pytest.mark.gpu

SHAPE = ti.AttnShape("kv", n_q_heads=8, n_kv_heads=2, prefix_len=32, n_branches=4, gamma=3,
                     branch_lens=(4, 17, 33, 50), permute_pages=True, extra_pages=3)


def bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("lens,rows", [((4, 17, 33, 50), 4), ((4, 18, 32, 49), 4), ((1, 16, 31, 64), 1), ((6, 22, 38, 70), 6)])
def test_append_matches_oracle_bytes(lens, rows):
    case = ti.make_attn_case(replace(SHAPE, branch_lens=lens, gamma=max(rows - 1, 0)), 11)
    rng = np.random.default_rng(rows)
    k_new = rng.integers(0, 1 << 15, size=(4, rows, 2, 128), dtype=np.uint16)
    v_new = rng.integers(0, 1 << 15, size=(4, rows, 2, 128), dtype=np.uint16)
    want_k, want_v = oracle.kv_append(case.k_pages, case.v_pages, k_new, v_new, case.block_table, case.prefix_len, case.branch_lens)
    ctx = make_ctx(case, max_rows=8)
    k, v = dev_bf16(case.k_pages), dev_bf16(case.v_pages)
    ctx.tts_kv_append(dev_bf16(k_new), dev_bf16(v_new), k, v, dev(case.block_table), case.prefix_len, dev(case.branch_lens), 4, rows)
    torch.cuda.synchronize()
    assert ctx.tts_last_status() == 0
    assert np.array_equal(bits(k), want_k) and np.array_equal(bits(v), want_v)
    ctx.close()


def test_append_then_attention_equals_attention_of_the_whole_cache():
    case = ti.make_attn_case(SHAPE, 3)
    rows = SHAPE.gamma + 1
    k_new = np.zeros((4, rows, 2, 128), np.uint16); v_new = np.zeros_like(k_new)
    wiped_k, wiped_v = case.k_pages.copy(), case.v_pages.copy()
    for b in range(4):
        for i in range(rows):
            page, slot = ti.token_slot(case, b, case.prefix_len + int(case.branch_lens[b]) - rows + i)
            k_new[b, i] = case.k_pages[page, :, slot, :]; v_new[b, i] = case.v_pages[page, :, slot, :]
            wiped_k[page, :, slot, :] = 0x7FC0; wiped_v[page, :, slot, :] = 0x7FC0
    ctx = make_ctx(case)
    k, v = dev_bf16(wiped_k), dev_bf16(wiped_v)
    bt, bl, q = dev(case.block_table), dev(case.branch_lens), dev_bf16(case.q)
    ctx.tts_kv_append(dev_bf16(k_new), dev_bf16(v_new), k, v, bt, case.prefix_len, bl, 4, rows)
    out = torch.empty_like(q)
    ctx.tts_verify_attn(q, k, v, bt, case.prefix_len, bl, 4, SHAPE.gamma, tts.MASK_CAUSAL, out)
    k0, v0 = dev_bf16(case.k_pages), dev_bf16(case.v_pages)
    out0 = torch.empty_like(q)
    ctx.tts_verify_attn(q, k0, v0, bt, case.prefix_len, bl, 4, SHAPE.gamma, tts.MASK_CAUSAL, out0)
    torch.cuda.synchronize()
    assert ctx.tts_last_status() == 0
    assert torch.equal(out.view(torch.int16), out0.view(torch.int16))
    ctx.close()


def test_append_bounds_are_reported_not_written():
    case = ti.make_attn_case(SHAPE, 4)
    rows = 4
    k_new = np.full((4, rows, 2, 128), 0x1234, np.uint16)
    ctx = make_ctx(case)
    # a branch shorter than the rows appended: nothing of that branch is written
    k, v = dev_bf16(case.k_pages), dev_bf16(case.v_pages)
    lens = case.branch_lens.copy(); lens[0] = 3
    ctx.tts_kv_append(dev_bf16(k_new), dev_bf16(k_new), k, v, dev(case.block_table), case.prefix_len, dev(lens), 4, rows)
    torch.cuda.synchronize()
    assert ctx.tts_last_status() == -4                      # TTS_ERR_DEVICE_BOUNDS
    lens_ok = lens.copy(); lens_ok[0] = case.branch_lens[0]
    want_k, _ = oracle.kv_append(case.k_pages, case.v_pages, k_new, k_new, case.block_table, case.prefix_len, lens_ok)
    got = bits(k)
    page0 = set(int(ti.token_slot(case, 0, case.prefix_len + i)[0]) for i in range(int(case.branch_lens[0])))
    other = [pg for pg in range(case.num_pages) if pg not in page0]
    assert np.array_equal(got[other], want_k[other])        # the other branches were appended
    assert np.array_equal(got[list(page0)], case.k_pages[list(page0)])   # branch 0 untouched
    # a page index outside the pool
    bt = case.block_table.copy(); bt[2, (case.prefix_len + int(case.branch_lens[2]) - 1) // 16] = case.num_pages + 7
    k, v = dev_bf16(case.k_pages), dev_bf16(case.v_pages)
    ctx.tts_kv_append(dev_bf16(k_new), dev_bf16(k_new), k, v, dev(bt), case.prefix_len, dev(case.branch_lens), 4, rows)
    torch.cuda.synchronize()
    assert ctx.tts_last_status() == -4
    ctx.close()


def test_rollback_matches_oracle():
    case = ti.make_attn_case(SHAPE, 5)
    ctx = make_ctx(case)
    gamma = 3
    acc = np.array([0, 3, 1, 2], np.int32)
    lens = dev(case.branch_lens.copy())
    ctx.tts_kv_rollback(lens, dev(acc), 4, gamma)
    torch.cuda.synchronize()
    assert ctx.tts_last_status() == 0
    assert np.array_equal(lens.cpu().numpy(), oracle.kv_rollback(case.branch_lens, acc, gamma))
    bad = np.array([0, 4, 1, -1], np.int32)
    lens = dev(case.branch_lens.copy())
    ctx.tts_kv_rollback(lens, dev(bad), 4, gamma)
    torch.cuda.synchronize()
    assert ctx.tts_last_status() == -4
    assert np.array_equal(lens.cpu().numpy(), case.branch_lens - np.array([3, 0, 2, 0]))
    ctx.close()
