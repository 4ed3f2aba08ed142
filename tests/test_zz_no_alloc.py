"""The no-allocation attention entry point against the regular one (collected last on purpose: a run
that stops at the first failure has then already run every other test).

tts_verify_attn_noalloc is meant for hosts that cannot allocate device memory at call time, so it
keeps its partial results in a fixed array inside the library.  That array survives between calls
and is shared by all of them; the test therefore makes two calls in a row with DIFFERENT problems
and checks each against tts_verify_attn on the same inputs, and against the CPU oracle, within the
tolerance of the other attention tests."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import paper_2505_19634_b200 as tts
import tts_inputs as ti
from gpu_harness import assert_attn_close, dev, dev_bf16, run_attn

pytestmark = pytest.mark.gpu


def run_noalloc(case):
    s = case.shape
    q, k, v = dev_bf16(case.q), dev_bf16(case.k_pages), dev_bf16(case.v_pages)
    bt, bl = dev(case.block_table), dev(case.branch_lens)
    out = torch.full(q.shape, float("nan"), device="cuda", dtype=torch.bfloat16)
    tts.tts_verify_attn_noalloc(q, k, v, bt, case.max_blocks, case.prefix_len, bl, s.n_branches, s.gamma,
                                s.n_q_heads, s.n_kv_heads, out, torch.cuda.current_stream())
    torch.cuda.synchronize()
    return out.float().cpu().numpy().astype(np.float64)


def test_two_calls_in_a_row_match_the_regular_entry_point():
    first = ti.make_attn_case(ti.CONFIGS["tiny"], 0x5EED)
    second = ti.make_attn_case(ti.AttnShape("ragged", n_q_heads=8, n_kv_heads=2, prefix_len=48, n_branches=3,
                                            gamma=2, branch_lens=(19, 3, 140), extra_pages=5), 77)
    ti.poison_unused_slots(second)
    for case in (first, second):
        want = run_attn(case, tts.ATTN_SIMT)
        got = run_noalloc(case)
        assert_attn_close(got, want, what=case.shape.name)
        assert_attn_close(got, oracle.verify_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.prefix_len,
                                                  case.branch_lens, case.shape.gamma), what=case.shape.name + " vs oracle")


def test_32b_layer_fits_and_larger_problems_are_refused():
    shp = replace(ti.CONFIGS["32b"], private_len=300, prefix_len=64)       # the 32B layer's rows, short lengths
    case = ti.make_attn_case(shp, 5)
    assert_attn_close(run_noalloc(case), run_attn(case, tts.ATTN_SIMT), what="32b rows")
    z = torch.zeros(64, device="cuda", dtype=torch.int32)
    with pytest.raises(tts.TtsError) as ei:                                 # 64 branches x 40 heads x 6 rows
        tts.tts_verify_attn_noalloc(z, z, z, z, 8, 16, z, 64, 5, 40, 8, z)
    assert ei.value.status == -6
