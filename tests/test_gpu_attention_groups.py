"""Several prefix groups per call (tts_verify_attn_groups) against the oracle, through the C-ABI: ragged
group sizes, a group without prefix, single-branch groups, all three kernels (the token-major kernel serves
all groups in one launch from one plan; the others run group by group)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2505_19634_b200 as tts
import tts_inputs as ti
from gpu_harness import ATTN_IMPLS, IMPL_NAMES, assert_attn_close, dev, dev_bf16

pytestmark = pytest.mark.gpu

impl_param = pytest.mark.parametrize("impl", ATTN_IMPLS + [tts.ATTN_AUTO], ids=lambda i: IMPL_NAMES[i])

CASES = {
    "ragged_groups": dict(n_q_heads=8, n_kv_heads=2, gamma=2, group_sizes=(2, 1, 3), group_prefix_lens=(48, 0, 160),
                          branch_lens=(19, 3, 140, 7, 300, 16), extra_pages=5),
    "one_group": dict(n_q_heads=8, n_kv_heads=2, gamma=2, group_sizes=(3,), group_prefix_lens=(48,),
                      branch_lens=(19, 3, 140)),
    "single_branch_groups": dict(n_q_heads=16, n_kv_heads=2, gamma=3, group_sizes=(1, 1, 1, 1), group_prefix_lens=(16, 272, 0, 128),
                                 branch_lens=(4, 260, 131, 77)),
    "many_groups_32b_heads": dict(n_q_heads=40, n_kv_heads=8, gamma=3, group_sizes=tuple([4] * 16),
                                  group_prefix_lens=tuple(16 * (3 + 5 * (g % 7)) for g in range(16)),
                                  branch_lens=tuple(4 + (37 * i) % 700 for i in range(64))),
    "no_prefix_anywhere": dict(n_q_heads=8, n_kv_heads=2, gamma=1, group_sizes=(2, 2), group_prefix_lens=(0, 0),
                               branch_lens=(2, 129, 40, 256)),
}


def oracle_groups(c):
    return oracle.verify_attn_groups(c.q, c.k_pages, c.v_pages, c.block_table, c.group_sizes, c.group_prefix_lens,
                                     c.branch_lens, c.gamma)


def run_groups(c, impl, ctx=None, planned=False):
    own = ctx is None
    if own:
        ctx = tts.TtsContext(c.n_q_heads, c.n_kv_heads, c.n_branches, c.gamma + 1, c.max_blocks, c.num_pages,
                             attn_impl=impl, debug_bounds=True)
    q, k, v = dev_bf16(c.q), dev_bf16(c.k_pages), dev_bf16(c.v_pages)
    bt, bl = dev(c.block_table), dev(c.branch_lens)
    out = torch.full(q.shape, float("nan"), device="cuda", dtype=torch.bfloat16)
    if planned:
        ctx.tts_attn_plan_groups(bt, c.group_sizes, c.group_prefix_lens, bl, c.n_branches, c.gamma + 1)
    ctx.tts_verify_attn_groups(q, k, v, bt, c.group_sizes, c.group_prefix_lens, bl, c.n_branches, c.gamma, out)
    torch.cuda.synchronize()
    assert ctx.tts_last_status() == 0
    if own:
        ctx.close()
    return out.float().cpu().numpy().astype(np.float64)


@impl_param
@pytest.mark.parametrize("name", list(CASES))
def test_groups_match_oracle(impl, name):
    c = ti.make_group_case(seed=41, **CASES[name])
    ti.poison_unused_slots_groups(c)
    assert_attn_close(run_groups(c, impl), oracle_groups(c), what=name)


def test_one_group_equals_the_single_prefix_call():
    c = ti.make_group_case(seed=42, **CASES["one_group"])
    single = c.as_single_group(0)
    from gpu_harness import run_attn
    for impl in (tts.ATTN_TCGEN05_TOKEN_MAJOR, tts.ATTN_SIMT):
        assert np.array_equal(run_groups(c, impl), run_attn(single, impl))


def test_planned_groups_and_plan_key():
    """tts_attn_plan_groups once, then calls with the same group arrays reuse the plan (two launches per call);
    a call with other prefix lengths plans for itself."""
    c = ti.make_group_case(seed=43, **CASES["ragged_groups"])
    want = oracle_groups(c)
    ctx = tts.TtsContext(c.n_q_heads, c.n_kv_heads, c.n_branches, c.gamma + 1, c.max_blocks, c.num_pages,
                         attn_impl=tts.ATTN_TCGEN05_TOKEN_MAJOR, debug_bounds=True)
    q, k, v = dev_bf16(c.q), dev_bf16(c.k_pages), dev_bf16(c.v_pages)
    bt, bl = dev(c.block_table), dev(c.branch_lens)
    out = torch.full(q.shape, float("nan"), device="cuda", dtype=torch.bfloat16)
    ctx.tts_attn_plan_groups(bt, c.group_sizes, c.group_prefix_lens, bl, c.n_branches, c.gamma + 1)
    n0 = ctx.tts_launch_count()
    for _ in range(2):
        ctx.tts_verify_attn_groups(q, k, v, bt, c.group_sizes, c.group_prefix_lens, bl, c.n_branches, c.gamma, out)
    torch.cuda.synchronize()
    assert ctx.tts_launch_count() - n0 == 4
    assert_attn_close(out.float().cpu().numpy().astype(np.float64), want, what="planned groups")
    # the same pointers with the groups merged differently: the kept plan must not be used
    ctx.tts_attn_plan_groups(bt, c.group_sizes, c.group_prefix_lens, bl, c.n_branches, c.gamma + 1)
    n1 = ctx.tts_launch_count()
    sizes2 = (2, 1, 1, 2)
    pre2 = (48, 0, 160, 160)                          # branches 3..5 share the 160-token prefix either way
    ctx.tts_verify_attn_groups(q, k, v, bt, sizes2, pre2, bl, c.n_branches, c.gamma, out)
    torch.cuda.synchronize()
    assert ctx.tts_launch_count() - n1 == 3
    assert_attn_close(out.float().cpu().numpy().astype(np.float64), want, what="regrouped")
    assert ctx.tts_last_status() == 0
    ctx.close()


def test_group_argument_errors():
    c = ti.make_group_case(seed=44, **CASES["ragged_groups"])
    ctx = tts.TtsContext(c.n_q_heads, c.n_kv_heads, c.n_branches, c.gamma + 1, c.max_blocks, c.num_pages)
    z = torch.zeros(64, device="cuda", dtype=torch.int32)
    for sizes, pre in (((2, 1, 2), (48, 0, 160)),        # sizes do not add up
                       ((2, 0, 4), (48, 0, 160)),        # empty group
                       ((2, 1, 3), (48, 8, 160)),        # prefix not a multiple of the page size
                       ((6,) + (0,) * 64, (0,) * 65)):   # too many groups
        with pytest.raises(tts.TtsError) as ei:
            ctx.tts_verify_attn_groups(z, z, z, z, sizes, pre, z, 6, c.gamma, z)
        assert ei.value.status == -1
    ctx.close()


def test_groups_under_a_capped_grid():
    """The cut of the concatenated tile lists moves with the number of CTAs; the result must not."""
    c = ti.make_group_case(seed=45, **CASES["ragged_groups"])
    ti.poison_unused_slots_groups(c)
    want = oracle_groups(c)
    for cap in (1, 3, 29):
        ctx = tts.TtsContext(c.n_q_heads, c.n_kv_heads, c.n_branches, c.gamma + 1, c.max_blocks, c.num_pages,
                             attn_impl=tts.ATTN_TCGEN05_TOKEN_MAJOR, debug_bounds=True, max_ctas=cap)
        assert_attn_close(run_groups(c, tts.ATTN_TCGEN05_TOKEN_MAJOR, ctx=ctx, planned=True), want, what=f"cap {cap}")
        ctx.close()
