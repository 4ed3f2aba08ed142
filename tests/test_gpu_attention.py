"""Parity of the CUDA attention path against the CPU oracle, through the C-ABI.
Tolerance (north-star): |gpu - oracle| <= 1e-2 + 1e-2 |oracle| per element for bf16 inputs with
fp32 accumulation; because that band is loose on N(0,1) data, every case is also gated on the
relative RMS error and there are sentinel / peaky-softmax cases whose errors would be O(1)."""
from dataclasses import replace

import numpy as np
import pytest

import oracle
import paper_2505_19634_b200 as tts
import tts_inputs as ti
from gpu_harness import ATTN_IMPLS, IMPL_NAMES, assert_attn_close, attn_errors, make_ctx, run_attn

pytestmark = pytest.mark.gpu

impl_param = pytest.mark.parametrize("impl", ATTN_IMPLS, ids=lambda i: IMPL_NAMES[i])


def oracle_out(case, **kw):
    return oracle.verify_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.prefix_len,
                              case.branch_lens, case.shape.gamma, **kw)


def bf16_round(x):
    return ti.bf16_bits_to_f32(ti.f32_to_bf16_bits(x.astype(np.float32))).astype(np.float64)


@impl_param
def test_tiny_config(impl):
    case = ti.make_attn_case(ti.CONFIGS["tiny"], 0x5EED)
    want = oracle_out(case)
    got = run_attn(case, impl)
    assert_attn_close(got, want, what="tiny")
    got32 = run_attn(case, impl, out_dtype=tts.OUT_FP32)
    assert attn_errors(got32, want)[1] < 4e-3          # only the bf16 rounding of P (tensor path) remains
    # bf16 output = round-to-nearest-even of the fp32 result
    assert np.array_equal(got, bf16_round(got32))


@impl_param
def test_3b_config(impl):
    case = ti.make_attn_case(ti.CONFIGS["3b"], 0x5EED + 1)
    ti.poison_unused_slots(case)
    assert_attn_close(run_attn(case, impl), oracle_out(case), what="3b")


SMALL = ti.AttnShape("small", n_q_heads=8, n_kv_heads=2, prefix_len=48, n_branches=3, gamma=2,
                     branch_lens=(19, 3, 140), permute_pages=True, extra_pages=5)

EDGE_SHAPES = {
    "ragged": SMALL,
    "no_prefix": replace(SMALL, prefix_len=0),
    "gamma0": replace(SMALL, gamma=0, branch_lens=(1, 16, 17)),
    "min_len": replace(SMALL, gamma=3, branch_lens=(4, 4, 4)),
    "one_branch": replace(SMALL, n_branches=1, branch_lens=(300,), gamma=4),
    "mha": replace(SMALL, n_q_heads=4, n_kv_heads=4),
    "group8_gamma5": replace(SMALL, n_q_heads=16, n_kv_heads=2, gamma=5, branch_lens=(6, 130, 257)),
    "page_multiple": replace(SMALL, branch_lens=(16, 128, 256), prefix_len=128),
    "long_prefix_short_private": replace(SMALL, prefix_len=640, branch_lens=(3, 5, 9)),
    "many_branches": replace(SMALL, n_branches=33, gamma=1, branch_lens=tuple(2 + 7 * i for i in range(33))),
    "tile_straddle": replace(SMALL, gamma=5, branch_lens=(130, 131, 258)),   # draft rows cross a 128-token tile edge
}


@impl_param
@pytest.mark.parametrize("name", list(EDGE_SHAPES))
def test_edge_shapes(impl, name):
    case = ti.make_attn_case(EDGE_SHAPES[name], 77)
    ti.poison_unused_slots(case)               # NaN wherever no query may look
    assert_attn_close(run_attn(case, impl), oracle_out(case), what=name)


@impl_param
def test_900_short_branches(impl):
    """Many short branches: every (branch, KV head) segment is a single tile, so a thread block of the
    token-major kernel works through more pieces than its plan record holds inline."""
    n = 900
    shp = replace(SMALL, n_branches=n, gamma=2, prefix_len=16, branch_lens=tuple(3 + (7 * i) % 23 for i in range(n)))
    case = ti.make_attn_case(shp, 11)
    assert_attn_close(run_attn(case, impl), oracle_out(case), what="900 branches")


def test_explicit_plan_is_reused_and_dropped():
    """tts_attn_plan once, then several layers (different K/V/Q, same table and lengths): same results as
    calls that plan for themselves, one launch fewer per call; a call with other arguments still works."""
    import torch
    from gpu_harness import dev, dev_bf16
    shp = replace(SMALL, n_q_heads=16, n_kv_heads=2, n_branches=6, gamma=3, branch_lens=(700, 4, 131, 1290, 257, 64))
    layers = [ti.make_attn_case(shp, 23, layer=l) for l in range(3)]
    ctx = make_ctx(layers[0], tts.ATTN_TCGEN05_TOKEN_MAJOR, debug=True)
    bt, bl = dev(layers[0].block_table), dev(layers[0].branch_lens)
    dev_in = [(dev_bf16(c.q), dev_bf16(c.k_pages), dev_bf16(c.v_pages)) for c in layers]

    def run_layers():
        nonlocal bl
        outs = []
        for q, k, v in dev_in:
            out = torch.full(q.shape, float("nan"), device="cuda", dtype=torch.bfloat16)
            ctx.tts_verify_attn(q, k, v, bt, shp.prefix_len, bl, shp.n_branches, shp.gamma, tts.MASK_CAUSAL, out)
            outs.append(out)
        torch.cuda.synchronize()
        return [o.float().cpu().numpy().astype(np.float64) for o in outs]

    n0 = ctx.tts_launch_count()
    unplanned = run_layers()
    n1 = ctx.tts_launch_count()
    ctx.tts_attn_plan(bt, shp.prefix_len, bl, shp.n_branches, shp.gamma + 1)
    n2 = ctx.tts_launch_count()
    planned = run_layers()
    n3 = ctx.tts_launch_count()
    assert n1 - n0 == 3 * 3 and n2 - n1 == 1 and n3 - n2 == 3 * 2
    for c, a, b in zip(layers, unplanned, planned):
        assert np.array_equal(a, b)
        assert_attn_close(b, oracle_out(c), what="planned layer")
    # other arguments (a copy of the lengths at another address): the kept plan does not apply, every call
    # plans for itself again and the kept plan is dropped
    bl_kept, bl = bl, bl.clone()
    n4 = ctx.tts_launch_count()
    again = run_layers()
    assert ctx.tts_launch_count() - n4 == 3 * 3
    bl = bl_kept
    run_layers()
    assert ctx.tts_launch_count() - n4 == 2 * 3 * 3
    for a, b in zip(again, planned):
        assert np.array_equal(a, b)
    assert ctx.tts_last_status() == 0
    ctx.close()


@impl_param
def test_sentinel_in_masked_positions(impl):
    """Enormous K/V in every position a row must not see: one leaked key changes out by O(1)."""
    shp = replace(SMALL, gamma=3, branch_lens=(19, 4, 140))
    case = ti.make_attn_case(shp, 5)
    clean = oracle_out(case)
    big = ti.f32_to_bf16_bits(np.array([3.0e4], np.float32))[0]
    for b in range(shp.n_branches):
        L = int(case.branch_lens[b])
        page, slot = ti.token_slot(case, b, case.prefix_len + L - 1)     # visible to the last row only
        case.k_pages[page, :, slot, :] = big
        case.v_pages[page, :, slot, :] = big
    ti.poison_unused_slots(case, bits=int(big))
    want = oracle_out(case)
    assert np.array_equal(want[:, :3], clean[:, :3])
    got = run_attn(case, impl)
    assert_attn_close(got[:, :3], want[:, :3], what="rows that must not see the sentinel")


@impl_param
def test_peaky_softmax(impl):
    """Queries scaled by 8: the softmax concentrates on a few keys and masking/ordering errors show."""
    case = ti.make_attn_case(replace(SMALL, branch_lens=(200, 77, 140)), 9, q_scale=8.0)
    want = oracle_out(case)
    got = run_attn(case, impl)
    assert_attn_close(got, want, rms_gate=8e-3, what="peaky")


@impl_param
def test_rescale_path_with_growing_scores(impl):
    """Keys whose scores grow along the sequence force the running max to move in every tile."""
    shp = replace(SMALL, n_branches=2, branch_lens=(700, 390), prefix_len=256, gamma=3)
    case = ti.make_attn_case(shp, 21)
    kf = ti.bf16_bits_to_f32(case.k_pages)
    qf = ti.bf16_bits_to_f32(case.q)
    qf[..., 0] = 4.0
    case.q = ti.f32_to_bf16_bits(qf)
    for b in range(2):
        total = case.prefix_len + int(case.branch_lens[b])
        for t in range(total):
            page, slot = ti.token_slot(case, b, t)
            kf[page, :, slot, 0] = 0.08 * t          # score contribution 4*0.08*t/sqrt(128) ~ 0.028 t
    case.k_pages = ti.f32_to_bf16_bits(kf)
    assert_attn_close(run_attn(case, impl), oracle_out(case), rms_gate=8e-3, what="growing scores")


@impl_param
def test_page_permutation_invariance(impl):
    shp = replace(SMALL, permute_pages=False, extra_pages=0)
    a = ti.make_attn_case(shp, 11)
    perm = np.random.default_rng(0).permutation(a.num_pages)
    inv = np.argsort(perm)
    b = ti.make_attn_case(shp, 11)
    b.k_pages = np.ascontiguousarray(a.k_pages[perm]); b.v_pages = np.ascontiguousarray(a.v_pages[perm])
    b.block_table = np.where(a.block_table >= 0, inv[np.maximum(a.block_table, 0)], -1).astype(np.int32)
    assert np.array_equal(run_attn(a, impl), run_attn(b, impl))


@impl_param
def test_tree_mask(impl):
    shp = replace(SMALL, gamma=11, branch_lens=(19, 12, 140))
    case = ti.make_attn_case(shp, 31)
    parents = ti.make_tree_parents(3, 12, 4, seed=8)
    want = oracle_out(case, mask_kind=1, tree_parents=parents)
    got = run_attn(case, impl, tree_parents=parents)
    assert_attn_close(got, want, what="tree")
    chain = np.tile(np.arange(-1, 11, dtype=np.int32), (3, 1))
    assert np.array_equal(run_attn(case, impl, tree_parents=chain), run_attn(case, impl))


@impl_param
def test_sweep_points(impl):
    """A few points of the branch/length sweep at reduced lengths (full shapes: Hq 40 / Hkv 8)."""
    for n, g, seed in ((1, 1, 1), (4, 5, 2), (16, 3, 3)):
        shp = ti.sweep_shape(n, g, seed, lo=40, hi=600)
        case = ti.make_attn_case(shp, seed)
        ti.poison_unused_slots(case)
        assert_attn_close(run_attn(case, impl), oracle_out(case), what=shp.name)


def test_context_reuse_and_launch_count():
    case = ti.make_attn_case(SMALL, 3)
    ctx = make_ctx(case, max_rows=6, max_branches=8)
    a = run_attn(case, ctx=ctx)
    n1 = ctx.tts_launch_count()
    b = run_attn(case, ctx=ctx)
    assert np.array_equal(a, b)
    assert n1 >= 2 and ctx.tts_launch_count() == 2 * n1
    ctx.close()


def test_argument_errors_are_status_codes():
    import torch
    case = ti.make_attn_case(SMALL, 3)
    ctx = make_ctx(case)
    z = torch.zeros(64, device="cuda", dtype=torch.int32)
    for kw, want in ((dict(prefix_len=8), -1), (dict(n_branches=0), -1), (dict(n_branches=99), -1),
                     (dict(gamma=-1), -1), (dict(gamma=40), -1), (dict(mask_kind=1), -2), (dict(mask_kind=7), -2)):
        args = dict(prefix_len=48, n_branches=3, gamma=2, mask_kind=0)
        args.update(kw)
        with pytest.raises(tts.TtsError) as ei:
            ctx.tts_verify_attn(z, z, z, z, args["prefix_len"], z, args["n_branches"], args["gamma"],
                                args["mask_kind"], z)
        assert ei.value.status == want, kw
    with pytest.raises(tts.TtsError):
        ctx.tts_verify_attn(None, z, z, z, 48, z, 3, 2, 0, z)
    with pytest.raises(tts.TtsError):                   # misaligned q
        ctx.tts_verify_attn(z.data_ptr() + 4, z, z, z, 48, z, 3, 2, 0, z)
    ctx.close()


def test_debug_bounds_reports_bad_page_id_without_faulting():
    case = ti.make_attn_case(SMALL, 3)
    case.block_table[1, 3] = case.num_pages + 1000        # out-of-range page of branch 1
    ctx = make_ctx(case, impl=tts.ATTN_SIMT, debug=True)
    run_attn(case, ctx=ctx, check_status=False)
    assert ctx.tts_last_status() == -4
    assert ctx.tts_last_status() == 0                     # reading clears it
    ctx.close()


def test_a_wait_that_runs_out_is_reported_and_leaves_the_context_usable():
    """The give-up path of the bounded device-side waits: a probe kernel waits 1 ms for a signal nobody
    sends; the status word then says timeout (-5), reading clears it, and attention calls on the same
    context still give the right result."""
    case = ti.make_attn_case(SMALL, 3)
    want = oracle_out(case)
    ctx = make_ctx(case, impl=tts.ATTN_TCGEN05_TOKEN_MAJOR, debug=True)
    assert_attn_close(run_attn(case, ctx=ctx), want, what="before")
    ctx.tts_debug_wait_timeout(1_000_000)
    assert ctx.tts_last_status() == -5
    assert ctx.tts_last_status() == 0
    assert_attn_close(run_attn(case, ctx=ctx), want, what="after a timed-out wait")
    for bad in (0, 999, 2_000_000_000):
        with pytest.raises(tts.TtsError):
            ctx.tts_debug_wait_timeout(bad)
    ctx.close()


@impl_param
def test_debug_bounds_reports_a_block_index_past_the_table_row(impl):
    """branch_lens lives on the device, so the host cannot see a branch that claims more tokens than its
    block-table row holds.  With the debug checks on, the kernels notice the block index, read page 0 in
    its place (no out-of-range access: the last branch's row ends the table) and report -4."""
    case = ti.make_attn_case(replace(SMALL, branch_lens=(19, 3, 144)), 3)       # 144 = 9 full pages: the longest row is full
    assert case.prefix_len + 144 == 16 * case.max_blocks
    case.branch_lens[2] += 16                                                   # one page more than the row has
    ctx = make_ctx(case, impl=impl, debug=True)
    run_attn(case, ctx=ctx, check_status=False)
    assert ctx.tts_last_status() == -4
    assert ctx.tts_last_status() == 0
    ctx.close()


def _check_all_rows(case, impl, what, tree_parents=None, rms_gate=5e-3, out_dtype=tts.OUT_BF16, **ctx_kw):
    """Every output row against the oracle, in the launch configuration the benchmark times (no debug checks)."""
    kw = dict(mask_kind=1, tree_parents=tree_parents) if tree_parents is not None else {}
    want = oracle_out(case, **kw)
    ctx = make_ctx(case, impl, out_dtype=out_dtype, debug=False, **ctx_kw)
    got = run_attn(case, out_dtype=out_dtype, ctx=ctx, tree_parents=tree_parents)
    ctx.close()
    assert_attn_close(got, want, rms_gate=rms_gate, what=what)
    return got


def test_32b_layer_full_size_all_rows():
    """One layer of the benchmark's workload at full size (16 x 4096 private + 512 prefix tokens, 258 MiB of
    K/V), automatic kernel choice, no debug checks: all 2560 output rows against the oracle, so every
    (branch, KV head) group and every piece boundary of the schedule is looked at."""
    case = ti.make_attn_case(replace(ti.CONFIGS["32b"], n_layers=1), 0x5EED + 2)
    _check_all_rows(case, tts.ATTN_AUTO, "32b layer")


@pytest.mark.parametrize("n,gamma", [(64, 1), (7, 5), (32, 3), (16, 5), (1, 3)])
def test_sweep_points_full_lengths_all_rows(n, gamma):
    """Points of the branch/length sweep at full lengths (ragged 1024..8192 private tokens, prefix
    256..1024, random page permutation, NaN in every slot no query may read): all rows."""
    shp = ti.sweep_shape(n, gamma, seed=100 + n)
    case = ti.make_attn_case(shp, 100 + n)
    ti.poison_unused_slots(case)
    _check_all_rows(case, tts.ATTN_AUTO, shp.name)


def test_tree_config_60_node_trees_full_size():
    """The tree-verification workload at full size: 32B layer shape, 8 branches, 60-node draft trees
    (random parents, depth <= 6), context 8192 of which 512 shared prefix, random page permutation:
    60 x 5 = 300 stacked rows per (branch, KV head), i.e. three 128-row blocks of the row-major kernel and
    the general merge kernel.  All rows against the oracle's ancestor mask."""
    shp = ti.AttnShape("tree", n_q_heads=40, n_kv_heads=8, prefix_len=512, n_branches=8, gamma=59,
                       private_len=8192 - 512)
    case = ti.make_attn_case(shp, 0x5EED + 5)
    ti.poison_unused_slots(case)
    parents = ti.make_tree_parents(8, 60, 6, seed=0x5EED + 5)
    _check_all_rows(case, tts.ATTN_AUTO, "tree config", tree_parents=parents)


@pytest.mark.parametrize("name,gamma,lens", [("rows_104", 12, (300, 45, 700, 13)), ("rows_160", 19, (300, 45, 700, 20)),
                                             ("rows_512", 63, (300, 64, 700, 129))])
def test_causal_chains_with_many_rows_per_kv_head(name, gamma, lens):
    """Causal chains whose stacked rows per KV head exceed one 128-row block (G = 8): 104 rows (one block,
    not replicated), 160 (two blocks), 512 (four blocks: the most a call can carry)."""
    shp = ti.AttnShape(name, n_q_heads=16, n_kv_heads=2, prefix_len=272, n_branches=4, gamma=gamma, branch_lens=lens,
                       extra_pages=3)
    case = ti.make_attn_case(shp, 61)
    ti.poison_unused_slots(case)
    for impl in (tts.ATTN_AUTO, tts.ATTN_TCGEN05_ROW_MAJOR, tts.ATTN_SIMT):
        _check_all_rows(case, impl, f"{name} impl {IMPL_NAMES[impl]}")


@impl_param
def test_split_invariance(impl):
    """The same ragged problem with the main kernel's grid capped at 1, 7, 37 CTAs and uncapped: the KV
    tokens are cut into different pieces each time, every result must lie inside the oracle's band and the
    results must agree with one another to 2e-3 relative RMS (compared in fp32 output: two bf16 roundings
    of nearly equal values differ by a whole bf16 step, 2^-9 relative, in a good part of the elements)."""
    shp = replace(SMALL, n_q_heads=16, n_kv_heads=2, n_branches=5, gamma=3, prefix_len=400 // 16 * 16,
                  branch_lens=(700, 4, 131, 1290, 257))
    case = ti.make_attn_case(shp, 17)
    ti.poison_unused_slots(case)
    want = oracle_out(case)
    outs = []
    for cap in (1, 7, 37, 0):
        _check_all_rows(case, impl, f"cap {cap}", max_ctas=cap)
        outs.append(_check_all_rows(case, impl, f"cap {cap} fp32", out_dtype=tts.OUT_FP32, max_ctas=cap))
    ref_rms = np.sqrt((want ** 2).mean())
    for o in outs[1:]:
        assert np.sqrt(((o - outs[0]) ** 2).mean()) / ref_rms <= 2e-3
