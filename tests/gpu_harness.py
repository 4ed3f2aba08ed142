"""Helpers for the GPU parity tests: move a seeded case to the device, call the C-ABI through the
Python binding, bring the result back as numpy.  No arithmetic of the method happens here."""
from __future__ import annotations

import numpy as np
import torch

import paper_2505_19634_b200 as tts
import tts_inputs as ti

ATTN_IMPLS = [tts.ATTN_SIMT, tts.ATTN_TCGEN05_TOKEN_MAJOR, tts.ATTN_TCGEN05_ROW_MAJOR]
IMPL_NAMES = {tts.ATTN_SIMT: "simt", tts.ATTN_TCGEN05: "tcgen05", tts.ATTN_AUTO: "auto",
              tts.ATTN_TCGEN05_TOKEN_MAJOR: "tcgen05_token_major", tts.ATTN_TCGEN05_ROW_MAJOR: "tcgen05_row_major"}


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def make_ctx(case: ti.AttnCase, impl=tts.ATTN_AUTO, out_dtype=tts.OUT_BF16, debug=False,
             max_rows=None, max_branches=None, max_ctas=0) -> tts.TtsContext:
    s = case.shape
    return tts.TtsContext(s.n_q_heads, s.n_kv_heads, max_branches or s.n_branches,
                          max_rows or s.rows_per_branch, case.max_blocks, case.num_pages,
                          out_dtype=out_dtype, attn_impl=impl, debug_bounds=debug, max_ctas=max_ctas)


def run_attn(case: ti.AttnCase, impl=tts.ATTN_AUTO, out_dtype=tts.OUT_BF16, tree_parents=None, debug=True,
             ctx=None, check_status=True) -> np.ndarray:
    """out as float64 numpy [N][R][Hq][D]."""
    s = case.shape
    own = ctx is None
    if own:
        ctx = make_ctx(case, impl, out_dtype, debug)
    q, k, v = dev_bf16(case.q), dev_bf16(case.k_pages), dev_bf16(case.v_pages)
    bt, bl = dev(case.block_table), dev(case.branch_lens)
    out = torch.full(q.shape, float("nan"), device="cuda",
                     dtype=torch.bfloat16 if out_dtype == tts.OUT_BF16 else torch.float32)
    if tree_parents is None:
        ctx.tts_verify_attn(q, k, v, bt, case.prefix_len, bl, s.n_branches, s.gamma, tts.MASK_CAUSAL, out)
    else:
        tp = dev(np.ascontiguousarray(tree_parents, dtype=np.int32))
        ctx.tts_verify_attn_tree(q, k, v, bt, case.prefix_len, bl, tp, s.n_branches, s.rows_per_branch, out)
    torch.cuda.synchronize()
    if check_status:
        st = ctx.tts_last_status()
        assert st == 0, f"device status {st}"
    res = out.float().cpu().numpy().astype(np.float64)
    if own:
        ctx.close()
    return res


def attn_errors(got: np.ndarray, want: np.ndarray):
    """(worst excess over the 1e-2 abs + 1e-2 rel band, relative RMS error, max abs error)."""
    diff = np.abs(got - want)
    band = 1e-2 + 1e-2 * np.abs(want)
    rms = float(np.sqrt((diff ** 2).mean()) / max(np.sqrt((want ** 2).mean()), 1e-30))
    return float((diff - band).max()), rms, float(diff.max())


def assert_attn_close(got, want, rms_gate=5e-3, what=""):
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    excess, rms, mx = attn_errors(got, want)
    assert excess <= 0, f"{what}: element outside 1e-2 abs + 1e-2 rel (max abs err {mx:.3e})"
    assert rms <= rms_gate, f"{what}: relative RMS error {rms:.3e} > {rms_gate}"


def run_accept(case: ti.AcceptCase, ctx=None):
    own = ctx is None
    if own:
        ctx = tts.TtsContext(8, 2, 1, 1, 4, 4)       # tts_accept takes its sizes per call
    p, u = dev(case.p_target), dev(case.uniforms)
    q = dev(case.q_draft) if case.gamma > 0 else None
    t = dev(case.draft_tokens) if case.gamma > 0 else None
    acc = torch.full((case.n_branches,), -7, dtype=torch.int32, device="cuda")
    nxt = torch.full((case.n_branches,), -7, dtype=torch.int32, device="cuda")
    ctx.tts_accept(p, q, t, u, case.n_branches, case.gamma, case.vocab, acc, nxt)
    torch.cuda.synchronize()
    assert ctx.tts_last_status() == 0
    if own:
        ctx.close()
    return acc.cpu().numpy(), nxt.cpu().numpy()
