"""The end-to-end entry point tts_verify_step_host (host buffers in, host buffers out: several layers
of attention plus one accept pass) against the CPU oracle, layer by layer."""
import numpy as np
import pytest
import torch

import oracle
import paper_2505_19634_b200 as tts
import tts_inputs as ti
from gpu_harness import assert_attn_close, dev_bf16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["tiny", "ragged"])
def test_step_from_host_buffers(name):
    shape = ti.CONFIGS["tiny"] if name == "tiny" else ti.AttnShape(
        "ragged", n_q_heads=8, n_kv_heads=2, prefix_len=48, n_branches=3, gamma=2, branch_lens=(19, 3, 140),
        extra_pages=5, vocab=132)
    n_layers = 3
    cases = [ti.make_attn_case(shape, 11, layer=l) for l in range(n_layers)]      # one block table, own K/V/Q per layer
    acc = ti.make_accept_case(shape.n_branches, shape.gamma, shape.vocab, 2.0, seed=12, draft_noise=0.6)
    c0 = cases[0]
    k_pools = [dev_bf16(c.k_pages) for c in cases]
    v_pools = [dev_bf16(c.v_pages) for c in cases]
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    q_host = pin(np.stack([c.q for c in cases]).view(np.int16))
    out_host = torch.zeros(q_host.shape, dtype=torch.int16).pin_memory()
    h_al = torch.full((shape.n_branches,), -7, dtype=torch.int32).pin_memory()
    h_nt = torch.full((shape.n_branches,), -7, dtype=torch.int32).pin_memory()
    ctx = tts.TtsContext(shape.n_q_heads, shape.n_kv_heads, shape.n_branches, shape.rows_per_branch, c0.max_blocks,
                         c0.num_pages)
    for _ in range(2):                                        # the second call reuses the staging buffers
        ctx.tts_verify_step_host(n_layers, q_host, k_pools, v_pools, pin(c0.block_table), c0.prefix_len,
                                 pin(c0.branch_lens), shape.n_branches, shape.gamma, pin(acc.p_target),
                                 pin(acc.q_draft), pin(acc.draft_tokens), pin(acc.uniforms), shape.vocab, out_host,
                                 h_al, h_nt)
    assert ctx.tts_last_status() == 0
    got = ti.bf16_bits_to_f32(out_host.numpy().view(np.uint16)).astype(np.float64)
    for l, c in enumerate(cases):
        want = oracle.verify_attn(c.q, c.k_pages, c.v_pages, c.block_table, c.prefix_len, c.branch_lens, shape.gamma)
        assert_attn_close(got[l], want, what=f"{name} layer {l}")
    a_o, n_o, near = oracle.accept(acc.p_target, acc.q_draft, acc.draft_tokens, acc.uniforms)
    ok = near == 0
    assert np.array_equal(h_al.numpy()[ok], a_o[ok]) and np.array_equal(h_nt.numpy()[ok], n_o[ok])
    ctx.close()


def test_step_from_host_buffers_with_bf16_logits():
    """The same end-to-end call with the accept pass fed with bf16 logits instead of fp32 probabilities."""
    shape = ti.CONFIGS["tiny"]
    n_layers = 2
    cases = [ti.make_attn_case(shape, 13, layer=l) for l in range(n_layers)]
    acc = ti.make_accept_logits_case(shape.n_branches, shape.gamma, shape.vocab, 2.0, seed=14, draft_noise=0.6, bf16=True)
    c0 = cases[0]
    k_pools = [dev_bf16(c.k_pages) for c in cases]
    v_pools = [dev_bf16(c.v_pages) for c in cases]
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    q_host = pin(np.stack([c.q for c in cases]).view(np.int16))
    out_host = torch.zeros(q_host.shape, dtype=torch.int16).pin_memory()
    h_al = torch.full((shape.n_branches,), -7, dtype=torch.int32).pin_memory()
    h_nt = torch.full((shape.n_branches,), -7, dtype=torch.int32).pin_memory()
    ctx = tts.TtsContext(shape.n_q_heads, shape.n_kv_heads, shape.n_branches, shape.rows_per_branch, c0.max_blocks,
                         c0.num_pages)
    ctx.tts_verify_step_host_logits(n_layers, q_host, k_pools, v_pools, pin(c0.block_table), c0.prefix_len,
                                    pin(c0.branch_lens), shape.n_branches, shape.gamma,
                                    pin(acc.target_logits.view(np.int16)), pin(acc.draft_logits.view(np.int16)),
                                    tts.LOGITS_BF16, pin(acc.draft_tokens), pin(acc.uniforms), shape.vocab, out_host,
                                    h_al, h_nt)
    assert ctx.tts_last_status() == 0
    got = ti.bf16_bits_to_f32(out_host.numpy().view(np.uint16)).astype(np.float64)
    for l, c in enumerate(cases):
        want = oracle.verify_attn(c.q, c.k_pages, c.v_pages, c.block_table, c.prefix_len, c.branch_lens, shape.gamma)
        assert_attn_close(got[l], want, what=f"layer {l}")
    a_o, n_o, near = oracle.accept_logits(acc.target_logits, acc.draft_logits, acc.draft_tokens, acc.uniforms)
    ok = near == 0
    assert np.array_equal(h_al.numpy()[ok], a_o[ok]) and np.array_equal(h_nt.numpy()[ok], n_o[ok])
    ctx.close()
