"""Seeded synthetic inputs for the speculative-decoding verify step.

This module only *draws* inputs (shapes, random values, page permutations, draft
tokens).  It contains none of the verify step's arithmetic and is the only code
that both the CPU oracle's tests and the CUDA path's tests may share.

Everything is numpy on the host; arrays are returned in the exact byte layout
the C-ABI expects (bf16 carried as uint16 bit patterns).

Workload shapes follow the paper: prompts of a few hundred tokens shared by all
branches (Appendix, prefill discussion), generated lengths 1024..8192 (Section 1,
Figure 1), B in {1..64} (Section 3.3), draft length up to 5 (Appendix,
latency-optimal configurations), KV bytes of the Qwen2.5-32B shape (Appendix A.1).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Optional

import numpy as np

PAGE = 16
HEAD_DIM = 128


# --------------------------------------------------------------------------- #
# bf16 helpers (format conversion only)
# --------------------------------------------------------------------------- #
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream)]))


def _normal_bf16(rng: np.random.Generator, shape, scale: float = 1.0) -> np.ndarray:
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if scale != 1.0:
        x *= np.float32(scale)
    return f32_to_bf16_bits(x)


# --------------------------------------------------------------------------- #
# shapes
# --------------------------------------------------------------------------- #
@dataclass(frozen=True)
class AttnShape:
    """One layer's verify-attention problem."""
    name: str
    n_q_heads: int
    n_kv_heads: int
    prefix_len: int                 # P, multiple of PAGE
    n_branches: int                 # N
    gamma: int                      # draft length; R = gamma + 1 query rows / branch
    private_len: int = 0            # L_b for every branch (if branch_lens is None)
    branch_lens: Optional[tuple] = None   # explicit ragged private lengths
    permute_pages: bool = True
    n_layers: int = 1
    vocab: int = 1024
    logit_sigma: float = 2.0
    head_dim: int = HEAD_DIM
    page_size: int = PAGE
    extra_pages: int = 0            # unused physical pages mixed into the pool

    @property
    def rows_per_branch(self) -> int:
        return self.gamma + 1

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def lens(self) -> np.ndarray:
        if self.branch_lens is not None:
            assert len(self.branch_lens) == self.n_branches
            return np.asarray(self.branch_lens, dtype=np.int32)
        return np.full(self.n_branches, self.private_len, dtype=np.int32)

    def unique_kv_tokens(self) -> int:
        return int(self.prefix_len + self.lens().astype(np.int64).sum())

    def unique_kv_bytes(self) -> int:
        """K+V bytes of every distinct KV token, the shared prefix counted once."""
        return self.unique_kv_tokens() * self.n_kv_heads * self.head_dim * 2 * 2

    def attn_flops(self) -> int:
        """4*D flops per (query row, visible key) pair, ignoring the causal corner."""
        lens = self.lens().astype(np.int64)
        rows = self.rows_per_branch * self.n_q_heads
        return int(4 * self.head_dim * rows * (self.prefix_len * self.n_branches + lens.sum()))


CONFIGS: Dict[str, AttnShape] = {
    # the small case (the oracle finishes it in seconds)
    "tiny": AttnShape("tiny", n_q_heads=8, n_kv_heads=2, prefix_len=256, n_branches=4, gamma=3,
                      private_len=256, permute_pages=False, vocab=1024, logit_sigma=2.0),
    # Qwen2.5-3B-shaped layer
    "3b": AttnShape("3b", n_q_heads=16, n_kv_heads=2, prefix_len=512, n_branches=8, gamma=4,
                    private_len=2048, vocab=151936, logit_sigma=3.0),
    # Qwen2.5-32B-shaped layer, 64 of them per step: the benchmark's workload
    "32b": AttnShape("32b", n_q_heads=40, n_kv_heads=8, prefix_len=512, n_branches=16, gamma=3,
                     private_len=4096, n_layers=64, vocab=152064, logit_sigma=3.0),
}

SWEEP_BRANCHES = (1, 2, 4, 8, 16, 32, 64)
SWEEP_GAMMAS = (1, 3, 5)


def sweep_shape(n_branches: int, gamma: int, seed: int, lo: int = 1024, hi: int = 8192) -> AttnShape:
    """The branch / gamma sweep: 32B layer shape, ragged private lengths U{lo..hi},
    shared prefix 16*U{16..64}, random page permutation."""
    rng = _rng(seed, 911)
    lens = rng.integers(lo, hi + 1, size=n_branches)
    lens = np.maximum(lens, gamma + 1)
    prefix = int(rng.integers(16, 65)) * PAGE
    return AttnShape(f"sweep_N{n_branches}_g{gamma}_s{seed}", n_q_heads=40, n_kv_heads=8,
                     prefix_len=prefix, n_branches=n_branches, gamma=gamma,
                     branch_lens=tuple(int(v) for v in lens), vocab=152064, logit_sigma=3.0)


# --------------------------------------------------------------------------- #
# attention inputs
# --------------------------------------------------------------------------- #
@dataclass
class AttnCase:
    shape: AttnShape
    q: np.ndarray             # uint16 [N][R][Hq][D]           bf16 bits
    k_pages: np.ndarray       # uint16 [num_pages][Hkv][16][D] bf16 bits
    v_pages: np.ndarray       # uint16 [num_pages][Hkv][16][D]
    block_table: np.ndarray   # int32  [N][max_blocks]; unused entries = -1
    branch_lens: np.ndarray   # int32  [N] private KV tokens incl. the R in-flight ones
    prefix_len: int
    num_pages: int
    max_blocks: int
    meta: dict = field(default_factory=dict)


def make_block_table(shape: AttnShape, seed: int):
    """Logical order [prefix | branch 0 | branch 1 | ...] mapped onto a page pool.

    Identity mapping when permute_pages is False, otherwise a seeded random
    permutation of exactly the pages needed (+ extra_pages unused ones).
    Returns (block_table[N][max_blocks], num_pages, max_blocks)."""
    lens = shape.lens()
    n_pre = shape.prefix_len // shape.page_size
    assert n_pre * shape.page_size == shape.prefix_len
    n_priv = (lens.astype(np.int64) + shape.page_size - 1) // shape.page_size
    used = int(n_pre + n_priv.sum())
    num_pages = used + shape.extra_pages
    if shape.permute_pages:
        perm = _rng(seed, 7).permutation(num_pages).astype(np.int32)
    else:
        perm = np.arange(num_pages, dtype=np.int32)
    max_blocks = int(n_pre + (n_priv.max() if len(n_priv) else 0))
    bt = np.full((shape.n_branches, max_blocks), -1, dtype=np.int32)
    cursor = n_pre
    for b in range(shape.n_branches):
        bt[b, :n_pre] = perm[:n_pre]
        nb = int(n_priv[b])
        bt[b, n_pre:n_pre + nb] = perm[cursor:cursor + nb]
        cursor += nb
    return bt, num_pages, max_blocks


def make_attn_case(shape: AttnShape, seed: int, layer: int = 0, q_scale: float = 1.0,
                   kv_scale: float = 1.0) -> AttnCase:
    """Q/K/V ~ N(0,1) rounded to bf16 (RNE).  `layer` selects an independent K/V/Q
    draw that shares the block table (one table serves all layers of a step)."""
    bt, num_pages, max_blocks = make_block_table(shape, seed)
    rng = _rng(seed + 1000003 * layer, 1)
    R = shape.rows_per_branch
    q = _normal_bf16(rng, (shape.n_branches, R, shape.n_q_heads, shape.head_dim), q_scale)
    k = _normal_bf16(rng, (num_pages, shape.n_kv_heads, shape.page_size, shape.head_dim), kv_scale)
    v = _normal_bf16(rng, (num_pages, shape.n_kv_heads, shape.page_size, shape.head_dim), kv_scale)
    return AttnCase(shape=shape, q=q, k_pages=k, v_pages=v, block_table=bt,
                    branch_lens=shape.lens().copy(), prefix_len=shape.prefix_len,
                    num_pages=num_pages, max_blocks=max_blocks, meta={"seed": seed, "layer": layer})


def token_slot(case: AttnCase, branch: int, logical_token: int):
    """(physical page, slot) of logical token t of a branch (prefix first, then private)."""
    page = int(case.block_table[branch, logical_token // case.shape.page_size])
    return page, logical_token % case.shape.page_size


def poison_unused_slots(case: AttnCase, bits: int = 0x7FC0) -> None:
    """Overwrite every KV slot no query may read (ragged tail of each branch's last page,
    unused pool pages) with a bf16 bit pattern (default NaN)."""
    used = np.zeros((case.num_pages, case.shape.page_size), dtype=bool)
    ps = case.shape.page_size
    n_pre = case.prefix_len // ps
    for b in range(case.shape.n_branches):
        used[case.block_table[b, :n_pre], :] = True
        L = int(case.branch_lens[b])
        for j in range((L + ps - 1) // ps):
            pg = case.block_table[b, n_pre + j]
            n = min(ps, L - j * ps)
            used[pg, :n] = True
    mask = ~used
    for arr in (case.k_pages, case.v_pages):
        view = arr.transpose(0, 2, 1, 3)      # [page][slot][head][d]
        view[mask] = np.uint16(bits)


# --------------------------------------------------------------------------- #
# several prefix groups per call (several questions in flight, each with its own shared prompt)
# --------------------------------------------------------------------------- #
@dataclass
class GroupCase:
    """Branches numbered group by group; the branches of group g share the first group_prefix_lens[g] / 16
    entries of their block-table rows."""
    n_q_heads: int
    n_kv_heads: int
    gamma: int
    group_sizes: np.ndarray        # int32 [n_groups]
    group_prefix_lens: np.ndarray  # int32 [n_groups], multiples of PAGE
    q: np.ndarray
    k_pages: np.ndarray
    v_pages: np.ndarray
    block_table: np.ndarray        # int32 [N][max_blocks]
    branch_lens: np.ndarray        # int32 [N]
    num_pages: int
    max_blocks: int

    @property
    def n_branches(self) -> int:
        return int(self.group_sizes.sum())

    def group_of_branch(self) -> np.ndarray:
        return np.repeat(np.arange(len(self.group_sizes)), self.group_sizes)

    def unique_kv_bytes(self) -> int:
        toks = int(self.group_prefix_lens.astype(np.int64).sum() + self.branch_lens.astype(np.int64).sum())
        return toks * self.n_kv_heads * HEAD_DIM * 2 * 2

    def as_single_group(self, g: int) -> AttnCase:
        """Group g alone as an ordinary one-prefix case on the same pools (views, not copies)."""
        b0 = int(self.group_sizes[:g].sum()); b1 = b0 + int(self.group_sizes[g])
        shape = AttnShape(f"group{g}", n_q_heads=self.n_q_heads, n_kv_heads=self.n_kv_heads,
                          prefix_len=int(self.group_prefix_lens[g]), n_branches=b1 - b0, gamma=self.gamma,
                          branch_lens=tuple(int(v) for v in self.branch_lens[b0:b1]))
        return AttnCase(shape=shape, q=self.q[b0:b1], k_pages=self.k_pages, v_pages=self.v_pages,
                        block_table=self.block_table[b0:b1], branch_lens=self.branch_lens[b0:b1],
                        prefix_len=int(self.group_prefix_lens[g]), num_pages=self.num_pages, max_blocks=self.max_blocks)


def make_group_case(n_q_heads: int, n_kv_heads: int, gamma: int, group_sizes, group_prefix_lens, branch_lens,
                    seed: int, permute_pages: bool = True, extra_pages: int = 0, layer: int = 0) -> GroupCase:
    group_sizes = np.asarray(group_sizes, dtype=np.int32)
    group_prefix_lens = np.asarray(group_prefix_lens, dtype=np.int32)
    lens = np.asarray(branch_lens, dtype=np.int32)
    assert len(group_sizes) == len(group_prefix_lens) and lens.shape == (int(group_sizes.sum()),)
    assert (group_prefix_lens % PAGE == 0).all()
    n_pre = group_prefix_lens // PAGE
    n_priv = (lens.astype(np.int64) + PAGE - 1) // PAGE
    used = int(n_pre.sum() + n_priv.sum())
    num_pages = used + extra_pages
    perm = _rng(seed, 7).permutation(num_pages).astype(np.int32) if permute_pages else np.arange(num_pages, dtype=np.int32)
    group = np.repeat(np.arange(len(group_sizes)), group_sizes)
    max_blocks = int((n_pre[group] + n_priv).max())
    bt = np.full((len(lens), max_blocks), -1, dtype=np.int32)
    cursor, b = 0, 0
    for g, size in enumerate(group_sizes):
        shared = perm[cursor:cursor + n_pre[g]]
        cursor += int(n_pre[g])
        for _ in range(int(size)):
            bt[b, :n_pre[g]] = shared
            nb = int(n_priv[b])
            bt[b, n_pre[g]:n_pre[g] + nb] = perm[cursor:cursor + nb]
            cursor += nb
            b += 1
    rng = _rng(seed + 1000003 * layer, 1)
    q = _normal_bf16(rng, (len(lens), gamma + 1, n_q_heads, HEAD_DIM))
    k = _normal_bf16(rng, (num_pages, n_kv_heads, PAGE, HEAD_DIM))
    v = _normal_bf16(rng, (num_pages, n_kv_heads, PAGE, HEAD_DIM))
    return GroupCase(n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, gamma=gamma, group_sizes=group_sizes,
                     group_prefix_lens=group_prefix_lens, q=q, k_pages=k, v_pages=v, block_table=bt,
                     branch_lens=lens.copy(), num_pages=num_pages, max_blocks=max_blocks)


def poison_unused_slots_groups(case: GroupCase, bits: int = 0x7FC0) -> None:
    """As poison_unused_slots, for a case with several prefix groups."""
    used = np.zeros((case.num_pages, PAGE), dtype=bool)
    group = case.group_of_branch()
    for b in range(case.n_branches):
        n_pre = int(case.group_prefix_lens[group[b]]) // PAGE
        used[case.block_table[b, :n_pre], :] = True
        L = int(case.branch_lens[b])
        for j in range((L + PAGE - 1) // PAGE):
            used[case.block_table[b, n_pre + j], :min(PAGE, L - j * PAGE)] = True
    for arr in (case.k_pages, case.v_pages):
        arr.transpose(0, 2, 1, 3)[~used] = np.uint16(bits)


# --------------------------------------------------------------------------- #
# draft token trees (tree verification)
# --------------------------------------------------------------------------- #
def make_tree_parents(n_branches: int, n_nodes: int, max_depth: int, seed: int) -> np.ndarray:
    """Random draft trees: parents[b][i] in [-1, i) (-1 = child of the last committed
    token), depth of every node <= max_depth (root children have depth 1)."""
    rng = _rng(seed, 31)
    parents = np.full((n_branches, n_nodes), -1, dtype=np.int32)
    for b in range(n_branches):
        depth = np.zeros(n_nodes, dtype=np.int32)
        for i in range(n_nodes):
            while True:
                p = int(rng.integers(-1, i))
                d = 1 if p < 0 else depth[p] + 1
                if d <= max_depth:
                    break
            parents[b, i] = p
            depth[i] = d
    return parents


# --------------------------------------------------------------------------- #
# accept inputs
# --------------------------------------------------------------------------- #
@dataclass
class AcceptCase:
    p_target: np.ndarray      # float32 [N][gamma+1][V]
    q_draft: np.ndarray       # float32 [N][gamma][V]
    draft_tokens: np.ndarray  # int32   [N][gamma]
    uniforms: np.ndarray      # float32 [N][gamma+1], 24-bit fractions in [0,1)
    n_branches: int
    gamma: int
    vocab: int


def _softmax_rows_f32(logits: np.ndarray) -> np.ndarray:
    """Turns logits into a probability vector (input preparation: fp64 softmax -> fp32)."""
    z = logits.astype(np.float64)
    z -= z.max(axis=-1, keepdims=True)
    np.exp(z, out=z)
    z /= z.sum(axis=-1, keepdims=True)
    return z.astype(np.float32)


def uniforms24(rng: np.random.Generator, shape) -> np.ndarray:
    """U[0,1) on a 2^-24 grid, exactly representable in fp32 and always < 1."""
    k = rng.integers(0, 1 << 24, size=shape, dtype=np.int64)
    return (k.astype(np.float64) / float(1 << 24)).astype(np.float32)


def sample_from_rows(rng: np.random.Generator, probs: np.ndarray) -> np.ndarray:
    """One categorical draw per row of probs[..., V] (inverse CDF in fp64)."""
    flat = probs.reshape(-1, probs.shape[-1]).astype(np.float64)
    cdf = np.cumsum(flat, axis=-1)
    u = rng.random(flat.shape[0]) * cdf[:, -1]
    idx = np.array([np.searchsorted(cdf[i], u[i], side="right") for i in range(flat.shape[0])])
    idx = np.minimum(idx, probs.shape[-1] - 1)
    return idx.reshape(probs.shape[:-1]).astype(np.int32)


def make_accept_case(n_branches: int, gamma: int, vocab: int, sigma: float, seed: int,
                     draft_noise: Optional[float] = None) -> AcceptCase:
    """Target and draft logits ~ N(0, sigma) (sigma = standard deviation).

    draft_noise=None: independent target and draft logits (the default recipe).
    draft_noise=tau: draft logits = target logits + N(0, tau), which gives the high
    acceptance rates (0.7..0.9) the paper reports for its model pairs (Appendix A.1).
    Draft tokens are drawn from q_draft."""
    rng = _rng(seed, 2)
    tl = rng.standard_normal(size=(n_branches, gamma + 1, vocab), dtype=np.float32) * np.float32(sigma)
    if draft_noise is None:
        dl = rng.standard_normal(size=(n_branches, gamma, vocab), dtype=np.float32) * np.float32(sigma)
    else:
        dl = tl[:, :gamma, :] + rng.standard_normal(size=(n_branches, gamma, vocab),
                                                    dtype=np.float32) * np.float32(draft_noise)
    p = _softmax_rows_f32(tl)
    q = _softmax_rows_f32(dl) if gamma > 0 else np.zeros((n_branches, 0, vocab), np.float32)
    toks = sample_from_rows(rng, q) if gamma > 0 else np.zeros((n_branches, 0), np.int32)
    u = uniforms24(rng, (n_branches, gamma + 1))
    return AcceptCase(p_target=p, q_draft=q, draft_tokens=toks, uniforms=u,
                      n_branches=n_branches, gamma=gamma, vocab=vocab)


@dataclass
class AcceptLogitsCase:
    target_logits: np.ndarray  # [N][gamma+1][V] float32, or uint16 bf16 bits when made with bf16=True
    draft_logits: np.ndarray   # [N][gamma][V]
    draft_tokens: np.ndarray   # int32 [N][gamma]
    uniforms: np.ndarray       # float32 [N][gamma+1]
    n_branches: int
    gamma: int
    vocab: int
    bf16: bool


def make_accept_logits_case(n_branches: int, gamma: int, vocab: int, sigma: float, seed: int,
                            draft_noise: Optional[float] = None, bf16: bool = False) -> AcceptLogitsCase:
    """The logits behind `make_accept_case` (same recipe: N(0, sigma) logits, independent or target + noise),
    kept as logits: fp32, or rounded to bf16 and carried as uint16 bit patterns.  Draft tokens are drawn from
    the fp64 softmax of the (rounded) draft logits."""
    rng = _rng(seed, 3)
    tl = rng.standard_normal(size=(n_branches, gamma + 1, vocab), dtype=np.float32) * np.float32(sigma)
    if draft_noise is None:
        dl = rng.standard_normal(size=(n_branches, gamma, vocab), dtype=np.float32) * np.float32(sigma)
    else:
        dl = tl[:, :gamma, :] + rng.standard_normal(size=(n_branches, gamma, vocab),
                                                    dtype=np.float32) * np.float32(draft_noise)
    if bf16:
        tl_out, dl_out = f32_to_bf16_bits(tl), f32_to_bf16_bits(dl)
        dl = bf16_bits_to_f32(dl_out)
    else:
        tl_out, dl_out = tl, dl
    toks = sample_from_rows(rng, _softmax_rows_f32(dl)) if gamma > 0 else np.zeros((n_branches, 0), np.int32)
    u = uniforms24(rng, (n_branches, gamma + 1))
    return AcceptLogitsCase(target_logits=tl_out, draft_logits=dl_out, draft_tokens=toks, uniforms=u,
                            n_branches=n_branches, gamma=gamma, vocab=vocab, bf16=bf16)


def with_branches(shape: AttnShape, **kw) -> AttnShape:
    return replace(shape, **kw)
