"""Python access to the CPU oracle (oracle/tts_oracle.cpp).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline / reference legs may import
this package; the product (paper_2505_19634_b200) never does.  It compiles the C++ file with
g++ into oracle/_build/ on first use and exposes numpy-in / numpy-out wrappers; the tree-path accept
rule and the KV-cache bookkeeping are written here in numpy (token by token, in the order of their
definitions).

Pins: tests/test_oracle_*.py.  Parity unpinned: one property only, the distribution of the token that
`accept_tree` emits (its rule is pinned; see its docstring).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "tts_oracle.cpp"
_LIB = _HERE / "_build" / "libtts_oracle.so"
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> Path:
    """g++ -O2 -ffp-contract=off (so the fp32 accept test is one rounded multiply)."""
    with _lock:
        if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
            _LIB.parent.mkdir(exist_ok=True)
            tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
            subprocess.run(["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-shared", "-fPIC",
                            "-pthread", str(_SRC), "-o", str(tmp)], check=True)
            os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
    return _lib


def n_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct)) if a is not None else None


def verify_attn(q, k_pages, v_pages, block_table, prefix_len, branch_lens, gamma,
                mask_kind: int = 0, tree_parents=None, scale=None, row_sel=None,
                n_threads=None, return_weight_sums: bool = False):
    """Exact attention of the verify step.  q/k_pages/v_pages are uint16 bf16 bit arrays
    shaped [N][R][Hq][D] and [num_pages][Hkv][page][D].  Returns fp64 out [N][R][Hq][D]
    (or [n_sel][D] when row_sel, an int array of (b, i, h) triples, is given)."""
    q = np.ascontiguousarray(q, dtype=np.uint16)
    k_pages = np.ascontiguousarray(k_pages, dtype=np.uint16)
    v_pages = np.ascontiguousarray(v_pages, dtype=np.uint16)
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    branch_lens = np.ascontiguousarray(branch_lens, dtype=np.int32)
    N, R, Hq, D = q.shape
    assert R == gamma + 1
    _, Hkv, page, D2 = k_pages.shape
    assert D2 == D and v_pages.shape == k_pages.shape
    assert block_table.shape[0] == N and branch_lens.shape == (N,)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    if tree_parents is not None:
        tree_parents = np.ascontiguousarray(tree_parents, dtype=np.int32)
        assert tree_parents.shape == (N, R)
    if row_sel is not None:
        row_sel = np.ascontiguousarray(row_sel, dtype=np.int32).reshape(-1, 3)
        n_sel = row_sel.shape[0]
        out = np.zeros((n_sel, D), dtype=np.float64)
    else:
        n_sel = 0
        out = np.zeros((N, R, Hq, D), dtype=np.float64)
    wsum = np.zeros(out.size // D, dtype=np.float64)
    rc = lib().oracle_verify_attn(
        _p(q, ctypes.c_uint16), _p(k_pages, ctypes.c_uint16), _p(v_pages, ctypes.c_uint16),
        _p(block_table, ctypes.c_int32), ctypes.c_int(block_table.shape[1]),
        ctypes.c_int(int(prefix_len)), _p(branch_lens, ctypes.c_int32), ctypes.c_int(N),
        ctypes.c_int(int(gamma)), ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(D),
        ctypes.c_int(page), ctypes.c_double(float(scale)), ctypes.c_int(int(mask_kind)),
        _p(tree_parents, ctypes.c_int32), _p(row_sel, ctypes.c_int32), ctypes.c_int(n_sel),
        _p(out, ctypes.c_double), _p(wsum, ctypes.c_double),
        ctypes.c_int(int(n_threads or n_cores())))
    if rc != 0:
        raise ValueError(f"oracle_verify_attn: inconsistent arguments (rc={rc})")
    if return_weight_sums:
        return out, wsum.reshape(out.shape[:-1])
    return out


def verify_attn_groups(q, k_pages, v_pages, block_table, group_sizes, group_prefix_lens, branch_lens, gamma,
                       n_threads=None):
    """Several questions in one call (the multi-request setting of the paper's appendix: #Req questions, each
    with B branches that share that question's prompt).  Branches are numbered group by group; the branches
    of group g share a prefix of group_prefix_lens[g] tokens, listed first in their block-table rows.  By
    definition the groups do not interact: the result for a branch is the single-question result
    (`verify_attn`) for its group alone, with that group's prefix length.  Returns fp64 out [N][R][Hq][D]."""
    q = np.ascontiguousarray(q, dtype=np.uint16)
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    branch_lens = np.ascontiguousarray(branch_lens, dtype=np.int32)
    sizes = [int(v) for v in group_sizes]
    assert sum(sizes) == q.shape[0] and len(sizes) == len(group_prefix_lens)
    out = np.zeros(q.shape, dtype=np.float64)
    b0 = 0
    for size, prefix_len in zip(sizes, group_prefix_lens):
        b1 = b0 + size
        if size > 0:
            out[b0:b1] = verify_attn(q[b0:b1], k_pages, v_pages, block_table[b0:b1], int(prefix_len),
                                     branch_lens[b0:b1], gamma, n_threads=n_threads)
        b0 = b1
    return out


def accept(p_target, q_draft, draft_tokens, uniforms, n_threads=None):
    """Speculative-sampling accept/resample.  Returns (accepted_len, next_token, near_flags)."""
    p_target = np.ascontiguousarray(p_target, dtype=np.float32)
    N, R, V = p_target.shape
    gamma = R - 1
    q_draft = np.ascontiguousarray(q_draft, dtype=np.float32).reshape(N, gamma, V)
    draft_tokens = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(N, gamma)
    uniforms = np.ascontiguousarray(uniforms, dtype=np.float32)
    assert uniforms.shape == (N, R)
    acc = np.zeros(N, dtype=np.int32)
    nxt = np.zeros(N, dtype=np.int32)
    near = np.zeros(N, dtype=np.int32)
    rc = lib().oracle_accept(_p(p_target, ctypes.c_float), _p(q_draft, ctypes.c_float),
                             _p(draft_tokens, ctypes.c_int32), _p(uniforms, ctypes.c_float),
                             ctypes.c_int(N), ctypes.c_int(gamma), ctypes.c_int(V),
                             _p(acc, ctypes.c_int32), _p(nxt, ctypes.c_int32),
                             _p(near, ctypes.c_int32), ctypes.c_int(int(n_threads or n_cores())))
    if rc != 0:
        raise ValueError("oracle_accept: inconsistent arguments")
    return acc, nxt, near


def softmax_rows(logits, n_threads=None):
    """fp32 probabilities from logits [..., V] (fp32, or uint16 bf16 bits, which are widened exactly), by the
    step-by-step fp32 arithmetic written out above `oracle_softmax_rows` in tts_oracle.cpp."""
    a = np.asarray(logits)
    if a.dtype == np.uint16:
        a = (a.astype(np.uint32) << np.uint32(16)).view(np.float32)
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty_like(a)
    V = a.shape[-1]
    rc = lib().oracle_softmax_rows(_p(a, ctypes.c_float), ctypes.c_long(a.size // V), ctypes.c_int(V),
                                   _p(out, ctypes.c_float), ctypes.c_int(int(n_threads or n_cores())))
    if rc != 0:
        raise ValueError("oracle_softmax_rows: inconsistent arguments")
    return out


def accept_logits(target_logits, draft_logits, draft_tokens, uniforms, n_threads=None):
    """The accept rule fed with logits: p_i = softmax_rows(target_logits[:, i]), q_i = softmax_rows(draft_logits
    [:, i]), then `accept` on those probabilities, unchanged.  Returns (accepted_len, next_token, near_flags)."""
    p = softmax_rows(target_logits, n_threads)
    N, R, V = p.shape
    q = softmax_rows(draft_logits, n_threads) if R > 1 else np.zeros((N, 0, V), np.float32)
    return accept(p, q, draft_tokens, uniforms, n_threads)


def majority_vote(answers, weights=None, mode: int = 0):
    """Returns (winner, votes, score)."""
    answers = np.ascontiguousarray(answers, dtype=np.int64)
    if weights is not None:
        weights = np.ascontiguousarray(weights, dtype=np.float32)
        assert weights.shape == answers.shape
    w = ctypes.c_int64(0)
    v = ctypes.c_int32(0)
    s = ctypes.c_double(0.0)
    rc = lib().oracle_majority_vote(_p(answers, ctypes.c_int64), _p(weights, ctypes.c_float),
                                    ctypes.c_int(answers.size), ctypes.c_int(mode),
                                    ctypes.byref(w), ctypes.byref(v), ctypes.byref(s))
    if rc != 0:
        raise ValueError("oracle_majority_vote: inconsistent arguments")
    return int(w.value), int(v.value), float(s.value)


def accept_tree(p_target, q_draft, draft_tokens, tree_parents, uniforms):
    """Accept test along the paths of a draft tree: the chain rule of `accept` applied along every
    root-to-leaf path (tree verification; the paper does not spell the rule out, Section 4.1 only names
    the drafting models).  Steps, per branch, in this order:
      1. node i passes iff p(x_i) > 0 and u_i * q_i(x_i) <= p(x_i) with one fp32 multiply, p being row 0
         of p_target for a child of the last committed token (parent -1) and row 1 + parent otherwise;
      2. a node is accepted iff it and all its ancestors pass; for every leaf, count the accepted nodes
         on its path; the leaf with the largest count wins, ties to the lowest leaf index;
      3. the final draw with u_n: from norm(max(0, p - q_k)) in fp32 (p if that is identically zero) for the
         first node k of the winning path that failed, p the row of k's parent; or from row 1 + leaf when
         the whole path was accepted; sums in fp64 in index order, smallest x whose running sum exceeds
         u_n * Z, else the last x with weight > 0.
    Returns (accepted_len, last_node, next_token, near_flags) with near_flags as in `accept`.
    Pinned: a chain reproduces `accept`; brute force over all pass patterns of small trees.  The
    DISTRIBUTION of the emitted token under this path-selection rule is parity unpinned (the rule is not
    lossless across siblings, so there is no closed form to test it against)."""
    P = np.ascontiguousarray(p_target, dtype=np.float32)
    N, n1, V = P.shape
    n = n1 - 1
    Q = np.ascontiguousarray(q_draft, dtype=np.float32).reshape(N, n, V)
    X = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(N, n)
    PAR = np.ascontiguousarray(tree_parents, dtype=np.int32).reshape(N, n)
    U = np.ascontiguousarray(uniforms, dtype=np.float32)
    assert U.shape == (N, n + 1)
    acc = np.zeros(N, np.int32); last = np.zeros(N, np.int32); nxt = np.zeros(N, np.int32); near = np.zeros(N, np.int32)
    for b in range(N):
        flags = 0
        passes = []
        for i in range(n):
            par = int(PAR[b, i])
            if par < -1 or par >= i:
                raise ValueError("accept_tree: a parent must be -1 or an earlier node")
            x = int(X[b, i])
            p = P[b, par + 1, x]
            q = Q[b, i, x]
            uq = np.float32(U[b, i]) * np.float32(q)                       # one fp32 multiply
            if abs(float(uq) - float(p)) <= 1e-6 * max(float(p), float(q)):
                flags |= 1
            passes.append(bool(p > np.float32(0) and uq <= p))
        children = [[] for _ in range(n)]
        for i in range(n):
            if PAR[b, i] >= 0:
                children[int(PAR[b, i])].append(i)
        best_leaf, best_count, best_path = -1, -1, []
        for leaf in range(n):
            if children[leaf]:
                continue
            path = []
            i = leaf
            while i >= 0:
                path.append(i)
                i = int(PAR[b, i])
            path.reverse()                                                # root side first
            count = 0
            for node in path:
                if not passes[node]:
                    break
                count += 1
            if count > best_count:
                best_leaf, best_count, best_path = leaf, count, path
        if best_leaf < 0:                                                 # no nodes: the bonus token of the committed prefix
            best_count, best_path = 0, []
        acc[b] = best_count
        last[b] = best_path[best_count - 1] if best_count > 0 else -1
        if best_count < len(best_path):
            k = best_path[best_count]
            pk = P[b, int(PAR[b, k]) + 1]
            r = np.maximum(pk - Q[b, k], np.float32(0)).astype(np.float32)
            if not (np.cumsum(r.astype(np.float64))[-1] > 0.0):
                r = pk.copy()
        else:
            r = P[b, best_leaf + 1].copy()
        C = np.cumsum(r.astype(np.float64))                               # sequential fp64 sums in index order
        Z = float(C[-1])
        t = float(U[b, n]) * Z
        over = np.nonzero(C > t)[0]
        if over.size:
            chosen = int(over[0])
            prev = float(C[chosen - 1]) if chosen > 0 else 0.0
            if abs(float(C[chosen]) - t) <= 1e-9 * Z or (chosen > 0 and abs(t - prev) <= 1e-9 * Z):
                flags |= 2
        else:
            pos = np.nonzero(r > 0)[0]
            chosen = int(pos[-1]) if pos.size else V - 1
            flags |= 2
        nxt[b] = chosen
        near[b] = flags
    return acc, last, nxt, near


def kv_append(k_pages, v_pages, k_new, v_new, block_table, prefix_len, branch_lens, page_size: int = 16):
    """KV-cache bookkeeping before the verify step (Section 3.2, speculative decoding: the target model
    scores the last committed token and the gamma drafts of every branch in one pass, so their keys and
    values join the cache first).  Token by token, as the definition reads: row i of branch b is private
    token branch_lens[b] - R + i, i.e. logical token prefix_len + branch_lens[b] - R + i, which lives in
    page block_table[b][token // page_size] at slot token % page_size.  Pools [num_pages][Hkv][page][D]
    and new rows [N][R][Hkv][D] as uint16 bf16 bits; returns the two updated pools (copies)."""
    k = np.array(k_pages, dtype=np.uint16, copy=True)
    v = np.array(v_pages, dtype=np.uint16, copy=True)
    k_new = np.asarray(k_new, dtype=np.uint16)
    v_new = np.asarray(v_new, dtype=np.uint16)
    n, r = k_new.shape[0], k_new.shape[1]
    for b in range(n):
        length = int(branch_lens[b])
        if length < r:
            raise ValueError("kv_append: a branch is shorter than the rows appended")
        for i in range(r):
            token = prefix_len + length - r + i
            page = int(block_table[b, token // page_size])
            slot = token % page_size
            for h in range(k_new.shape[2]):
                k[page, h, slot, :] = k_new[b, i, h, :]
                v[page, h, slot, :] = v_new[b, i, h, :]
    return k, v


def kv_rollback(branch_lens, accepted_len, gamma: int):
    """After the accept test the gamma - accepted_len rejected drafts of every branch leave the cache
    (Section 3.2; the resampled or bonus token has no key yet: it is the first row of the next step)."""
    lens = np.array(branch_lens, dtype=np.int64, copy=True)
    for b in range(lens.shape[0]):
        a = int(accepted_len[b])
        if a < 0 or a > gamma:
            raise ValueError("kv_rollback: accepted_len outside [0, gamma]")
        lens[b] = lens[b] - (gamma - a)
    return lens.astype(np.int32)


def greedy_search(acc_table):
    """Algorithm 1 on a dense accuracy table acc[log2 B][gamma].
    Returns (B, gamma, acc, steps, evaluations)."""
    t = np.ascontiguousarray(acc_table, dtype=np.float64)
    lb = ctypes.c_int(0); g = ctypes.c_int(0); a = ctypes.c_double(0)
    st = ctypes.c_int(0); ev = ctypes.c_int(0)
    rc = lib().oracle_greedy_search(_p(t, ctypes.c_double), ctypes.c_int(t.shape[0]),
                                    ctypes.c_int(t.shape[1]), ctypes.byref(lb), ctypes.byref(g),
                                    ctypes.byref(a), ctypes.byref(st), ctypes.byref(ev))
    if rc != 0:
        raise ValueError("oracle_greedy_search: inconsistent arguments")
    return 1 << lb.value, g.value, a.value, st.value, ev.value


def grid_search(acc_table):
    """The exhaustive baseline of Section 3.3 / Section 4.5: every configuration of the table
    acc[log2 B][gamma] is evaluated once and the most accurate one is kept (equal optima: the first
    in (B, gamma) order).  Returns (B, gamma, acc, evaluations)."""
    t = np.asarray(acc_table, dtype=np.float64)
    best, evaluations = None, 0
    for lb in range(t.shape[0]):
        for g in range(t.shape[1]):
            evaluations += 1
            if best is None or t[lb, g] > best[2]:
                best = (1 << lb, g, float(t[lb, g]))
    return best[0], best[1], best[2], evaluations
