"""Python access to the CPU oracle (oracle/tts_oracle.cpp).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline / reference legs may import
this package; the product (paper_2505_19634_b200) never does.  It compiles the C++ file with
g++ into oracle/_build/ on first use and exposes numpy-in / numpy-out wrappers.
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
