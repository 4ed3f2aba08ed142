"""CPU checks of the boundary: the shared library builds, loads without a GPU and exports every
symbol include/tts.h declares; host-only entry points agree with the oracle; argument errors
are reported as status codes."""
import re
from collections import Counter
from itertools import product
from pathlib import Path

import numpy as np
import pytest

import oracle
import paper_2505_19634_b200 as tts
from paper_2505_19634_b200.build import build_library

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def test_header_symbols_are_exported():
    header = (ROOT / "include" / "tts.h").read_text()
    declared = set(re.findall(r"TTS_API\s+[\w\s\*]+?\b(tts_\w+)\s*\(", header))
    assert declared == set(tts.EXPORTED_SYMBOLS)
    lib = tts.load_library()
    for name in declared:
        assert getattr(lib, name) is not None


def test_strerror():
    assert tts.tts_strerror(0) == "ok"
    assert "invalid" in tts.tts_strerror(-1)
    assert "unknown" in tts.tts_strerror(-99)


def _counter_vote(answers, weights=None):
    """Brute force with collections.Counter / a dict of fp64 sums: (winner, branches that gave it)."""
    answers = [int(a) for a in answers]
    if weights is None:
        score = Counter(answers)
    else:
        score = {}
        for a, w in zip(answers, weights):
            score[a] = score.get(a, 0.0) + float(w)
    top = max(score.values())
    winner = next(a for a in answers if score[a] == top)          # first-occurring among the tied
    return winner, answers.count(winner)


def test_majority_vote_against_counter_brute_force():
    for assign in product((10, 20, 30), repeat=5):
        assert tts.tts_majority_vote(assign) == _counter_vote(assign)
        assert tts.tts_majority_vote(assign) == oracle.majority_vote(np.array(assign))[:2]
    rng = np.random.default_rng(1)
    for _ in range(300):
        n = int(rng.integers(1, 12))
        a = rng.integers(-3, 3, size=n)
        w = rng.integers(0, 16, size=n).astype(np.float32) / 16       # dyadic: the sums are exact
        assert tts.tts_majority_vote(a, w) == _counter_vote(a, w)
        assert tts.tts_majority_vote(a, w) == oracle.majority_vote(a, w, 0)[:2]
        best_branch = int(np.argmax(w))                                # first of equal maxima
        assert tts.tts_confidence_max(a, w) == (int(a[best_branch]), int((a == a[best_branch]).sum()))
        assert tts.tts_confidence_max(a, w) == oracle.majority_vote(a, w, 1)[:2]
    # many branches, large and negative answer ids
    a = rng.integers(-2**40, 2**40, size=6)[rng.integers(0, 6, size=257)]
    assert tts.tts_majority_vote(a) == _counter_vote(a)


def test_vote_argument_errors():
    with pytest.raises(tts.TtsError):
        tts.tts_majority_vote([])
    with pytest.raises(tts.TtsError):
        tts.tts_confidence_max([1, 2], None)


def _golden_rows(name):
    return [tuple(map(int, l.split())) for l in (ROOT / "tests/golden" / name).read_text().splitlines()
            if l and not l.startswith("#")]


def _surface(b_opt, g_opt, n_logb=7, n_gamma=8):
    lb, g = np.meshgrid(np.arange(n_logb), np.arange(n_gamma), indexing="ij")
    return 90.0 - 3.0 * np.abs(lb - int(np.log2(b_opt))) - 2.0 * np.abs(g - g_opt)


def test_greedy_search_matches_oracle_and_paper_step_counts():
    for b_opt, g_opt, steps in _golden_rows("greedy_search_steps.txt"):
        acc = _surface(b_opt, g_opt)
        got = tts.tts_greedy_search(lambda B, gamma: acc[int(np.log2(B)), gamma])       # default lattice: 7 x 8
        want = oracle.greedy_search(acc)
        assert got[:4] == want[:4]
        assert got[:2] == (b_opt, g_opt) and got[3] == steps
    rng = np.random.default_rng(2)
    for _ in range(50):
        acc = rng.integers(0, 6, size=(4, 5)).astype(np.float64)
        got = tts.tts_greedy_search(lambda B, g: acc[int(np.log2(B)), g], max_branches=8, max_gamma=4)
        assert got[:4] == oracle.greedy_search(acc)[:4]
        # the same lattice expressed through "unavailable" points instead of limits
        got2 = tts.tts_greedy_search(lambda B, g: acc[int(np.log2(B)), g] if B <= 8 and g < 5 else -1.0)
        assert got2[:4] == got[:4]


def test_greedy_search_limits():
    calls = []

    def ever_better(B, gamma):            # improves with every move: only the limits stop the search
        calls.append((B, gamma))
        return float(np.log2(B) + gamma)
    B, gamma, acc, steps, evals = tts.tts_greedy_search(ever_better, max_branches=16, max_gamma=3)
    assert (B, gamma) == (16, 3) and acc == 7.0
    assert all(b <= 16 and g <= 3 for b, g in calls) and evals == len(calls)
    B, gamma, acc, steps, evals = tts.tts_greedy_search(ever_better, max_branches=1 << 20, max_gamma=4096, max_steps=5)
    assert steps == 5 and np.log2(B) + gamma == 5
    for kw in (dict(max_branches=0), dict(max_gamma=-1), dict(max_branches=1 << 21), dict(max_gamma=5000)):
        with pytest.raises(tts.TtsError):
            tts.tts_greedy_search(ever_better, **kw)


def test_grid_search_counts_and_optimum():
    b_max, n_gamma, evals = _golden_rows("grid_search_evaluations.txt")[0]
    for b_opt, g_opt, _ in _golden_rows("greedy_search_steps.txt"):
        acc = _surface(b_opt, g_opt)
        task = lambda B, gamma: acc[int(np.log2(B)), gamma]
        got = tts.tts_grid_search(task, max_branches=b_max, max_gamma=n_gamma - 1)
        assert got == oracle.grid_search(acc)
        assert got[3] == evals and got[:2] == (b_opt, g_opt)
        assert tts.tts_grid_search(task)[3] == evals                   # the default lattice is the paper's
        assert tts.tts_greedy_search(task)[:3] == got[:3]              # greedy reaches the grid optimum here
    acc = np.zeros((7, 8)); acc[0, 0], acc[1, 0], acc[0, 1], acc[5, 6] = 5.0, 4.0, 4.0, 9.0
    task = lambda B, gamma: acc[int(np.log2(B)), gamma]
    assert tts.tts_grid_search(task)[:3] == (32, 6, 9.0) == oracle.grid_search(acc)[:3]
    assert tts.tts_greedy_search(task)[:3] == (1, 0, 5.0)              # a local optimum the grid does not stop at
    rng = np.random.default_rng(4)
    for _ in range(30):
        acc = rng.integers(0, 6, size=(3, 6)).astype(np.float64)
        got = tts.tts_grid_search(lambda B, g: acc[int(np.log2(B)), g], max_branches=4, max_gamma=5)
        assert got == oracle.grid_search(acc)


def test_create_rejects_bad_configs_without_a_gpu():
    lib = tts.load_library()
    import ctypes
    h = ctypes.c_void_p(0)
    good = dict(n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, max_branches=4, max_rows_per_branch=4,
                max_blocks_per_branch=8, num_pages=8, out_dtype=0, attn_impl=0, softmax_scale=0.0, debug_bounds=0, max_ctas=0)
    for bad, want in ((dict(head_dim=64), -2), (dict(page_size=32), -2), (dict(n_kv_heads=3), -1),
                      (dict(max_branches=0), -1), (dict(max_rows_per_branch=65), -1), (dict(out_dtype=5), -2),
                      (dict(attn_impl=9), -2), (dict(num_pages=0), -1)):
        cfg = tts.TtsConfig(**{**good, **bad})
        assert lib.tts_create(ctypes.byref(cfg), ctypes.byref(h)) == want, bad
        assert not h.value
    assert lib.tts_create(None, ctypes.byref(h)) == -1


def test_entry_points_reject_null_contexts_and_bad_groups_without_a_gpu():
    """Host-side argument checks that need no device: every context-taking entry point returns
    TTS_ERR_INVALID for a null context, and the group arrays of the multi-question calls are validated
    before anything else."""
    import ctypes
    lib = tts.load_library()
    i32 = lambda *v: (ctypes.c_int32 * len(v))(*v)
    z = ctypes.c_void_p(0)
    assert lib.tts_attn_plan(z, z, 16, z, 1, 1) == -1
    assert lib.tts_attn_plan_drop(z) == -1
    assert lib.tts_verify_attn(z, z, z, z, z, 16, z, 1, 0, 0, z) == -1
    assert lib.tts_accept_logits(z, z, z, 0, z, z, 1, 0, 8, z, z) == -1
    assert lib.tts_debug_wait_timeout(z, 1000000) == -1
    assert lib.tts_kv_rollback(z, z, z, 1, 0) == -1
    # groups: sizes must be >= 1 and add up to n_branches, at most 64 groups
    for sizes, pre, n in (((2, 1), (16, 0), 4), ((2, 0, 2), (16, 0, 16), 4), ((1,) * 65, (0,) * 65, 65)):
        assert lib.tts_verify_attn_groups(z, z, z, z, z, i32(*sizes), i32(*pre), len(sizes), z, n, 1, z) == -1
        assert lib.tts_attn_plan_groups(z, z, i32(*sizes), i32(*pre), len(sizes), z, n, 2) == -1
