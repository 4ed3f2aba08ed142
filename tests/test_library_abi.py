"""CPU checks of the boundary: the shared library builds, loads without a GPU and exports every
symbol include/tts.h declares; host-only entry points agree with the oracle; argument errors
are reported as status codes."""
import re
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


def test_majority_vote_matches_oracle_exhaustively():
    for assign in product((10, 20, 30), repeat=5):
        assert tts.tts_majority_vote(assign) == oracle.majority_vote(np.array(assign))[:2]
    rng = np.random.default_rng(1)
    for _ in range(300):
        n = int(rng.integers(1, 12))
        a = rng.integers(-3, 3, size=n)
        w = rng.integers(0, 16, size=n).astype(np.float32) / 16
        assert tts.tts_majority_vote(a, w) == oracle.majority_vote(a, w, 0)[:2]
        assert tts.tts_confidence_max(a, w) == oracle.majority_vote(a, w, 1)[:2]


def test_vote_argument_errors():
    with pytest.raises(tts.TtsError):
        tts.tts_majority_vote([])
    with pytest.raises(tts.TtsError):
        tts.tts_confidence_max([1, 2], None)


def test_greedy_search_matches_oracle_and_paper_step_counts():
    rows = [tuple(map(int, l.split())) for l in (ROOT / "tests/golden/greedy_search_steps.txt").read_text().splitlines()
            if l and not l.startswith("#")]
    for b_opt, g_opt, steps in rows:
        lb_opt = int(np.log2(b_opt))
        lb, g = np.meshgrid(np.arange(7), np.arange(8), indexing="ij")
        acc = 90.0 - 3.0 * np.abs(lb - lb_opt) - 2.0 * np.abs(g - g_opt)

        def task(B, gamma):
            i = int(np.log2(B))
            return acc[i, gamma] if i < 7 and gamma < 8 else -1.0
        got = tts.tts_greedy_search(task)
        want = oracle.greedy_search(acc)
        assert got == (want[0], want[1], want[2], want[3])
        assert got[:2] == (b_opt, g_opt) and got[3] == steps
    rng = np.random.default_rng(2)
    for _ in range(50):
        acc = rng.integers(0, 6, size=(4, 5)).astype(np.float64)
        got = tts.tts_greedy_search(lambda B, g: acc[int(np.log2(B)), g] if B <= 8 and g < 5 else -1.0)
        want = oracle.greedy_search(acc)
        assert got == (want[0], want[1], want[2], want[3])


def test_create_rejects_bad_configs_without_a_gpu():
    lib = tts.load_library()
    import ctypes
    h = ctypes.c_void_p(0)
    good = dict(n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16, max_branches=4, max_rows_per_branch=4,
                max_blocks_per_branch=8, num_pages=8, out_dtype=0, attn_impl=0, softmax_scale=0.0, debug_bounds=0)
    for bad, want in ((dict(head_dim=64), -2), (dict(page_size=32), -2), (dict(n_kv_heads=3), -1),
                      (dict(max_branches=0), -1), (dict(max_rows_per_branch=65), -1), (dict(out_dtype=5), -2),
                      (dict(attn_impl=9), -2), (dict(num_pages=0), -1)):
        cfg = tts.TtsConfig(**{**good, **bad})
        assert lib.tts_create(ctypes.byref(cfg), ctypes.byref(h)) == want, bad
        assert not h.value
    assert lib.tts_create(None, ctypes.byref(h)) == -1
