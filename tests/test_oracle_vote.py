"""Pins for the host-side helpers of the oracle: majority vote (Section 3.2), the
confidence-weighted variants (Section 4.6) and greedy search (Algorithm 1)."""
from collections import Counter
from itertools import product
from pathlib import Path

import numpy as np

import oracle

GOLDEN = Path(__file__).parent / "golden"


def test_majority_vote_all_assignments_of_5_branches_to_3_answers():
    for assign in product((10, 20, 30), repeat=5):
        cnt = Counter(assign)
        top = max(cnt.values())
        want = next(a for a in assign if cnt[a] == top)       # first-occurring among the tied
        w, v, s = oracle.majority_vote(np.array(assign))
        assert (w, v, s) == (want, top, float(top))


def test_weighted_vote_and_max_modes():
    ans = np.array([7, 8, 7, 9, 8], np.int64)
    wts = np.array([0.2, 0.5, 0.2, 0.45, 0.0], np.float32)
    w, v, s = oracle.majority_vote(ans, wts, mode=0)          # sums: 7 -> .4, 8 -> .5, 9 -> .45
    assert (w, v) == (8, 2) and abs(s - 0.5) < 1e-7
    w, v, s = oracle.majority_vote(ans, wts, mode=1)          # single best branch
    assert (w, v) == (8, 2) and abs(s - 0.5) < 1e-7
    wts2 = np.array([0.3, 0.5, 0.3, 0.45, 0.0], np.float32)   # 7 -> .6 wins the vote, 8 the max
    assert oracle.majority_vote(ans, wts2, mode=0)[0] == 7
    assert oracle.majority_vote(ans, wts2, mode=1)[0] == 8
    # brute force over small random cases
    rng = np.random.default_rng(0)
    for _ in range(200):
        n = int(rng.integers(1, 9))
        a = rng.integers(0, 4, size=n)
        wt = rng.integers(0, 8, size=n).astype(np.float32) / 8
        sums = {}
        for x, y in zip(a, wt):
            sums[x] = sums.get(x, 0.0) + float(y)
        best = max(sums.values())
        want = next(x for x in a if sums[x] == best)
        assert oracle.majority_vote(a, wt, 0)[0] == want
        assert oracle.majority_vote(a, wt, 1)[0] == a[int(np.argmax(wt))]


def test_greedy_search_step_counts_match_the_paper_table():
    """On a surface that rises monotonically towards (B*, gamma*) and falls beyond it, greedy
    search reaches the optimum in log2 B* + gamma* + 1 steps; grid search needs 7 x 8 = 56."""
    rows = [tuple(map(int, l.split())) for l in (GOLDEN / "greedy_search_steps.txt").read_text().splitlines()
            if l and not l.startswith("#")]
    assert len(rows) == 4
    for b_opt, g_opt, steps in rows:
        lb_opt = int(np.log2(b_opt))
        lb, g = np.meshgrid(np.arange(7), np.arange(8), indexing="ij")
        acc = 90.0 - 3.0 * np.abs(lb - lb_opt) - 2.0 * np.abs(g - g_opt)
        assert acc.size == 56
        B, gamma, best, n_steps, n_evals = oracle.greedy_search(acc)
        assert (B, gamma) == (b_opt, g_opt) and best == acc.max()
        assert n_steps == steps == lb_opt + g_opt + 1
        assert n_evals == 1 + 2 * n_steps


def test_greedy_search_stops_at_local_optimum_and_table_edge():
    acc = np.array([[1.0, 0.5], [0.9, 3.0]])                  # (2,1) is better but unreachable
    assert oracle.greedy_search(acc)[:2] == (1, 0)
    acc = np.arange(12, dtype=np.float64).reshape(3, 4)       # always improving: ends at the edge
    assert oracle.greedy_search(acc)[:2] == (4, 3)


def test_grid_search_evaluation_count_and_optimum():
    """56 evaluations on the paper's 7 x 8 lattice; the optimum is the table's maximum, which greedy
    search also reaches on the unimodal surfaces of the search-comparison table (Section 4.5)."""
    b_max, n_gamma, evals = [tuple(map(int, l.split())) for l in
                             (GOLDEN / "grid_search_evaluations.txt").read_text().splitlines()
                             if l and not l.startswith("#")][0]
    n_logb = int(np.log2(b_max)) + 1
    rows = [tuple(map(int, l.split())) for l in (GOLDEN / "greedy_search_steps.txt").read_text().splitlines()
            if l and not l.startswith("#")]
    for b_opt, g_opt, _ in rows:
        lb, g = np.meshgrid(np.arange(n_logb), np.arange(n_gamma), indexing="ij")
        acc = 90.0 - 3.0 * np.abs(lb - int(np.log2(b_opt))) - 2.0 * np.abs(g - g_opt)
        B, gamma, best, n = oracle.grid_search(acc)
        assert n == evals
        assert (B, gamma) == (b_opt, g_opt) and best == acc.max()
        assert oracle.greedy_search(acc)[:3] == (B, gamma, best)
    # a second hill that greedy search cannot see from (1, 0): the grid finds it, greedy does not
    acc = np.zeros((n_logb, n_gamma))
    acc[0, 0], acc[1, 0], acc[0, 1] = 5.0, 4.0, 4.0
    acc[5, 6] = 9.0
    assert oracle.grid_search(acc)[:3] == (32, 6, 9.0)
    assert oracle.greedy_search(acc)[:3] == (1, 0, 5.0)
    # equal optima: the first in (B, gamma) order
    acc = np.ones((3, 3))
    assert oracle.grid_search(acc)[:2] == (1, 0)
