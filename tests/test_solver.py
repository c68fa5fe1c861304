"""Pins for the off-path host solver: the paper's worked toy batch, its bounds, brute force on tiny instances (no GPU)."""
import itertools
import os

import numpy as np
import pytest

from paper_2608_13057_b200 import solver as S

GOLD = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "paper_cost_numbers.txt")) as fh:
    for line in fh:
        line = line.split("#")[0].split()
        if line:
            GOLD[line[0]] = [float(v) for v in line[1:]]


def _feasible(x, counts, replicas):
    assert np.all(x >= 0)
    assert np.array_equal(x.sum(1), np.asarray(counts))
    for e, r in enumerate(replicas):
        off = [g for g in range(x.shape[1]) if g not in r]
        assert np.all(x[e, off] == 0)


def test_figure_1b_time_balancing_splits_only_the_hot_expert():
    p = S.CostParams(a=0, b=GOLD["fig1b_b"][0], c=0, beta=GOLD["fig1b_beta"][0])
    counts = [600] + [30] * 6
    replicas = [[0, 1]] * 7
    x = S.tempo_fast(counts, replicas, 2, p)
    _feasible(x, counts, replicas)
    assert abs(S.makespan(x, p) - GOLD["fig1b_time_balancing_us"][0]) < 1e-9          # 60 us
    assert int((x[1:] > 0).sum()) == 6                                                    # cold experts stay whole
    # the two proxies the figure compares against
    assert abs(S.makespan(S.uniform_split(counts, replicas, 2), p) - GOLD["fig1b_token_balancing_us"][0]) < 1e-9
    act = np.zeros((7, 2), np.int64)
    act[[0, 1, 2, 3], 0] = [600, 30, 30, 30]
    act[[4, 5, 6], 1] = 30
    assert abs(S.makespan(act, p) - GOLD["fig1b_activation_balancing_us"][0]) < 1e-9


def _brute_force(counts, replicas, n_gpus, p):
    """Exact integer optimum for tiny instances with at most two replicas per expert."""
    best = None
    ranges = []
    for e, n in enumerate(counts):
        r = replicas[e]
        ranges.append(range(n + 1) if len(r) == 2 else [n])
    for choice in itertools.product(*ranges):
        x = np.zeros((len(counts), n_gpus), np.int64)
        for e, m in enumerate(choice):
            r = replicas[e]
            x[e, r[0]] = m
            if len(r) == 2:
                x[e, r[1]] = counts[e] - m
        ms = S.makespan(x, p)
        best = ms if best is None else min(best, ms)
    return best


@pytest.mark.parametrize("seed", range(12))
def test_against_brute_force_and_bounds_on_tiny_instances(seed):
    g = np.random.default_rng(seed)
    n_gpus = 2
    E = int(g.integers(2, 6))
    counts = [int(v) for v in g.integers(0, 9, size=E)]
    full = bool(g.integers(0, 2))
    replicas = [[0, 1] if (full or g.random() < 0.5) else [int(g.integers(0, 2))] for _ in range(E)]
    p = S.CostParams(a=float(g.uniform(0, 2)), b=float(g.uniform(0.5, 3)), c=float(g.uniform(0, 2)),
                     beta=float(g.uniform(0.1, 1.0)))
    x = S.tempo_fast(counts, replicas, n_gpus, p)
    _feasible(x, counts, replicas)
    opt = _brute_force(counts, replicas, n_gpus, p)
    got = S.makespan(x, p)
    assert got >= opt - 1e-9
    assert got <= 1.15 * opt + 1e-9                      # the paper reports <= 1.14x OPT worst case
    if full:
        lb = S.lower_bound(counts, n_gpus, p)
        assert lb <= opt + 1e-9                           # LB <= OPT
        a3 = S.makespan(S.round_robin_a3(counts, n_gpus), p)
        n_max = max(counts)
        assert a3 <= opt + max(p.b, p.beta * n_max) + 1e-9    # Theorem 2 (the integer optimum bounds the real one from above)
        assert got <= (opt + max(p.b, p.beta * n_max)) / (1 - 0.01) + 1e-9   # the ensemble carries the bound, weakened by tau


def test_degenerate_limits():
    g = np.random.default_rng(3)
    counts = [int(v) for v in g.integers(1, 400, size=12)]
    replicas = [[0, 1, 2, 3]] * 12
    # b -> 0: only tokens matter, the optimum is perfect token balance (Lemma 1)
    p = S.CostParams(a=0, b=0, c=0, beta=1.0)
    x = S.tempo_fast(counts, replicas, 4, p)
    assert S.makespan(x, p) <= -(-sum(counts) // 4) + 1e-9
    # beta -> 0: only activations matter, the optimum is ceil(E/g) whole experts per GPU (Lemma 2)
    p = S.CostParams(a=0, b=1.0, c=0, beta=0)
    x = S.tempo_fast(counts, replicas, 4, p)
    assert S.makespan(x, p) == 3.0


def test_never_worse_than_token_lp_beyond_the_tolerance_and_tile_snapping():
    g = np.random.default_rng(5)
    for trial in range(6):
        E, n_gpus = 24, 4
        counts = [int(v) for v in (g.zipf(1.6, size=E) * 40).clip(0, 4000)]
        replicas = [sorted(g.choice(n_gpus, size=int(g.integers(1, 4)), replace=False).tolist()) for _ in range(E)]
        p = S.CostParams(a=34.9, b=3.95, c=34.8, beta=0.0154, b2=1.23)     # the paper's Testbed-B Qwen3-235B fit
        x = S.tempo_fast(counts, replicas, n_gpus, p)
        _feasible(x, counts, replicas)
        lp = S.makespan(S.token_lp(counts, replicas, n_gpus), p)
        assert S.makespan(x, p) <= lp / (1 - 0.01) + 1e-9
        assert S.makespan(x, p) <= S.makespan(S.uniform_split(counts, replicas, n_gpus), p) + 1e-9


def test_quota_table_layout():
    x = np.array([[5, 0, 3], [0, 7, 0]])
    q = S.quota_table(x, [[2, 0], [1]], 2)
    assert q.tolist() == [[3, 5], [7, 0]]
