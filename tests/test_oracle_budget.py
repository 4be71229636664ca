"""Pins for the oracle's budget search (threshold chosen on a grid to land on a kept fraction).

The search is this build's reading (the paper gives budgets, Table 1, and the trend of Table 4b, not
a procedure), so the pins are: a closed form on keys whose kept fraction is a known step function of
the threshold, brute force over the whole grid, the end cases, and the grid's float32 values.
"""
import math

import numpy as np
import pytest

import oracle

DELIM = (7,)


def _pairs_at_angles(angles_deg, d=16):
    """One sequence, one head: chunks of two tokens (then a delimiter) whose keys are unit vectors
    `angle` apart, so a pair merges iff cos(angle) > tau.  Returns ids, K, V (float32)."""
    P = len(angles_deg)
    n = 3 * P
    ids = np.full((1, n), 100, dtype=np.int32)
    ids[0, 2::3] = DELIM[0]
    K = np.zeros((1, 1, n, d), dtype=np.float32)
    rng = np.random.default_rng(3)
    for p, a in enumerate(angles_deg):
        K[0, 0, 3 * p, 0] = 1.0
        K[0, 0, 3 * p + 1, 0] = math.cos(math.radians(a))
        K[0, 0, 3 * p + 1, 1] = math.sin(math.radians(a))
        K[0, 0, 3 * p + 2] = rng.normal(size=d)          # the delimiter's own key
    V = rng.normal(size=K.shape).astype(np.float32)
    return ids, K, V


def test_grid_is_float32_arithmetic_in_the_stated_order():
    g = oracle.tau_grid(0.5, 0.9, 9)
    assert g.dtype == np.float32 and len(g) == 9 and g[0] == np.float32(0.5)
    step = (np.float32(0.9) - np.float32(0.5)) / np.float32(8)
    assert g[3] == np.float32(np.float32(0.5) + np.float32(np.float32(3) * step))
    assert abs(float(g[8]) - 0.9) < 1e-6 and np.all(np.diff(g) > 0)


def test_closed_form_on_pairs_at_known_angles():
    # cos: 10 deg .985, 30 .866, 45 .707, 60 .5, 75 .259, 85 .087; kept cores = 6 delimiters + 6 + (pairs with cos <= tau)
    angles = [10, 30, 45, 60, 75, 85]
    ids, K, V = _pairs_at_angles(angles)
    cosines = [math.cos(math.radians(a)) for a in angles]
    grid = oracle.tau_grid(0.0, 1.0, 21)            # steps of 0.05
    n = ids.shape[1]
    for target_cores in range(12, 19):
        target = target_cores / n
        want_cores = [12 + sum(c <= float(t) for c in cosines) for t in grid]
        r = oracle.budget(ids, DELIM, K, V, target, 0.0, 1.0, 21)
        assert r["target_cores"] == target_cores
        # the first grid threshold that keeps at least the target, or its predecessor if that is nearer
        first = next(i for i, c in enumerate(want_cores) if c >= target_cores)
        if first > 0 and (target_cores - want_cores[first - 1]) <= (want_cores[first] - target_cores):
            first -= 1
        # the search assumes a monotone count, and every index with the same count is as good: compare counts
        assert want_cores[r["index"]] == want_cores[first], (target_cores, r["index"], first)
        assert int(r["core_len"].sum()) == want_cores[r["index"]]
        assert r["tau"] == float(grid[r["index"]])


def test_end_cases_and_tie_rule():
    ids, K, V = _pairs_at_angles([20, 40, 70])
    n = ids.shape[1]
    lo = oracle.budget(ids, DELIM, K, V, 0.0, 0.1, 0.99, 5)       # even the lowest threshold keeps more than nothing
    assert lo["index"] == 0 and len(lo["visited"]) == 2
    hi = oracle.budget(ids, DELIM, K, V, 1.0, 0.1, 0.5, 5)        # cos 20 = .94 stays merged at every threshold
    assert hi["index"] == 4 and int(hi["core_len"].sum()) < n
    # tie rule, worked by hand: pairs at 20, 50, 50 degrees (cos .940, .643, .643), n = 9 tokens.
    # cores = 3 delimiters + 3 first tokens + pairs with cos <= tau: 6 up to tau = 0.6, 8 from 0.7 on, 9 at 1.0.
    # Aim at 7 cores: the interval closes on indices 6 (6 cores) and 7 (8 cores), equally far: the lower one.
    ids, K, V = _pairs_at_angles([20, 50, 50])
    r = oracle.budget(ids, DELIM, K, V, 7 / 9, 0.0, 1.0, 11)
    assert r["target_cores"] == 7 and r["index"] == 6 and int(r["core_len"].sum()) == 6
    assert [i for i, _ in r["visited"]] == [0, 10, 5, 7, 6]
    assert [c for _, c in r["visited"]] == [6, 9, 6, 8, 6]
    # aim at 8: index 7 is the first that keeps 8
    r = oracle.budget(ids, DELIM, K, V, 8 / 9, 0.0, 1.0, 11)
    assert r["index"] == 7 and int(r["core_len"].sum()) == 8


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_search_agrees_with_brute_force_over_the_grid_when_counts_are_monotone(seed):
    rng = np.random.default_rng(seed)
    B, Hkv, n, d = 2, 2, 96, 24
    ids = rng.integers(100, 200, size=(B, n)).astype(np.int32)
    ids[rng.random((B, n)) < 0.08] = DELIM[0]
    cent = rng.normal(size=(4, d))
    K = (cent[rng.integers(0, 4, size=(B, Hkv, n))] + 0.55 * rng.normal(size=(B, Hkv, n, d))).astype(np.float32)
    V = rng.normal(size=K.shape).astype(np.float32)
    T = 17
    grid = oracle.tau_grid(0.3, 0.95, T)
    counts = [int(oracle.compress(ids, DELIM, K, V, float(t))["core_len"].sum()) for t in grid]
    if any(b < a for a, b in zip(counts, counts[1:])):
        pytest.skip("greedy counts not monotone for this seed: bisection is then a heuristic")
    for frac in (0.35, 0.5, 0.7):
        r = oracle.budget(ids, DELIM, K, V, frac, 0.3, 0.95, T)
        tc = r["target_cores"]
        best = min(abs(c - tc) for c in counts)
        assert abs(counts[r["index"]] - tc) == best
        assert len(r["visited"]) <= 2 + math.ceil(math.log2(T - 1))
        for i, c in r["visited"]:
            assert counts[i] == c
