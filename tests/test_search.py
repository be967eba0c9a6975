"""The library's host-side latency model and T search against the oracle's (no GPU needed)."""
import itertools

import numpy as np

from oracle import latency as L
from paper_2510_19705_b200 import binding


def test_expected_latency_matches_oracle():
    costs = [0.3, 0.9, 2.2, 5.0]
    alphas = [0.55, 0.6, 0.7]
    for T in itertools.product((1, 2, 5), repeat=3):
        a = binding.hsd_expected_latency(costs, alphas, list(T))
        b = L.expected_latency(costs, alphas, list(T))
        assert abs(a - b) <= 1e-12 * b
    assert binding.hsd_expected_latency([7.0], [], []) == 7.0
    # Table 1, row 2 of the paper: target 33, drafter 4, alpha 0.8, T = 5 -> 14.37
    assert abs(binding.hsd_expected_latency([4, 33], [0.8], [5]) - 14.37) < 0.005


def test_search_T_matches_oracle():
    cases = [([0.311, 0.851, 2.202], [0.56, 0.57]), ([1.0, 256.0, 1024.0], [0.7, 0.5]),
             ([0.1, 0.5, 1.0, 4.0], [0.8, 0.75, 0.8]), ([4.0, 33.0], [0.8])]
    for costs, alphas in cases:
        for mono in (True, False):
            T, lat = binding.hsd_search_T(costs, alphas, 15 if len(costs) < 4 else 6, mono)
            want = L.search_T(costs, alphas, 15 if len(costs) < 4 else 6, mono)
            assert T == tuple(want[1]) and abs(lat - want[0]) <= 1e-12 * want[0]
    assert binding.hsd_search_T([4.0, 33.0], [0.8])[0] == (5,)


def _example1():
    """Appendix B, first example of the paper (the golden file holds the numbers)."""
    import os
    costs, rows, lat = None, [], {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "latency_example1.txt")) as f:
        for line in f:
            p = line.split()
            if not p or p[0].startswith("#"):
                continue
            if p[0] == "costs":
                costs = [float(x) for x in p[1:]]
            elif p[0] == "alpha":
                rows.append([None if x == "-" else float(x) for x in p[1:]])
            elif p[0] == "latency":
                lat[int(p[1])] = (float(p[2]), float(p[3]), p[4] == "pinned")
    n = len(costs)
    alpha = [[0.0] * n for _ in range(n)]
    for i, row in enumerate(rows):
        for j, a in enumerate(row, start=1):
            if a is not None:
                alpha[i][j] = a
    return costs, alpha, lat


def test_search_hierarchy_matches_oracle_and_brute_force():
    import random
    rng = random.Random(5)
    for n in (1, 2, 3, 4, 5):
        for _ in range(6):
            costs = sorted(rng.uniform(0.01, 1.0) * 4 ** i for i in range(n))
            alpha = [[0.0] * n for _ in range(n)]
            for i in range(n):
                for j in range(i + 1, n):
                    alpha[i][j] = rng.uniform(0.05, 0.95) * (0.9 ** (j - i - 1))
            T_max = 5 if n > 3 else 8
            lat, sigma, T = binding.hsd_search_hierarchy(costs, alpha, T_max)
            want = L.search_hierarchy(costs, alpha, T_max)
            brute = L.brute_force_hierarchy(costs, alpha, T_max)
            assert abs(lat - want[0]) <= 1e-12 * want[0] and abs(lat - brute[0]) <= 1e-9 * brute[0]
            assert sigma == tuple(want[1]) and T == tuple(want[2])
            assert sigma[-1] == n - 1 and list(sigma) == sorted(set(sigma)) and len(T) == len(sigma) - 1
            assert all(T[k] >= T[k - 1] for k in range(1, len(T)))
            if len(sigma) > 1:      # the returned pair really has the returned latency
                assert abs(L.subset_latency(costs, alpha, list(sigma), list(T)) - lat) <= 1e-12 * lat


def test_search_hierarchy_on_the_papers_worked_example():
    costs, alpha, table = _example1()
    n = len(costs)
    for k, (want, tol, pinned) in table.items():          # the k largest models: adding a smaller one each time
        sub = list(range(n - k, n))
        c = [costs[i] for i in sub]
        a = [[alpha[i][j] for j in sub] for i in sub]
        lat, sigma, T = binding.hsd_search_hierarchy(c, a, 15)
        assert abs(lat - L.search_hierarchy(c, a, 15)[0]) <= 1e-12 * lat
        if pinned:
            assert abs(lat - want) <= tol, (k, lat, want)
    # 3 models: (M5, T=8) under the target, M4 below it with T=4 (indices within the last three: 0 -> 1 -> 2)
    lat, sigma, T = binding.hsd_search_hierarchy(costs[3:], [row[3:] for row in alpha[3:]], 15)
    assert sigma == (0, 1, 2) and T == (4, 8)


def test_search_hierarchy_rejects_bad_arguments():
    import pytest
    with pytest.raises(binding.HsdError):
        binding.hsd_search_hierarchy([1.0, 2.0], [[0.0, 1.5], [0.0, 0.0]], 4)
    with pytest.raises(binding.HsdError):
        binding.hsd_search_hierarchy([1.0, 2.0], [[0.0, 0.5], [0.0, 0.0]], 0)


def test_literal_latency_matches_the_oracle():
    from oracle import latency
    from paper_2510_19705_b200 import binding
    rng = np.random.default_rng(5)
    for _ in range(40):
        n = int(rng.integers(1, 6))
        costs = sorted(rng.uniform(0.1, 10.0, n).tolist())
        alphas = rng.uniform(0.0, 1.0, n - 1).tolist()
        T = [int(t) for t in rng.integers(1, 9, n - 1)]
        want = latency.literal_latency(tuple(costs), tuple(alphas), tuple(T))
        got = binding.hsd_expected_latency_literal(costs, alphas, T)
        assert abs(got - want) <= 1e-12 * max(1.0, abs(want)), (costs, alphas, T)
        if n <= 2:
            assert abs(got - binding.hsd_expected_latency(costs, alphas, T)) <= 1e-12 * max(1.0, got)
        else:
            assert got <= binding.hsd_expected_latency(costs, alphas, T) * (1 + 1e-12)
    # extremes: every draft accepted / every first draft rejected
    assert abs(binding.hsd_expected_latency_literal([1.0, 2.0, 4.0], [1.0, 1.0], [2, 3]) - (1 * (2 * 1.0 + 2.0) + 4.0) / 4.0) < 1e-12   # one round of 3 tokens below, 3 + 1 at the target
    assert abs(binding.hsd_expected_latency_literal([1.0, 2.0, 4.0], [0.0, 0.0], [2, 3]) - (3 * (2 * 1.0 + 2.0) + 4.0) / 1.0) < 1e-12
