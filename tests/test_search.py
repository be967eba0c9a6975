"""The library's host-side latency model and T search against the oracle's (no GPU needed)."""
import itertools

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
