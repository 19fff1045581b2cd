"""The cost-model helpers (Section 3.2) against the numbers the paper prints in Table 1 / Section 4.2,
for the plain restatement in oracle/cost_model.py and for the library's host functions."""
import os

import numpy as np
import pytest

from oracle import cost_model
from paper_2510_26527_b200 import binding, buildlib

HERE = os.path.dirname(os.path.abspath(__file__))


def _rows():
    out = []
    with open(os.path.join(HERE, "golden", "table1_model_insertion.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                p = line.split()
                out.append((p[0],) + tuple(float(x) for x in p[1:]))
    return out


@pytest.fixture(scope="module")
def lib():
    buildlib.build()
    return binding.load_library()


@pytest.mark.parametrize("row", _rows(), ids=lambda r: r[0])
def test_insertion_criterion_reproduces_table_1(lib, row):
    name, T_i, L_i_new, T_new, L_new, T_next, L_i, p_lhs, p_rhs, improves = row
    lhs, rhs = cost_model.insertion_sides(T_new, T_i, L_new, L_i, L_i_new)
    assert abs(lhs - p_lhs) < 2e-3                         # the paper prints two or three digits
    assert abs(abs(rhs) - p_rhs) < 2e-3                    # case 1 prints the magnitude of a negative number
    assert (lhs < rhs) == bool(improves)
    if name == "non_compliant":
        assert rhs < 0
    got, g_lhs, g_rhs = binding.polyspec_cost_insertion(T_new, T_i, L_new, L_i, L_i_new)
    assert got == bool(improves) and g_lhs == pytest.approx(lhs, rel=1e-15) and g_rhs == pytest.approx(rhs, rel=1e-15)


def test_total_time_matches_the_dualistic_formula_and_the_restatement(lib):
    # n = 2 reduces to the dualistic expression of Section 3.2: N/L_1 T_1 + beta N/L_1 T_2
    N, T1, T2, L1, beta = 1000.0, 22.0, 4.0, 4.34, 1.7
    want = N / L1 * T1 + beta * N / L1 * T2
    assert cost_model.total_time([T1, T2], [L1], beta, N) == pytest.approx(want, rel=1e-15)
    assert binding.polyspec_cost_total_time([T1, T2], [L1], beta, N) == pytest.approx(want, rel=1e-15)
    r = np.random.default_rng(0)
    for n in (3, 4, 6):
        T = r.uniform(1, 30, n).tolist()
        L = r.uniform(1.5, 9, n - 1).tolist()
        assert binding.polyspec_cost_total_time(T, L, 1.3, 512) == pytest.approx(cost_model.total_time(T, L, 1.3, 512), rel=1e-14)
    assert np.isnan(binding.polyspec_cost_total_time([1.0, 2.0], [0.0], 1.0, 10))
    with pytest.raises(ValueError):
        binding.polyspec_cost_insertion(1.0, 0.0, 1.0, 1.0, 1.0)
