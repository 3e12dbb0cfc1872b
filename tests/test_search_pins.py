"""Pins of the oracle's Algorithm 1 (Gradual Binary Search, the loop for one projection): hand-worked
traces, the bracket invariants, convergence on convex objectives, and the evaluation count."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "alg1_traces.txt")
OBJECTIVES = {"(x-0.3)^2": lambda x: (x - 0.3) ** 2, "x": lambda x: x}


def _golden():
    cases, cur = [], None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("objective"):
            _, name, _, eps = line.split()
            cur = (name, float(eps), [])
            cases.append(cur)
        else:
            cur[2].append(tuple(float(v) for v in line.split()))
    return cases


def test_hand_worked_traces():
    cases = _golden()
    assert len(cases) == 2
    for name, eps, want in cases:
        trace = []
        m, f_m, iterations = oracle.gradual_binary_search(OBJECTIVES[name], eps, trace)
        assert iterations == len(want)
        for got, exp in zip(trace, want):
            np.testing.assert_allclose(got, exp, rtol=1e-12, atol=1e-15)
        assert m == want[-1][5]


@pytest.mark.parametrize("xstar", [0.07, 0.3, 0.5, 0.77, 0.99])
@pytest.mark.parametrize("eps", [1 / 8, 1 / 64, 1 / 1024])
def test_bracket_invariants_and_convergence_on_convex_objectives(xstar, eps):
    calls = []

    def f(x):
        calls.append(x)
        return abs(x - xstar) ** 1.5 + 0.25 * (x - xstar) ** 2

    trace = []
    m, f_m, iterations = oracle.gradual_binary_search(f, eps, trace)
    assert len(calls) == iterations + 1                      # one evaluation per pass, plus f(1/2)
    width = 1.0
    for (_, x, f_x, a, b, mm) in trace:
        assert 0.0 <= a <= mm <= b <= 1.0 and 0.0 < x < 1.0
        assert a <= xstar <= b                                # the minimiser never leaves the bracket
        assert b - a <= width
        width = b - a
    assert width <= eps and abs(m - xstar) <= eps
    assert f_m == f(m)


def test_search_on_rows_returns_a_clip_ratio_that_beats_its_neighbours():
    rng = np.random.Generator(np.random.PCG64(5))
    x = (0.5 * rng.standard_t(3, size=(16, 256))).astype(np.float32)
    m, f_m, it = oracle.search_clip_ratio_rows(x, 256, 256, 1, 3, 0, 1 / 64)
    assert 0.0 < m < 1.0
    grid = oracle.clip_error_rows(x, 256, 256, 1, 3, 0, np.linspace(0.05, 1.0, 96))
    assert f_m <= 1.05 * grid.min()                           # close to the best of a fine grid
