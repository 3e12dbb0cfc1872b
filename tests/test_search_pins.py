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


# ----------------------------------------------------------------------------------------------
# The library's own state machine (gbs_search_clip_ratio_fn, host only) against the oracle's Algorithm 1
# ----------------------------------------------------------------------------------------------
import ctypes

from paper_2504_13989_b200 import binding
from paper_2504_13989_b200 import build as gbs_build


def _objectives():
    yield "(x-0.3)^2", (lambda x: (x - 0.3) ** 2)
    yield "x", (lambda x: x)
    yield "1-x", (lambda x: 1.0 - x)
    yield "|x-0.71|", (lambda x: abs(x - 0.71))
    yield "bumpy", (lambda x: (x - 0.55) ** 2 + 0.01 * np.sin(40.0 * x))
    yield "flat", (lambda x: 1.0)


@pytest.mark.parametrize("eps", [1 / 8, 1 / 64, 1 / 1000])
def test_library_state_machine_visits_the_states_of_algorithm_1(eps):
    """Same objective, evaluated at the float32 clip ratio both sides see: same m, f_m, iteration count, and the
    same sequence of probes."""
    gbs_build.build()
    for name, f in _objectives():
        seen_ref, seen_lib = [], []

        def f32(x, sink):
            x = float(np.float32(x))
            sink.append(x)
            return float(f(x))
        trace = []
        m_ref, fm_ref, it_ref = oracle.gradual_binary_search(lambda x: f32(x, seen_ref), eps, trace)
        st = binding.gbs_search_clip_ratio_fn(lambda a: f32(a, seen_lib), eps)
        assert st.done == 1 and st.iteration == it_ref and st.evaluations == it_ref + 1, name
        assert st.m == m_ref and st.f_m == fm_ref, name
        assert (st.a, st.b) == (trace[-1][3], trace[-1][4]) if trace else (st.a, st.b) == (0.0, 1.0)
        assert seen_lib == seen_ref, name


def test_library_state_machine_resumes_from_a_stored_state():
    """One pass at a time, the state stored as bytes in between, ends where the one-shot call ends."""
    gbs_build.build()
    f = lambda x: (x - 0.37) ** 2
    whole = binding.gbs_search_clip_ratio_fn(f, 1 / 256)
    st = binding.gbs_search_state_init()
    passes = 0
    while not st.done:
        st = binding.gbs_search_clip_ratio_fn(f, 1 / 256, state=st, max_iterations=1)
        st = binding.SearchState.from_buffer_copy(bytes(st))          # "serialised" and read back
        passes += 1
        assert passes < 100
    assert bytes(st) == bytes(whole) and passes >= whole.iteration


def test_library_state_machine_rejects_bad_arguments():
    gbs_build.build()
    lib = binding.lib()
    st = binding.gbs_search_state_init()
    cb = binding.OBJECTIVE_FN(lambda a, c: 0.0)
    assert lib.gbs_search_clip_ratio_fn(cb, None, 0.0, ctypes.byref(st), 0) == binding.GBS_ERR_INVALID_ARG
    assert lib.gbs_search_clip_ratio_fn(cb, None, 0.1, None, 0) == binding.GBS_ERR_INVALID_ARG
    bad = binding.gbs_search_state_init()
    bad.a, bad.b = 0.9, 0.1
    assert lib.gbs_search_clip_ratio_fn(cb, None, 0.1, ctypes.byref(bad), 0) == binding.GBS_ERR_INVALID_ARG
    assert lib.gbs_search_clip_ratio_batch(None, 1, 0.1, None, 0, None, None, None, None) == binding.GBS_ERR_INVALID_ARG
