"""gbs_search_clip_ratio (Algorithm 1's loop with the quantization error as objective) against the
oracle's Algorithm 1 driven by the oracle's own clip error, on the same seeded rows.  Both visit the
same states unless two objective values are closer than the clip-error tolerance; then the first pass
where they part must be such a near-tie."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_13989_b200 import Plan, binding, synth
from paper_2504_13989_b200 import build as gbs_build
from parity_util import TOL_CLIP

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

CASES = [
    # workload, rows, bits, eps
    ("tiny", 64, 4, 1 / 64),
    ("llama4096", 96, 3, 1 / 64),
    ("llama4096", 33, 4, 1 / 256),
    ("qwen3584", 64, 3, 1 / 32),
    ("kv128", 1000, 3, 1 / 64),
    ("mlp18944", 8, 4, 1 / 16),
]


@pytest.mark.parametrize("name,rows,bits,eps", CASES)
def test_search_matches_algorithm_1_on_the_oracle(name, rows, bits, eps):
    gbs_build.build()
    w = synth.WORKLOADS[name]
    x = synth.make_host(name, rows)
    trace = []
    m_ref, f_ref, it_ref = oracle.search_clip_ratio_rows(synth.to_oracle_array(x), w.d, w.d_pad, w.m, bits, w.group,
                                                         eps, trace)
    with Plan(w.d, w.d_pad, w.m, bits, w.group, w.alpha) as plan:
        res = plan.search_clip_ratio(x.to(DEV), eps)
        assert plan.device_status() == 0
    assert res.evaluations == res.iterations + 1
    assert res.rounds <= (res.iterations + 4) // 5 + 1
    assert res.b - res.a <= eps and res.a <= res.alpha <= res.b
    if res.alpha == np.float32(m_ref) and res.iterations == it_ref:
        np.testing.assert_allclose(res.err, f_ref, rtol=TOL_CLIP)
        return
    # the two parted: some pass of the oracle's trace must have compared two values within the tolerance
    f_m, near_tie = None, False
    fm_hist = [oracle.clip_error_rows(synth.to_oracle_array(x), w.d, w.d_pad, w.m, bits, w.group, np.array([0.5]))[0]]
    for (_, xq, f_x, a, b, mm) in trace:
        f_m = fm_hist[-1]
        if abs(f_x - f_m) <= 4 * TOL_CLIP * f_m:
            near_tie = True
        fm_hist.append(min(f_m, f_x))
    assert near_tie, "search diverged from Algorithm 1 without a near-tie: %r vs %r" % (
        (res.alpha, res.iterations), (m_ref, it_ref))


def test_search_argument_errors():
    with Plan(128, 128, 1, 4, 0, 1.0) as plan:
        x = torch.zeros((4, 128), dtype=torch.bfloat16, device=DEV)
        for eps in (0.0, 1.0, -0.5, float("nan")):
            with pytest.raises(binding.GbsError):
                plan.search_clip_ratio(x, eps)


def test_batched_search_equals_independent_searches_and_resumes():
    """P projections of different shapes searched together visit, each, the states of its own single search;
    stopping after every round and resuming from the stored states gives the same list L."""
    gbs_build.build()
    specs = [("llama4096", 96, 3), ("qwen3584", 64, 3), ("kv128", 1000, 3), ("llama4096", 33, 4), ("mlp18944", 8, 4),
             ("tiny", 64, 4)]
    eps = 1 / 64
    plans, xs, singles = [], [], []
    for name, rows, bits in specs:
        w = synth.WORKLOADS[name]
        pl = Plan(w.d, w.d_pad, w.m, bits, w.group, w.alpha)
        x = synth.make_host(name, rows).to(DEV)
        plans.append(pl)
        xs.append(x)
        singles.append(pl.search_clip_ratio(x, eps))
    alphas, states, rounds = binding.gbs_search_clip_ratio_batch([p.handle for p in plans], xs, eps)
    assert rounds == max(s.rounds for s in singles)               # one wait per round, not per projection
    for a, st, s in zip(alphas, states, singles):
        assert st.done == 1 and a == s.alpha and st.iteration == s.iterations and st.evaluations == s.evaluations
        # the K sums are accumulated with fp64 atomics across CTAs: equal up to summation order
        assert np.isclose(st.f_m, s.err, rtol=1e-9) and (np.float32(st.a), np.float32(st.b)) == (np.float32(s.a), np.float32(s.b))
    # resumable: one round per call, states copied through bytes in between
    sts, total = None, 0
    while True:
        al2, sts, r = binding.gbs_search_clip_ratio_batch([p.handle for p in plans], xs, eps, states=sts, max_rounds=1)
        sts = [binding.SearchState.from_buffer_copy(bytes(s)) for s in sts]
        total += r
        if all(s.done for s in sts):
            break
        assert total < 20
    assert al2 == alphas and total == rounds
    for p in plans:
        assert p.device_status() == 0
        p.close()
