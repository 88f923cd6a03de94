"""Prefill-time model (Eq. 2) and placement cost (Section 5.3): host arithmetic, no GPU."""
import numpy as np

from paper_2609_04774_b200 import prefill_model as pm


def test_remaining_workload_matches_eq1():
    assert pm.remaining_workload(4096, 12288) == 58722304
    assert pm.remaining_workload(1, 0) == 1


def test_fit_recovers_planted_coefficients():
    true = pm.PrefillModel(d=2.0e-5, a=0.0, b=3.0e-9, c=1.0e-8, alpha=4.0e-13)
    rows = [(R, P, C) for R in (1024, 4096, 16384, 65536) for P in (0, 2048, 16384, 65536) for C in (1, 2, 4, 8)]
    R, P, C = (np.array(x, dtype=np.float64) for x in zip(*rows))
    t = true.predict(R, P, C)
    got = pm.fit(R, P, C, t)
    pred = got.predict(R, P, C)
    assert np.abs(pred / t - 1).max() < 1e-6
    assert abs(got.alpha / true.alpha - 1) < 1e-4 and abs(got.b / true.b - 1) < 1e-3
    assert min(got.d, got.a, got.b, got.c, got.alpha) >= 0


def test_placement_cost_formula_and_choice():
    m = pm.PrefillModel(d=1e-4, a=2e-8, b=1e-9, c=1e-8, alpha=5e-13)
    R, P = 60000, 4096
    s4, s8 = float(m.predict(R, P, 4)), float(m.predict(R, P, 8))
    assert s8 < s4                                                   # more ranks: shorter service time
    j4 = pm.placement_cost(0.0, s4, 4, s4, 4, beta=1.5, lam=0.2)
    j8 = pm.placement_cost(0.0, s8, 8, s4, 4, beta=1.5, lam=0.2)
    assert j4 == 1.5 * s4                                            # no extra GPU time at the smallest degree
    assert abs(j8 - (1.5 * s8 + 0.2 * (8 * s8 - 4 * s4))) < 1e-15
    # a short request prefers the small degree once GPU time is charged; a queue on that worker flips it
    short = [{"C": 4, "R": 512, "P": 0}, {"C": 8, "R": 512, "P": 0}]
    assert pm.choose_worker(m, short, beta=1.0, lam=1.0)[0] == 0
    short[0]["queue_delay"] = 1.0
    assert pm.choose_worker(m, short, beta=1.0, lam=1.0)[0] == 1
    # a cache hit on the larger-degree worker lowers its service time
    hit = [{"C": 4, "R": 20000, "P": 0}, {"C": 8, "R": 2000, "P": 18000}]
    assert pm.choose_worker(m, hit, beta=2.0, lam=0.1)[0] == 1
