"""Pins for the oracle's exhaustive optimal-deployment search (the paper's placement-quality experiment):
an independent itertools enumeration with exact rationals, counts, hand cases."""
import itertools
from fractions import Fraction

import numpy as np
import pytest


def brute(Pm, models, G, R):
    n = len(models)
    best, count = None, 0
    for rest in itertools.product(range(G), repeat=n - 1):
        assign = (0,) + rest
        if max(assign.count(g) for g in range(G)) > R:
            continue
        count += 1
        cost = sum(Fraction(float(Pm[models[i], models[j]])) + Fraction(float(Pm[models[j], models[i]]))
                   for i in range(n) for j in range(i + 1, n) if assign[i] == assign[j]) / n
        if best is None or cost < best:
            best = cost
    return best, count


@pytest.mark.parametrize("seed", range(5))
def test_optimal_against_itertools(oracle, seed):
    rng = np.random.default_rng(seed)
    P = 7
    Pm = (rng.integers(0, 64, (P, P)) / 64.0).astype(np.float32)       # exact in float32 and in the sums
    n, G, R = int(rng.integers(3, 8)), int(rng.integers(2, 4)), int(rng.integers(2, 4))
    if n > G * R:
        n = G * R
    models = rng.integers(0, P, n)
    want, count = brute(Pm, models, G, R)
    cost, assign, tried = oracle.optimal_assignment(Pm, models, G, R)
    assert tried == count
    # the pair sums are exact (multiples of 1/64); the definition ends with one float32 division by n
    assert cost == np.float32(float(want * n)) / np.float32(n)
    assert assign[0] == 0 and max(np.bincount(assign, minlength=G)) <= R
    c32, c64 = oracle.assignment_cost(Pm, models, assign)
    assert c32 == cost and c64 == pytest.approx(float(want), rel=1e-12)


def test_hand_cases(oracle):
    # two models that hurt each other, two GPUs: apart costs 0, together (0.3 + 0.1) / 2
    Pm = np.array([[0, 0.3], [0.1, 0]], dtype=np.float32)
    assert oracle.optimal_assignment(Pm, [0, 1], 2, 2)[0] == 0.0
    assert oracle.optimal_assignment(Pm, [0, 1], 1, 2)[0] == np.float32((np.float32(0.3) + np.float32(0.1)) / np.float32(2))
    assert oracle.assignment_cost(Pm, [0, 1], [0, 0])[0] == oracle.optimal_assignment(Pm, [0, 1], 1, 2)[0]
    # no feasible deployment
    assert oracle.optimal_assignment(Pm, [0, 1, 0], 1, 2)[0] == -1.0
    # three models, one slot pair: the cheapest pair shares, the third is alone
    Pm = np.zeros((3, 3), dtype=np.float32)
    Pm[0, 1] = Pm[1, 0] = 0.5; Pm[0, 2] = Pm[2, 0] = 0.25; Pm[1, 2] = Pm[2, 1] = 0.125
    cost, assign, tried = oracle.optimal_assignment(Pm, [0, 1, 2], 2, 2)
    assert cost == np.float32(0.25 / 3) and assign[1] == assign[2] != assign[0]
    assert tried == 3                       # {0,1|2}, {0,2|1}, {0|1,2}; all three together does not fit
    # replicas of one model are distinct models of the deployment
    assert oracle.optimal_assignment(np.full((1, 1), 0.2, np.float32), [0, 0, 0], 3, 3)[0] == 0.0
