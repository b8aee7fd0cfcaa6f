"""Pins of the oracle's attention density (Sec. 4.1) against what the definition fixes."""
import numpy as np

import oracle


def _segments(rng, n, sides, D):
    return [rng.standard_normal((n, s * s, D)) for s in sides]


def test_total_mass_equals_the_number_of_queries():
    rng = np.random.default_rng(1)
    sides, heads, rows, D = (1, 2, 3, 4), 3, 2, 8
    Ks = _segments(rng, rows * heads, sides, D)
    Q = rng.standard_normal((rows * heads, 16, D))
    runs = [(0, 0, 1), (1, 0, 4), (3, 0, 16)]
    d = oracle.attention_density(Q, Ks, runs, 0.4, heads)
    counts = np.array([c for _, _, c in runs], dtype=np.float64)
    # every query's probabilities sum to 1, so count-weighted densities add up to T per head
    assert np.allclose(d @ counts, 16.0, rtol=0, atol=1e-12)


def test_uniform_attention_gives_every_key_the_same_density():
    rng = np.random.default_rng(2)
    sides, heads, rows, D = (1, 2, 3), 2, 3, 4
    Ks = _segments(rng, rows * heads, sides, D)
    Q = np.zeros((rows * heads, 9, D))
    runs = [(0, 0, 1), (1, 1, 2), (2, 0, 9)]
    d = oracle.attention_density(Q, Ks, runs, 1.0, heads)
    assert np.allclose(d, 9.0 / 12.0, rtol=0, atol=1e-13)    # T queries spread over L = 12 keys


def test_brute_force_on_a_tiny_case():
    rng = np.random.default_rng(3)
    sides, heads, rows, D = (1, 2), 2, 2, 3
    Ks = _segments(rng, rows * heads, sides, D)
    Q = rng.standard_normal((rows * heads, 4, D))
    runs = [(0, 0, 1), (1, 0, 4)]
    d = oracle.attention_density(Q, Ks, runs, 0.7, heads)
    want = np.zeros((heads, 2))
    for item in range(rows * heads):
        head = item % heads
        keys = [Ks[0][item, 0]] + [Ks[1][item, t] for t in range(4)]
        for q in range(4):
            w = [np.exp(0.7 * float(np.dot(Q[item, q], k))) for k in keys]
            z = sum(w)
            want[head, 0] += w[0] / z / 1 / rows
            want[head, 1] += sum(w[1:]) / z / 4 / rows
    assert np.allclose(d, want, rtol=1e-12, atol=0)


def test_a_key_that_dominates_collects_the_mass_of_its_scale():
    # one key of scale 1 is aligned with every query and very long: its scale's density approaches T / T_1
    heads, rows, D = 1, 1, 4
    K0 = np.zeros((1, 1, D))
    K1 = np.zeros((1, 4, D))
    K1[0, 2, 0] = 50.0
    Q = np.zeros((1, 6, D))
    Q[:, :, 0] = 1.0
    d = oracle.attention_density(Q, [K0, K1], [(0, 0, 1), (1, 0, 4)], 1.0, heads)
    assert abs(d[0, 1] - 6.0 / 4.0) < 1e-12 and d[0, 0] < 1e-12
