"""Pins for the oracle's inter-scale similarity (Eq. 4), CPU only."""
import math

import numpy as np
import torch
import torch.nn.functional as F

import oracle
from paper_2511_16047_b200 import synth


def _torch_resize(src, s_in, s_out):
    n, _, D = src.shape
    x = torch.from_numpy(src).reshape(n, s_in, s_in, D).permute(0, 3, 1, 2)
    y = F.interpolate(x, size=(s_out, s_out), mode="bilinear", align_corners=False)
    return y.permute(0, 2, 3, 1).reshape(n, s_out * s_out, D).numpy()


def test_resize_matches_library_bilinear_half_pixel():
    rng = np.random.default_rng(0)
    for s_in, s_out in [(1, 2), (2, 3), (3, 4), (5, 6), (6, 8), (13, 16), (8, 12), (4, 4), (6, 3)]:
        src = rng.standard_normal((3, s_in * s_in, 5))
        np.testing.assert_allclose(oracle.bilinear_resize(src, s_in, s_out), _torch_resize(src, s_in, s_out),
                                   rtol=0, atol=1e-13)


def test_identity_and_constant_fields():
    rng = np.random.default_rng(1)
    K = rng.standard_normal((2, 25, 4))
    assert oracle.similarity_ss(K, 5, K, 5) == 0.0
    assert oracle.similarity(K, 5, K, 5) == 0.0
    const_prev = np.full((2, 9, 4), 0.75)
    const_cur = np.full((2, 16, 4), 0.75)
    assert oracle.similarity_ss(const_prev, 3, const_cur, 4) < 1e-26
    # a linear ramp along x is reproduced exactly in the interior by bilinear interpolation
    s_in, s_out = 4, 8
    xs_in = (np.arange(s_in) + 0.5) / s_in
    xs_out = (np.arange(s_out) + 0.5) / s_out
    src = np.tile(xs_in[None, :], (s_in, 1)).reshape(1, -1, 1)
    dst = oracle.bilinear_resize(src, s_in, s_out).reshape(s_out, s_out)
    np.testing.assert_allclose(dst[:, 1:-1], np.tile(xs_out[None, 1:-1], (s_out, 1)), atol=1e-14)


def test_similarity_is_negative_l2_norm():
    rng = np.random.default_rng(2)
    Kp, Kc = rng.standard_normal((2, 9, 3)), rng.standard_normal((2, 16, 3))
    khat = _torch_resize(Kp, 3, 4)
    ss = float(((Kc - khat) ** 2).sum())
    assert abs(oracle.similarity_ss(Kp, 3, Kc, 4) - ss) < 1e-10
    assert abs(oracle.similarity(Kp, 3, Kc, 4) + math.sqrt(ss)) < 1e-10
    # swapping the operands of the difference leaves the norm unchanged, scaling scales it
    assert abs(oracle.similarity(2 * Kp, 3, 2 * Kc, 4) - 2 * oracle.similarity(Kp, 3, Kc, 4)) < 1e-10


def test_expected_value_for_iid_gaussian_fields():
    # E[ss] = sigma^2 * n_items * D * sum_pixels (1 + sum_j w_j^2) for independent N(0, sigma^2) maps
    s_in, s_out, n, D, sigma = 5, 6, 64, 32, 0.125
    eye = np.eye(s_in * s_in).reshape(s_in * s_in, s_in * s_in, 1)   # each basis map as an item
    W = _torch_resize(eye, s_in, s_out)[:, :, 0]                     # [basis, out pixel]
    expect = sigma ** 2 * n * D * float((1.0 + (W ** 2).sum(axis=0)).sum())
    rng = np.random.default_rng(3)
    Kp = rng.standard_normal((n, s_in * s_in, D)) * sigma
    Kc = rng.standard_normal((n, s_out * s_out, D)) * sigma
    ss = oracle.similarity_ss(Kp, s_in, Kc, s_out)
    assert abs(ss - expect) / expect < 0.03


def test_correlated_layers_score_higher_than_independent_ones():
    sides = (4, 5, 6, 8)
    corr = synth.smooth_field_keys(2, 4, sides, 16, seed=9, rho=0.9)
    ind = synth.smooth_field_keys(2, 4, sides, 16, seed=9, rho=0.0)
    for i in range(1, len(sides)):
        def sim(ks):
            a = ks[i - 1].reshape(8, -1, 16).double().numpy()
            b = ks[i].reshape(8, -1, 16).double().numpy()
            return oracle.similarity(a, sides[i - 1], b, sides[i])
        assert sim(corr) > sim(ind)
        assert sim(corr) < 0


def test_classification_rules():
    scores = [-3.0, -1.0, -2.0, -1.0]
    assert oracle.classify_layers(scores, -2.0) == [True, False, False, False]   # strict <
    assert oracle.lowest_similarity_layers(scores, 2) == [True, False, True, False]
    assert oracle.lowest_similarity_layers([-1.0, -1.0, -1.0], 1) == [True, False, False]
