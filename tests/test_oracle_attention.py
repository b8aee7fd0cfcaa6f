"""Pins for the oracle's attention (fp64, CPU only)."""
import math

import numpy as np
import torch

import oracle
from paper_2511_16047_b200 import synth

SIDES = (1, 2, 3, 4, 5)


def _segments(n, D, seed, sides=SIDES):
    rng = np.random.default_rng(seed)
    Q = [rng.standard_normal((n, s * s, D)) for s in sides]
    K = [rng.standard_normal((n, s * s, D)) for s in sides]
    V = [rng.standard_normal((n, s * s, D)) for s in sides]
    return Q, K, V


def test_full_retention_equals_vanilla_block_causal():
    n, D = 3, 8
    Q, K, V = _segments(n, D, 1)
    scale = 1.0 / math.sqrt(D)
    van = oracle.block_causal_attention(np.concatenate(Q, 1), np.concatenate(K, 1),
                                        np.concatenate(V, 1), SIDES, scale)
    off = 0
    for k, s in enumerate(SIDES):
        keep = oracle.keep_set(k, 2, 2, True)
        out = oracle.attend_selected(Q[k], K, V, keep, scale)
        np.testing.assert_allclose(out, van[:, off:off + s * s], rtol=0, atol=1e-12)
        off += s * s


def test_eviction_changes_the_result_only_when_something_is_evicted():
    n, D = 2, 8
    Q, K, V = _segments(n, D, 2)
    scale = 0.7
    for k in range(len(SIDES)):
        full = oracle.attend_selected(Q[k], K, V, oracle.keep_set(k, 1, 1, True), scale)
        eff = oracle.attend_selected(Q[k], K, V, oracle.keep_set(k, 1, 1, False), scale)
        if k < 2:
            np.testing.assert_array_equal(full, eff)
        else:
            assert np.abs(full - eff).max() > 1e-3


def test_rows_sum_to_one_and_single_key_returns_v():
    n, D = 2, 16
    Q, K, V = _segments(n, D, 3)
    ones = [np.ones_like(v) for v in V]
    out = oracle.attend_selected(Q[4], K, ones, [0, 1, 3, 4], 0.3)
    np.testing.assert_allclose(out, 1.0, rtol=0, atol=1e-14)
    # scale 0 has one query and one key: the output is that key's value, exactly
    out0 = oracle.attend_selected(Q[0], K, V, [0], 0.3)
    np.testing.assert_array_equal(out0, V[0])


def test_zero_queries_give_mean_of_kept_values():
    n, D = 2, 8
    Q, K, V = _segments(n, D, 4)
    keep = [0, 1, 4]
    out = oracle.attend_selected(np.zeros_like(Q[4]), K, V, keep, 1.0)
    mean = np.concatenate([V[s] for s in keep], 1).mean(axis=1, keepdims=True)
    np.testing.assert_allclose(out, np.broadcast_to(mean, out.shape), rtol=0, atol=1e-13)


def test_key_permutation_invariance():
    n, T, L, D = 2, 5, 37, 8
    rng = np.random.default_rng(5)
    Q, K, V = rng.standard_normal((n, T, D)), rng.standard_normal((n, L, D)), rng.standard_normal((n, L, D))
    perm = rng.permutation(L)
    a = oracle.attention(Q, K, V, 0.5)
    b = oracle.attention(Q, K[:, perm], V[:, perm], 0.5)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)


def test_matches_library_softmax_matmul():
    # reduces to a textbook routine: softmax(Q K^T s) V; distinct T, L, D catch transposes
    n, T, L, D = 3, 7, 19, 12
    g = torch.Generator().manual_seed(6)
    Q = torch.randn(n, T, D, generator=g, dtype=torch.float64)
    K = torch.randn(n, L, D, generator=g, dtype=torch.float64)
    V = torch.randn(n, L, D, generator=g, dtype=torch.float64)
    ref = torch.softmax(Q @ K.transpose(1, 2) * 0.37, dim=-1) @ V
    out = oracle.attention(Q.numpy(), K.numpy(), V.numpy(), 0.37)
    np.testing.assert_allclose(out, ref.numpy(), rtol=0, atol=1e-13)


def test_brute_force_python_loops_tiny():
    n, T, L, D = 1, 2, 3, 2
    Q = np.array([[[1.0, 2.0], [0.5, -1.0]]])
    K = np.array([[[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]]])
    V = np.array([[[1.0, 10.0], [2.0, 20.0], [3.0, 30.0]]])
    s = 0.5
    out = oracle.attention(Q, K, V, s)
    for q in range(T):
        z = [s * sum(Q[0, q, d] * K[0, j, d] for d in range(D)) for j in range(L)]
        e = [math.exp(v) for v in z]
        p = [v / sum(e) for v in e]
        for d in range(D):
            assert abs(out[0, q, d] - sum(p[j] * V[0, j, d] for j in range(L))) < 1e-14
    # hand value: query 0 logits are (0.5, 1.0, 1.5)
    e = [math.exp(0.5), math.exp(1.0), math.exp(1.5)]
    assert abs(out[0, 0, 0] - (e[0] * 1 + e[1] * 2 + e[2] * 3) / sum(e)) < 1e-14


def test_large_logits_do_not_overflow():
    n, T, L, D = 1, 3, 9, 4
    rng = np.random.default_rng(7)
    Q, K, V = rng.standard_normal((n, T, D)) * 200, rng.standard_normal((n, L, D)) * 200, rng.standard_normal((n, L, D))
    out = oracle.attention(Q, K, V, 1.0)
    assert np.isfinite(out).all()
    # argmax key dominates completely
    z = np.einsum("ntd,nld->ntl", Q, K)
    j = z.argmax(-1)
    np.testing.assert_allclose(out[0], V[0, j[0]], rtol=0, atol=1e-9)


def test_bf16_inputs_are_widened_exactly():
    q, k, v = synth.qkv_for_scale(2, 2, 9, 16, seed=11, scale=2)
    n = 4
    out = oracle.attention(q.reshape(n, 9, 16).double().numpy(), k.reshape(n, 9, 16).double().numpy(),
                           v.reshape(n, 9, 16).double().numpy(), 0.25)
    ref = torch.softmax(q.double().reshape(n, 9, 16) @ k.double().reshape(n, 9, 16).transpose(1, 2) * 0.25, -1) \
        @ v.double().reshape(n, 9, 16)
    np.testing.assert_allclose(out, ref.numpy(), rtol=0, atol=1e-14)


def test_attend_tokens_whole_segments_equals_attend_selected():
    """A token list made of whole segments is the kept-segment form, bit for bit."""
    n, D = 3, 8
    Q, K, V = _segments(n, D, 11)
    for keep in ([0, 1, 3, 4], [4], [0, 2, 4]):
        tokens = [(s, t) for s in keep for t in range(SIDES[s] ** 2)]
        a = oracle.attend_tokens(Q[4], K, V, tokens, 0.3)
        b = oracle.attend_selected(Q[4], K, V, keep, 0.3)
        np.testing.assert_array_equal(a, b)


def test_attend_tokens_partial_segments_equals_attention_on_hand_gathered_keys():
    """Part of a segment, a segment split in two runs, and an unsorted list: the keys are exactly the listed
    (segment, token) pairs, gathered here by hand one by one."""
    n, D = 2, 8
    Q, K, V = _segments(n, D, 12)
    tokens = [(0, 0), (1, 1), (1, 3), (3, 5), (3, 6), (3, 15), (2, 8), (4, 0), (4, 24), (3, 0)]
    Kc = np.stack([K[s][:, t, :] for s, t in tokens], axis=1)
    Vc = np.stack([V[s][:, t, :] for s, t in tokens], axis=1)
    want = oracle.attention(Q[4], Kc, Vc, 0.5)
    got = oracle.attend_tokens(Q[4], K, V, tokens, 0.5)
    np.testing.assert_array_equal(got, want)
    # and against the definition written out in Python for one query
    z = 0.5 * Kc[1] @ Q[4][1, 7]
    p = np.exp(z - z.max())
    p /= p.sum()
    np.testing.assert_allclose(got[1, 7], p @ Vc[1], rtol=0, atol=1e-13)
    # a wrong token would be seen: dropping one key changes the result
    other = oracle.attend_tokens(Q[4], K, V, tokens[:-1], 0.5)
    assert np.abs(other - got).max() > 1e-4
