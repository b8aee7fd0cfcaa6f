"""AMS-KV oracle: slow fp64 CPU definitions used only to check the CUDA library.

TEST INFRASTRUCTURE ONLY.  Importers allowed: the tests, the smoke check and the
benchmark's CPU-baseline / reference arm.  The product package never imports this, and
this package imports nothing from the product.

Arithmetic lives in `amskv_oracle.c` (fp64, OpenMP over items) and is reached through
ctypes; selection (integers) lives in `selection.py`.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Sequence

import numpy as np

from .selection import (algorithm1_tokens, algorithm1_trace, attended_tokens, clru_tokens, evicted_at,  # noqa: F401
                        keep_set, keep_set_simulated, kept_tokens, kv_bytes)

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "amskv_oracle.c")
_LIB = os.path.join(_HERE, "libamskv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C part with gcc (fp64, OpenMP, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int)
        lib.amskv_oracle_threads.restype = ctypes.c_int
        lib.amskv_oracle_attention.argtypes = [dp, dp, dp, dp, ctypes.c_long, ctypes.c_long,
                                               ctypes.c_long, ctypes.c_long, ctypes.c_double]
        lib.amskv_oracle_attention.restype = None
        lib.amskv_oracle_block_causal_attention.argtypes = [dp, dp, dp, dp, ip, ctypes.c_long,
                                                            ctypes.c_long, ctypes.c_long,
                                                            ctypes.c_double]
        lib.amskv_oracle_block_causal_attention.restype = None
        lib.amskv_oracle_bilinear_resize.argtypes = [dp, ctypes.c_long, dp, ctypes.c_long,
                                                     ctypes.c_long, ctypes.c_long]
        lib.amskv_oracle_bilinear_resize.restype = None
        lib.amskv_oracle_similarity_ss.argtypes = [dp, ctypes.c_long, dp, ctypes.c_long,
                                                   ctypes.c_long, ctypes.c_long]
        lib.amskv_oracle_similarity_ss.restype = ctypes.c_double
        _lib = lib
    return _lib


def threads() -> int:
    """Host threads the C part uses (OpenMP max threads)."""
    return int(_load().amskv_oracle_threads())


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def attention(Q, K, V, scale: float) -> np.ndarray:
    """softmax(scale * Q K^T) V per item.  Q: [n, T, D]; K, V: [n, L, D] -> [n, T, D] fp64."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    n, T, D = Q.shape
    L = K.shape[1]
    assert K.shape == (n, L, D) and V.shape == (n, L, D) and L >= 1
    out = np.empty_like(Q)
    _load().amskv_oracle_attention(_ptr(Q), _ptr(K), _ptr(V), _ptr(out), n, T, L, D, float(scale))
    return out


def attend_selected(Q, K_segments: Sequence, V_segments: Sequence, keep: Sequence[int],
                    scale: float) -> np.ndarray:
    """Scale-adaptive attention: queries attend to exactly the kept segments.

    K_segments[s], V_segments[s]: [n, T_s, D] for every scale s that is available; `keep`
    lists the segment ids the policy retains (the current scale included).  The kept keys
    are gathered in ascending scale order and attended without any mask.
    """
    Kc = np.concatenate([_f64(K_segments[s]) for s in keep], axis=1)
    Vc = np.concatenate([_f64(V_segments[s]) for s in keep], axis=1)
    return attention(Q, Kc, Vc, scale)


def attend_tokens(Q, K_segments: Sequence, V_segments: Sequence, tokens: Sequence, scale: float) -> np.ndarray:
    """Attention of Q over an explicit list of (segment, token) keys (token budgets may keep part
    of a segment).  K_segments[s], V_segments[s]: [n, T_s, D]."""
    tokens = list(tokens)
    k_parts, v_parts = [], []
    i = 0
    while i < len(tokens):  # gather run by run of equal segment id, in list order
        s = tokens[i][0]
        j = i
        while j < len(tokens) and tokens[j][0] == s:
            j += 1
        idx = [t for _, t in tokens[i:j]]
        k_parts.append(_f64(K_segments[s])[:, idx, :])
        v_parts.append(_f64(V_segments[s])[:, idx, :])
        i = j
    return attention(Q, np.concatenate(k_parts, axis=1), np.concatenate(v_parts, axis=1), scale)


def attention_density(Q, K_segments: Sequence, runs: Sequence, scale: float, heads: int) -> np.ndarray:
    """Attention density (Sec. 4.1) of the queries Q over runs of retained keys.

    Q: [n, T, D] with n = rows * heads (item = row * heads + head); K_segments[s]: [n, T_s, D];
    runs: (segment, first token, count) triples.  P = softmax(scale * Q Kc^T) over the concatenated
    keys of all runs; the density of a run is the sum of P over all queries and over the run's keys,
    divided by the run's token count; the result [heads, len(runs)] is the mean over rows.
    """
    Q = _f64(Q)
    n, T, D = Q.shape
    Kc = np.concatenate([_f64(K_segments[s])[:, first:first + count, :] for s, first, count in runs], axis=1)
    logits = scale * np.einsum("ntd,nld->ntl", Q, Kc)
    logits -= logits.max(axis=2, keepdims=True)
    P = np.exp(logits)
    P /= P.sum(axis=2, keepdims=True)
    out = np.zeros((heads, len(runs)), dtype=np.float64)
    rows = n // heads
    at = 0
    for r, (_, _, count) in enumerate(runs):
        mass = P[:, :, at:at + count].sum(axis=(1, 2)) / count      # per item
        out[:, r] = mass.reshape(rows, heads).mean(axis=0)
        at += count
    return out


def block_causal_attention(Q_all, K_all, V_all, sides: Sequence[int], scale: float) -> np.ndarray:
    """Vanilla next-scale attention over all tokens at once with the scale-block mask."""
    Q_all, K_all, V_all = _f64(Q_all), _f64(K_all), _f64(V_all)
    n, N, D = Q_all.shape
    scale_of = np.concatenate([np.full(int(s) * int(s), i, dtype=np.int32)
                               for i, s in enumerate(sides)])
    assert scale_of.shape[0] == N
    scale_of = np.ascontiguousarray(scale_of)
    out = np.empty_like(Q_all)
    _load().amskv_oracle_block_causal_attention(
        _ptr(Q_all), _ptr(K_all), _ptr(V_all), _ptr(out),
        scale_of.ctypes.data_as(ctypes.POINTER(ctypes.c_int)), n, N, D, float(scale))
    return out


def bilinear_resize(src, s_in: int, s_out: int) -> np.ndarray:
    """Resize [n, s_in^2, D] token maps to [n, s_out^2, D] (bilinear, half-pixel, clamped)."""
    src = _f64(src)
    n, t, D = src.shape
    assert t == s_in * s_in
    dst = np.empty((n, s_out * s_out, D), dtype=np.float64)
    _load().amskv_oracle_bilinear_resize(_ptr(src), s_in, _ptr(dst), s_out, n, D)
    return dst


def similarity_ss(K_prev, s_prev: int, K_cur, s_cur: int) -> float:
    """Sum of squares of (K_cur - resize(K_prev)); Eq. 4 is S = -sqrt of this."""
    K_prev, K_cur = _f64(K_prev), _f64(K_cur)
    n, tp, D = K_prev.shape
    assert tp == s_prev * s_prev and K_cur.shape == (n, s_cur * s_cur, D)
    return float(_load().amskv_oracle_similarity_ss(_ptr(K_prev), s_prev, _ptr(K_cur), s_cur, n, D))


def similarity(K_prev, s_prev: int, K_cur, s_cur: int) -> float:
    """Eq. 4: S(k_i, k-hat_{i-1}) = -|| k_i - k-hat_{i-1} ||_2 over all items/tokens/channels.

    The arithmetic of this reading (bilinear resize, half-pixel centres, edge clamp, plain L2 norm) is
    pinned by the tests.  Parity unpinned: the paper's threshold values (around -0.01, Appendix E) imply
    a normalisation of the norm that the text does not state, and its per-layer values exist only as a
    figure, so nothing ties the magnitude of this score to the paper's."""
    return -float(np.sqrt(similarity_ss(K_prev, s_prev, K_cur, s_cur)))


def classify_layers(scores: Sequence[float], theta: float) -> List[bool]:
    """A layer is cache-demanding iff its similarity is strictly below theta (Algorithm 1)."""
    return [bool(s < theta) for s in scores]


def lowest_similarity_layers(scores: Sequence[float], n_demanding: int) -> List[bool]:
    """Similarity-aware allocation (S2): the n lowest-similarity layers are cache-demanding;
    ties go to the lower layer index."""
    order = sorted(range(len(scores)), key=lambda i: (scores[i], i))
    chosen = set(order[:n_demanding])
    return [i in chosen for i in range(len(scores))]
