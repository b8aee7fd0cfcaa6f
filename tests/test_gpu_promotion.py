"""GPU parity of a generation pass that follows Algorithm 1 on line: every layer starts cache-efficient; at the
scale where its cache first overflows, the similarity of that scale's keys to the previous scale's (Eq. 4)
is computed on the device and compared with theta, and the layer is promoted before the scale is appended."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

from gpu_common import Cache, check_close, to_items

pytestmark = pytest.mark.gpu

SIDES = synth.SIDES_256


@pytest.mark.parametrize("fused", [False, True], ids=["separate", "fused"])
def test_paper_budgets_promoted_on_line_from_the_similarity_of_the_overflowing_scale(fused):
    rows, heads, D = 2, 4, 64
    c_cds, c_min, c_max = 5, 174, 430                      # Sec. 5.1: condensed scales, + penultimate, + last two
    # layer 0: adjacent scales' keys share a smooth field (high similarity); layers 1 and 2: independent keys
    keys = [synth.smooth_field_keys(rows, heads, SIDES, D, 31 + l, rho, "cuda") for l, rho in enumerate((0.9, 0.0, 0.0))]
    qv = [synth.qkv_for_scale(rows, heads, s * s, D, 77, k, "cuda") for k, s in enumerate(SIDES)]
    pols = [(2, 2, False), (2, 2, False), (2, 2, B.LAYER_PROMOTABLE)]
    budgets = [(c_min, c_cds, c_max), (c_min, c_cds, c_max), (0, 0)]
    n_ws = B.amskv_similarity_workspace_bytes()
    ws = torch.empty(n_ws, dtype=torch.uint8, device="cuda")
    ss = torch.zeros(1, dtype=torch.float64, device="cuda")
    scale = 1.0 / math.sqrt(D)
    with Cache(3, heads, D, rows, SIDES, pols, token_budgets=budgets) as cache:
        first = [B.amskv_first_overflow_scale(cache.h, l) for l in range(3)]
        assert first == [7, 7, 4]
        # the score each layer will see at its overflow, from the oracle, and a threshold between the two kinds
        # (the size-normalised form -sqrt(ss / n): the layers overflow at scales of different sizes)
        n_at = [rows * heads * SIDES[first[l]] ** 2 * D for l in range(3)]
        want_s = [-math.sqrt(oracle.similarity_ss(to_items(keys[l][first[l] - 1]), SIDES[first[l] - 1],
                                                  to_items(keys[l][first[l]]), SIDES[first[l]]) / n_at[l]) for l in range(3)]
        theta = 0.5 * (want_s[0] + want_s[1])
        assert want_s[1] < theta < want_s[0]
        promoted = [False] * 3
        outs = {l: [] for l in range(3)}
        for k in range(len(SIDES)):
            for l in range(3):
                kk = keys[l][k]
                q, _, v = qv[k]
                if k == first[l]:
                    B.amskv_layer_similarity(keys[l][k - 1], SIDES[k - 1], kk, SIDES[k], rows, heads, D, ss, ws, n_ws)
                    torch.cuda.synchronize()
                    s_lib = -math.sqrt(float(ss.item()) / n_at[l])
                    assert abs(s_lib - want_s[l]) <= 1e-5 * abs(want_s[l])
                    # layer 2 (whole scales) is given layer 1's keys' verdict through its own keys: also independent
                    if B.amskv_classify_by_threshold([s_lib], theta)[0]:
                        B.amskv_promote_layer(cache.h, l)
                        promoted[l] = True
                o = torch.full_like(q, float("nan"))
                if fused:
                    B.amskv_append_attend(cache.h, l, k, kk, v, q, o)
                else:
                    B.amskv_append(cache.h, l, k, kk, v)
                    B.amskv_attend(cache.h, l, k, q, o)
                outs[l].append(o)
        torch.cuda.synchronize()
        assert B.amskv_status(cache.h) == 0
        assert promoted == oracle.classify_layers(want_s, theta) == [False, True, True]
        for l in range(3):
            Ks = [to_items(keys[l][k]) for k in range(len(SIDES))]
            Vs = [to_items(qv[k][2]) for k in range(len(SIDES))]
            outcome = [promoted[l]] * len(SIDES)
            for k in range(len(SIDES)):
                Q = to_items(qv[k][0])
                if l < 2:
                    tokens = oracle.attended_tokens(SIDES, k, c_min, c_cds, c_max=c_max, below_theta=outcome)
                    want = oracle.attend_tokens(Q, Ks, Vs, tokens, scale)
                else:
                    want = oracle.attend_selected(Q, Ks, Vs, oracle.keep_set(k, 2, 2, promoted[l] and k >= first[l]), scale)
                check_close(outs[l][k], want, "layer %d scale %d" % (l, k))
        assert B.amskv_kept_segments(cache.h, 0, 9) == [0, 1, 8] and B.amskv_kept_segments(cache.h, 1, 9) == [0, 1, 8, 9]
        assert B.amskv_kept_segments(cache.h, 2, 9) == list(range(10))
