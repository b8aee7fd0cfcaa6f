"""GPU parity: amskv_attention_density through the C ABI against the oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

from gpu_common import Cache, make_qkv, to_items

pytestmark = pytest.mark.gpu


def _density(cache, layer, k, q, heads):
    runs = B.amskv_attended_tokens(cache.h, layer, k)
    out = torch.full((heads, len(runs)), float("nan"), dtype=torch.float64, device="cuda")
    B.amskv_attention_density(cache.h, layer, k, q, out, out.numel())
    torch.cuda.synchronize()
    return runs, out.cpu().numpy()


@pytest.mark.parametrize("D", [64, 128])
def test_matches_oracle_for_whole_scales_and_token_budgets(D):
    sides, rows, heads = (1, 2, 3, 4, 5, 6, 8), 3, 5
    qkv = make_qkv(rows, heads, sides, D, seed=61, peaked=(D == 64))
    pols = [(2, 2, False), (2, 2, True), (1, 3, False), (2, 2, False), (2, 2, False)]
    budgets = [(0, 0), (0, 0), (0, 0), (40, 5), (13, 3)]
    scale = 1.0 / math.sqrt(D)
    Ks = [to_items(k) for _, k, _ in qkv]
    with Cache(len(pols), heads, D, rows, sides, pols, token_budgets=budgets) as c:
        for k, (q, kk, v) in enumerate(qkv):
            for layer in range(len(pols)):
                B.amskv_append(c.h, layer, k, kk, v)
                runs, got = _density(c, layer, k, q, heads)
                want = oracle.attention_density(to_items(q), Ks, runs, scale, heads)
                assert np.allclose(got, want, rtol=2e-4, atol=1e-7), (layer, k, np.abs(got - want).max())
                counts = np.array([n for _, _, n in runs], dtype=np.float64)
                assert np.allclose(got @ counts, sides[k] ** 2, rtol=1e-5)
        assert B.amskv_status(c.h) == 0


def test_order_and_argument_errors():
    sides, rows, heads, D = (2, 3), 1, 2, 64
    qkv = make_qkv(rows, heads, sides, D, seed=62)
    with Cache(1, heads, D, rows, sides, [(2, 2, False)]) as c:
        q, k, v = qkv[0]
        out = torch.zeros(heads * 2, dtype=torch.float64, device="cuda")
        f = B.lib.amskv_attention_density
        assert f(c.h, 0, 0, q.data_ptr(), None, out.data_ptr(), out.numel(), None) == B.ERR_ORDER
        B.amskv_append(c.h, 0, 0, k, v)
        assert f(c.h, 0, 0, q.data_ptr(), None, out.data_ptr(), 1, None) == B.ERR_NOMEM
        assert f(c.h, 0, 0, q.data_ptr(), None, None, out.numel(), None) == B.ERR_INVALID
        assert f(c.h, 0, 0, q.data_ptr(), None, out.data_ptr(), out.numel(), None) == B.OK
    with Cache(1, heads, D, rows, sides, [(2, 2, False)], flags=B.FLAG_TRANSIENT_LAST_SCALE) as c:
        for kk, (q, k, v) in enumerate(qkv):
            o = torch.empty_like(q)
            B.amskv_append_attend(c.h, 0, kk, k, v, q, o)
        out = torch.zeros(heads * 2, dtype=torch.float64, device="cuda")
        assert B.lib.amskv_attention_density(c.h, 0, 1, q.data_ptr(), None, out.data_ptr(), out.numel(), None) == B.ERR_UNSUPPORTED
        torch.cuda.synchronize()


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("peaked", [False, True], ids=["flat", "peaked"])
def test_density_as_a_by_product_of_the_attention_launch(D, peaked):
    """amskv_attend_density: the output equals amskv_attend's bit for bit where both run the paired kernel on
    the same tiles (and the oracle everywhere), and the density equals the oracle's -- whole scales and token
    budgets, more units than CTAs, query tiles with idle warps, rows whose reference maximum moves (peaked)."""
    from gpu_common import check_close, oracle_outputs
    sides, rows, heads = (1, 2, 3, 5, 6, 8, 13), 6, 40
    qkv = make_qkv(rows, heads, sides, D, seed=63, peaked=peaked)
    pols = [(2, 2, False), (2, 2, True), (1, 3, False), (2, 2, False)]
    budgets = [(0, 0), (0, 0), (0, 0), (120, 5)]
    scale = 1.0 / math.sqrt(D)
    Ks = [to_items(k) for _, k, _ in qkv]
    Vs = [to_items(v) for _, _, v in qkv]
    with Cache(len(pols), heads, D, rows, sides, pols, token_budgets=budgets) as c:
        for k, (q, kk, v) in enumerate(qkv):
            for layer in range(len(pols)):
                B.amskv_append(c.h, layer, k, kk, v)
                runs = B.amskv_attended_tokens(c.h, layer, k)
                den = torch.full((heads, len(runs)), float("nan"), dtype=torch.float64, device="cuda")
                out = torch.full_like(q, float("nan"))
                B.amskv_attend_density(c.h, layer, k, q, out, den, den.numel())
                torch.cuda.synchronize()
                tokens = [(s, t) for s, first, count in runs for t in range(first, first + count)]
                want_out = oracle.attend_tokens(to_items(q), Ks, Vs, tokens, scale)
                check_close(out, want_out, "output, layer %d scale %d" % (layer, k), max_abs=4e-2 if peaked else 1e-2)
                want = oracle.attention_density(to_items(q), Ks, runs, scale, heads)
                got = den.cpu().numpy()
                assert np.allclose(got, want, rtol=2e-4, atol=1e-7), (layer, k, np.abs(got / want - 1).max())
                counts = np.array([n for _, _, n in runs], dtype=np.float64)
                assert np.allclose(got @ counts, sides[k] ** 2, rtol=1e-4)
        assert B.amskv_status(c.h) == 0
