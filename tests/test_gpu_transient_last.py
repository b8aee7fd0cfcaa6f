"""GPU parity with AMSKV_FLAG_TRANSIENT_LAST_SCALE: the last scale is attended straight from the
caller's K and V and never stored; every output must equal the oracle's, as without the flag."""
import math

import pytest
import torch

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

from gpu_common import Cache, check_close, make_qkv, oracle_outputs, run_pass, tensor_path_available, to_items

pytestmark = pytest.mark.gpu

FLAG = B.FLAG_TRANSIENT_LAST_SCALE
PATHS = {"auto": B.PATH_AUTO, "pair": B.PATH_TENSOR_PAIR, "simt": B.PATH_SIMT, "small": B.PATH_SMALL}


def _need(path, D=64):
    if path != B.PATH_SIMT and not tensor_path_available(D):
        pytest.skip("tensor-core path not available")


@pytest.mark.parametrize("path", list(PATHS), ids=list(PATHS))
def test_every_element_every_scale(path):
    _need(PATHS[path])
    wl = synth.WORKLOADS["single"]
    qkv = make_qkv(wl.rows, wl.heads, wl.sides, wl.head_dim, wl.seed)
    scale = 1.0 / math.sqrt(wl.head_dim)
    pols = [(2, 2, False), (2, 2, True), (0, 1, False), (1, 3, False)]
    with Cache(len(pols), wl.heads, wl.head_dim, wl.rows, wl.sides, pols, flags=FLAG) as c:
        per_token = 2 * 2 * wl.rows * wl.heads * wl.head_dim
        assert B.amskv_cache_required_bytes(c.desc) == 256 + (274 + 424 + 169 + 334) * per_token
        outs = run_pass(c, qkv, PATHS[path], fused=True)
        for layer, pol in enumerate(pols):
            want = oracle_outputs(qkv, pol, scale)
            for k in range(len(wl.sides)):
                check_close(outs[layer][k], want[k], "layer %d scale %d" % (layer, k))


@pytest.mark.parametrize("D", [64, 128])
def test_short_schedules_and_token_budgets(D):
    """A single-scale schedule (nothing is ever stored), a last scale of one token, ragged key counts,
    strided inputs, and token budgets beside whole-scale layers."""
    _need(B.PATH_AUTO, D)
    for sides in [(5,), (3, 1), (2, 9, 17)]:
        rows, heads = 3, 5
        g = torch.Generator(device="cuda").manual_seed(51 + len(sides))
        qkv = []
        for s in sides:
            packed = (torch.randn(rows, s * s, 3, heads, D, generator=g, device="cuda") / 8).to(torch.bfloat16)
            qkv.append(tuple(packed[:, :, i].permute(0, 2, 1, 3) for i in range(3)))
        pols = [(1, 1, False), (2, 2, True), (2, 2, False)]
        budgets = [(0, 0), (0, 0), (90, 4)]
        scale = 1.0 / math.sqrt(D)
        Ks = [to_items(k) for _, k, _ in qkv]
        Vs = [to_items(v) for _, _, v in qkv]
        for path in (B.PATH_AUTO, B.PATH_SIMT):
            with Cache(len(pols), heads, D, rows, sides, pols, flags=FLAG, token_budgets=budgets) as c:
                outs = run_pass(c, qkv, path, fused=True)
                for layer in (0, 1):
                    want = oracle_outputs(qkv, pols[layer], scale)
                    for k in range(len(sides)):
                        check_close(outs[layer][k], want[k], "sides %s layer %d scale %d" % (sides, layer, k))
                for k, (q, _, _) in enumerate(qkv):
                    want = oracle.attend_tokens(to_items(q), Ks, Vs, oracle.attended_tokens(sides, k, 90, 4), scale)
                    check_close(outs[2][k], want, "sides %s token budget scale %d" % (sides, k))


def test_append_refuses_the_last_scale():
    _need(B.PATH_AUTO)
    sides, rows, heads, D = (2, 3), 1, 2, 64
    qkv = make_qkv(rows, heads, sides, D, seed=52)
    with Cache(1, heads, D, rows, sides, [(2, 2, False)], flags=FLAG) as c:
        q, k, v = qkv[0]
        B.amskv_append(c.h, 0, 0, k, v)
        q, k, v = qkv[1]
        assert B.lib.amskv_append(c.h, 0, 1, k.data_ptr(), v.data_ptr(), None, None) == B.ERR_UNSUPPORTED
        o = torch.empty_like(q)
        B.amskv_append_attend(c.h, 0, 1, k, v, q, o)
        torch.cuda.synchronize()
        assert B.amskv_status(c.h) == 0
        want = oracle_outputs(qkv, (2, 2, False), 1.0 / math.sqrt(D))
        check_close(o, want[1], "last scale")
