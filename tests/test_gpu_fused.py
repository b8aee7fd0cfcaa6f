"""GPU parity of amskv_append_attend (the append fused into the paired attention kernel): same
outputs as the oracle at every scale -- later scales read what the fused calls wrote to the cache,
so a wrong or misplaced write shows up there -- and the same cache state as the two separate calls."""
import math

import pytest
import torch

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

from gpu_common import (Cache, check_close, make_qkv, oracle_outputs, run_pass, tensor_path_available, to_items)

pytestmark = pytest.mark.gpu


def _need(D=64):
    if not tensor_path_available(D):
        pytest.skip("tensor-core path not available")


@pytest.mark.parametrize("path", [B.PATH_AUTO, B.PATH_TENSOR_PAIR], ids=["auto", "pair"])
@pytest.mark.parametrize("fused", [True, (3, 5, 9), (0, 8)], ids=["all", "some", "ends"])
def test_single_layer_every_element_every_scale(path, fused):
    _need()
    wl = synth.WORKLOADS["single"]
    qkv = make_qkv(wl.rows, wl.heads, wl.sides, wl.head_dim, wl.seed)
    scale = 1.0 / math.sqrt(wl.head_dim)
    pols = [(2, 2, False), (2, 2, True), (0, 1, False), (1, 3, False)]
    with Cache(len(pols), wl.heads, wl.head_dim, wl.rows, wl.sides, pols) as c:
        outs = run_pass(c, qkv, path, fused=fused)
        for layer, pol in enumerate(pols):
            want = oracle_outputs(qkv, pol, scale)
            for k in range(len(wl.sides)):
                check_close(outs[layer][k], want[k], "layer %d scale %d" % (layer, k))
        assert B.amskv_cache_bytes(c.h)[1] == oracle.kv_bytes(wl.sides, pols, wl.rows, wl.heads, wl.head_dim)


@pytest.mark.parametrize("path", [B.PATH_TENSOR_PAIR, B.PATH_AUTO, B.PATH_SMALL], ids=["pair", "auto", "small"])
def test_cache_contents_equal_those_of_the_separate_calls(path):
    """Byte-for-byte: the arena after a fused pass equals the arena after append + attend."""
    _need()
    sides, rows, heads, D = (1, 2, 3, 5, 7, 9, 12, 17), 3, 5, 64
    qkv = make_qkv(rows, heads, sides, D, seed=41)
    pols = [(2, 2, False), (1, 1, False), (2, 2, True)]
    arenas = []
    for fused in (False, True):
        with Cache(len(pols), heads, D, rows, sides, pols) as c:
            c.arena.zero_()
            run_pass(c, qkv, path, fused=fused)
            arenas.append(c.arena[256:].clone())
    assert torch.equal(arenas[0], arenas[1])


@pytest.mark.parametrize("D", [64, 128])
def test_ragged_tiles_many_items_and_strided_inputs(D):
    """Key counts that end inside a 64-token tile and inside a 16-token box, an odd number of items,
    more units than CTAs, and K/V/Q handed over as strided views of a packed [rows, T, 3, heads, D] tensor."""
    _need(D)
    sides, rows, heads = (4, 7, 17), 10, 37
    g = torch.Generator(device="cuda").manual_seed(42)
    qkv = []
    for s in sides:
        packed = (torch.randn(rows, s * s, 3, heads, D, generator=g, device="cuda") / 8).to(torch.bfloat16)
        q, k, v = (packed[:, :, i].permute(0, 2, 1, 3) for i in range(3))
        qkv.append((q, k, v))
    pols = [(1, 1, False), (0, 2, False), (2, 2, True)]
    with Cache(len(pols), heads, D, rows, sides, pols) as c:
        outs = run_pass(c, qkv, B.PATH_TENSOR_PAIR, fused=True)
        scale = 1.0 / math.sqrt(D)
        for layer, pol in enumerate(pols):
            want = oracle_outputs(qkv, pol, scale)
            for k in range(len(sides)):
                check_close(outs[layer][k], want[k], "D %d layer %d scale %d" % (D, layer, k))


@pytest.mark.parametrize("D", [64, 128])
def test_left_over_cache_tokens_ride_in_the_spare_box_of_the_last_tile(D):
    """5 condensed tokens behind a 64-token scale would be a key tile of their own; with a 100-token current
    scale (last tile 36 tokens) they are loaded into that tile's fourth 16-token box instead.  Also a
    one-token and a 16-token remainder, and an odd number of items (a unit with a single stream)."""
    _need(D)
    for sides, pols in [((1, 2, 8, 10), [(2, 2, False)]), ((1, 6), [(1, 1, False), (2, 2, True)]), ((4, 8, 5), [(1, 2, False)])]:
        rows, heads = 3, 5
        qkv = make_qkv(rows, heads, sides, D, seed=46 + len(sides))
        scale = 1.0 / math.sqrt(D)
        for path in (B.PATH_AUTO, B.PATH_TENSOR_PAIR):
            with Cache(len(pols), heads, D, rows, sides, pols) as c:
                outs = run_pass(c, qkv, path, fused=True)
                for layer, pol in enumerate(pols):
                    want = oracle_outputs(qkv, pol, scale)
                    for k in range(len(sides)):
                        check_close(outs[layer][k], want[k], "sides %s layer %d scale %d" % (sides, layer, k))


def test_token_budgets_fused():
    """Under token budgets the fused path takes the appends that are one copy; the rest run as two calls."""
    _need()
    sides, rows, heads, D = (1, 2, 3, 4, 5, 6, 8, 10), 2, 6, 64
    budgets = [(500, 5), (100, 5), (70, 0), (13, 3), (64, 14), (120, 5)]
    qkv = make_qkv(rows, heads, sides, D, seed=43)
    scale = 1.0 / math.sqrt(D)
    Ks = [to_items(k) for _, k, _ in qkv]
    Vs = [to_items(v) for _, _, v in qkv]
    with Cache(len(budgets), heads, D, rows, sides, [(2, 2, False)] * len(budgets), token_budgets=budgets) as cache:
        outs = run_pass(cache, qkv, B.PATH_TENSOR_PAIR, fused=True)
        for layer, (b, c) in enumerate(budgets):
            for k, (q, _, _) in enumerate(qkv):
                want = oracle.attend_tokens(to_items(q), Ks, Vs, oracle.attended_tokens(sides, k, b, c), scale)
                check_close(outs[layer][k], want, "budget %d/%d scale %d" % (b, c, k))


def test_var_d30_shape_sampled_fused():
    """The VAR-d30 head layout at 128 rows (more units than CTAs at every scale), sampled items."""
    _need()
    wl = synth.WORKLOADS["var_d30"].replace(batch=64)
    pols = [(2, 2, False), (2, 2, True)]
    qkv = make_qkv(wl.rows, wl.heads, wl.sides, wl.head_dim, wl.seed)
    items = wl.rows * wl.heads
    g = torch.Generator().manual_seed(44)
    sample = sorted(set([0, 1, items - 2, items - 1] + torch.randint(0, items, (28,), generator=g).tolist()))
    idx = torch.tensor(sample, device="cuda")

    def pick(x):
        r, h, t, d = x.shape
        return x.reshape(r * h, t, d)[idx]

    scale = 1.0 / math.sqrt(wl.head_dim)
    with Cache(2, wl.heads, wl.head_dim, wl.rows, wl.sides, pols) as cache:
        outs = run_pass(cache, qkv, fused=True)
        Ks = [pick(k).cpu().double().numpy() for _, k, _ in qkv]
        Vs = [pick(v).cpu().double().numpy() for _, _, v in qkv]
        for k, (q, _, _) in enumerate(qkv):
            Qs = pick(q).cpu().double().numpy()
            for layer, (c, w, dem) in enumerate(pols):
                want = oracle.attend_selected(Qs, Ks, Vs, oracle.keep_set(k, c, w, dem), scale)
                check_close(pick(outs[layer][k]).cpu().double(), want, "layer %d scale %d" % (layer, k))


def test_order_contract():
    _need()
    sides, rows, heads, D = (2, 9), 1, 2, 64
    qkv = make_qkv(rows, heads, sides, D, seed=45)
    with Cache(1, heads, D, rows, sides, [(2, 2, False)]) as c:
        q, k, v = qkv[1]
        o = torch.empty_like(q)
        assert B.lib.amskv_append_attend(c.h, 0, 1, k.data_ptr(), v.data_ptr(), None, q.data_ptr(), o.data_ptr(),
                                         None, None, None) == B.ERR_ORDER
        q, k, v = qkv[0]
        o = torch.empty_like(q)
        B.amskv_append_attend(c.h, 0, 0, k, v, q, o)
        assert B.lib.amskv_append_attend(c.h, 0, 0, k.data_ptr(), v.data_ptr(), None, q.data_ptr(), o.data_ptr(),
                                         None, None, None) == B.ERR_ORDER
        torch.cuda.synchronize()
        assert B.amskv_status(c.h) == 0
