"""GPU parity: amskv_append + amskv_attend through the C ABI against the fp64 oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

from gpu_common import (Cache, check_close, make_qkv, oracle_outputs, run_pass, tensor_path_available, to_items)

pytestmark = pytest.mark.gpu

PATHS = [B.PATH_SIMT, B.PATH_AUTO, B.PATH_TENSOR, B.PATH_TENSOR_PAIR, B.PATH_SMALL]
PATH_NAMES = {B.PATH_SIMT: "simt", B.PATH_AUTO: "auto", B.PATH_TENSOR: "tensor", B.PATH_TENSOR_PAIR: "pair", B.PATH_SMALL: "small"}


def _need(path, head_dim=64):
    if path in (B.PATH_TENSOR, B.PATH_TENSOR_PAIR, B.PATH_SMALL) and not tensor_path_available(head_dim):
        pytest.skip("tensor-core path not available for head_dim %d" % head_dim)


@pytest.mark.parametrize("path", PATHS, ids=lambda p: PATH_NAMES[p])
def test_single_layer_every_element_every_scale(path):
    """Single layer, 2 rows x 16 heads x 64, the 680-token schedule, condensed 2 / local 2."""
    _need(path)
    wl = synth.WORKLOADS["single"]
    qkv = make_qkv(wl.rows, wl.heads, wl.sides, wl.head_dim, wl.seed)
    scale = 1.0 / math.sqrt(wl.head_dim)
    pols = [(2, 2, False), (2, 2, True)]
    with Cache(2, wl.heads, wl.head_dim, wl.rows, wl.sides, pols) as c:
        outs = run_pass(c, qkv, path)
        for layer, pol in enumerate(pols):
            want = oracle_outputs(qkv, pol, scale)
            for k in range(len(wl.sides)):
                check_close(outs[layer][k], want[k], "layer %d scale %d" % (layer, k))
        # full retention is vanilla next-scale attention: compare with the one-shot masked form
        Qa = np.concatenate([to_items(q) for q, _, _ in qkv], 1)
        Ka = np.concatenate([to_items(k) for _, k, _ in qkv], 1)
        Va = np.concatenate([to_items(v) for _, _, v in qkv], 1)
        van = oracle.block_causal_attention(Qa, Ka, Va, wl.sides, scale)
        got = np.concatenate([to_items(o) for o in outs[1]], 1)
        check_close(torch.from_numpy(got), van, "full retention vs vanilla")


@pytest.mark.parametrize("path", PATHS, ids=lambda p: PATH_NAMES[p])
@pytest.mark.parametrize("c,w", [(0, 1), (1, 1), (2, 1), (0, 3), (1, 3), (3, 2), (2, 4), (9, 9)])
def test_policy_sweep_small(path, c, w):
    _need(path)
    sides = (1, 2, 3, 4, 5, 6, 8, 10)
    rows, heads, D = 2, 3, 64
    qkv = make_qkv(rows, heads, sides, D, seed=100 + 7 * c + w)
    with Cache(1, heads, D, rows, sides, [(c, w, False)]) as cache:
        outs = run_pass(cache, qkv, path)
        want = oracle_outputs(qkv, (c, w, False), 1.0 / math.sqrt(D))
        for k in range(len(sides)):
            check_close(outs[0][k], want[k], "c=%d w=%d scale %d" % (c, w, k))
            assert B.amskv_kept_segments(cache.h, 0, k) == oracle.keep_set(k, c, w, False)


@pytest.mark.parametrize("path", PATHS, ids=lambda p: PATH_NAMES[p])
def test_closed_form_properties(path):
    _need(path)
    sides = (1, 2, 4, 7, 12)
    rows, heads, D = 2, 2, 64
    qkv = make_qkv(rows, heads, sides, D, seed=5)
    # (a) values all one -> every output is one (softmax rows sum to one)
    ones = [(q, k, torch.ones_like(v)) for q, k, v in qkv]
    # (b) queries all zero -> output is the mean of the kept values
    zeros = [(torch.zeros_like(q), k, v) for q, k, v in qkv]
    with Cache(1, heads, D, rows, sides, [(1, 2, False)]) as cache:
        outs = run_pass(cache, ones, path)
        for k, o in enumerate(outs[0]):
            assert torch.allclose(o.float(), torch.ones_like(o, dtype=torch.float32), atol=4e-3), k
        outs = run_pass(cache, zeros, path)
        for k, o in enumerate(outs[0]):
            keep = oracle.keep_set(k, 1, 2, False)
            mean = np.concatenate([to_items(qkv[s][2]) for s in keep], 1).mean(axis=1, keepdims=True)
            check_close(o, np.broadcast_to(mean, to_items(o).shape), "mean of kept values, scale %d" % k)
        # (c) scale 0 has a single key: the output is that key's value, bit for bit
        outs = run_pass(cache, qkv, path)
        assert torch.equal(outs[0][0], qkv[0][2])


@pytest.mark.parametrize("path", PATHS, ids=lambda p: PATH_NAMES[p])
def test_peaked_softmax_rows(path):
    """Logit spread of several units, so the running maximum of the tiled softmax moves."""
    _need(path)
    sides = (2, 5, 9, 14)
    rows, heads, D = 1, 4, 64
    qkv = make_qkv(rows, heads, sides, D, seed=8, peaked=True)
    with Cache(1, heads, D, rows, sides, [(1, 2, True)]) as cache:
        outs = run_pass(cache, qkv, path)
        want = oracle_outputs(qkv, (1, 2, True), 1.0 / math.sqrt(D))
        for k in range(len(sides)):
            # outputs are O(1) here, so the absolute bound scales with them
            check_close(outs[0][k], want[k], "peaked scale %d" % k, max_abs=4e-2, rel_fro=REL)


REL = 5e-3


@pytest.mark.parametrize("path", PATHS, ids=lambda p: PATH_NAMES[p])
def test_head_dim_128_and_custom_scale(path):
    _need(path, 128)
    sides = (1, 2, 4, 6, 8, 12)
    rows, heads, D = 2, 2, 128
    qkv = make_qkv(rows, heads, sides, D, seed=21)
    with Cache(2, heads, D, rows, sides, [(3, 2, False), (3, 2, True)], softmax_scale=0.2) as cache:
        outs = run_pass(cache, qkv, path)
        for layer, pol in enumerate(cache.policies):
            want = oracle_outputs(qkv, pol, 0.2)
            for k in range(len(sides)):
                check_close(outs[layer][k], want[k], "D=128 layer %d scale %d" % (layer, k))


@pytest.mark.parametrize("path", PATHS, ids=lambda p: PATH_NAMES[p])
def test_strided_inputs_and_library_owned_arena(path):
    _need(path)
    sides = (1, 3, 6, 9)
    rows, heads, D = 2, 4, 64
    qkv = make_qkv(rows, heads, sides, D, seed=33)
    # token-major storage [rows, T, heads, D] viewed as [rows, heads, T, D]
    strided = []
    for q, k, v in qkv:
        strided.append(tuple(t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for t in (q, k, v)))
        assert not strided[-1][0].is_contiguous() or q.shape[2] == 1 or heads == 1
    with Cache(1, heads, D, rows, sides, [(1, 2, False)], own_arena=False) as cache:
        B.amskv_set_attend_path(cache.h, path)
        want = oracle_outputs(qkv, (1, 2, False), 1.0 / math.sqrt(D))
        for k, (q, kk, v) in enumerate(strided):
            B.amskv_append(cache.h, 0, k, kk, v)
            o = torch.full_like(q, float("nan"))          # keeps q's strides
            B.amskv_attend(cache.h, 0, k, q, o)
            torch.cuda.synchronize()
            check_close(o, want[k], "strided scale %d" % k)
        assert B.amskv_status(cache.h) == 0


@pytest.mark.parametrize("path", PATHS, ids=lambda p: PATH_NAMES[p])
def test_rerun_is_bitwise_reproducible_and_reset_works(path):
    _need(path)
    sides = (1, 2, 3, 4, 5, 6, 8)
    qkv = make_qkv(2, 2, sides, 64, seed=44)
    with Cache(1, 2, 64, 2, sides, [(2, 2, False)]) as cache:
        a = run_pass(cache, qkv, path)
        b = run_pass(cache, qkv, path)
        for x, y in zip(a[0], b[0]):
            assert torch.equal(x, y)


def test_tensor_and_simt_paths_agree():
    _need(B.PATH_TENSOR)
    wl = synth.WORKLOADS["single"]
    qkv = make_qkv(wl.rows, wl.heads, wl.sides, wl.head_dim, wl.seed + 1)
    with Cache(1, wl.heads, wl.head_dim, wl.rows, wl.sides, [(2, 2, False)]) as cache:
        a = run_pass(cache, qkv, B.PATH_SIMT)
        b = run_pass(cache, qkv, B.PATH_TENSOR)
        for k, (x, y) in enumerate(zip(a[0], b[0])):
            check_close(y, to_items(x), "tensor vs simt scale %d" % k)


def test_order_errors_on_device_cache():
    with Cache(1, 2, 64, 2, (1, 2, 3), [(1, 1, False)]) as cache:
        q, k, v = synth.qkv_for_scale(2, 2, 1, 64, 1, 0, "cuda")
        o = torch.empty_like(q)
        assert B.lib.amskv_attend(cache.h, 0, 0, q.data_ptr(), o.data_ptr(), None, None, None) == B.ERR_ORDER
        B.amskv_append(cache.h, 0, 0, k, v)
        B.amskv_attend(cache.h, 0, 0, q, o)
        assert B.lib.amskv_attend(cache.h, 0, 1, q.data_ptr(), o.data_ptr(), None, None, None) == B.ERR_ORDER
        assert B.lib.amskv_append(cache.h, 0, 0, k.data_ptr(), v.data_ptr(), None, None) == B.ERR_ORDER
        assert B.lib.amskv_append(cache.h, 0, 1, k.data_ptr() + 2, v.data_ptr(), None, None) == B.ERR_INVALID
        assert B.lib.amskv_append(cache.h, 0, 1, None, v.data_ptr(), None, None) == B.ERR_INVALID
        torch.cuda.synchronize()
    # an arena that is too small is refused
    d, keep = B.make_desc(1, 2, 64, 2, (1, 2, 3), [(1, 1, False)])
    small = torch.empty(512, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.AmskvError) as e:
        B.amskv_cache_create(d, small, 512)
    assert e.value.code == B.ERR_NOMEM


def test_step_host_matches_device_calls():
    sides = (1, 2, 4, 6)
    rows, heads, D = 2, 3, 64
    qkv = make_qkv(rows, heads, sides, D, seed=55, device="cpu")
    with Cache(1, heads, D, rows, sides, [(1, 2, False)]) as cache:
        nbytes = B.amskv_step_staging_bytes(cache.h)
        staging = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        want = oracle_outputs(qkv, (1, 2, False), 1.0 / math.sqrt(D))
        for k, (q, kk, v) in enumerate(qkv):
            hq, hk, hv = (t.pin_memory() for t in (q, kk, v))
            ho = torch.empty_like(hq).pin_memory()
            B.amskv_step_host(cache.h, 0, k, hk, hv, hq, ho, staging, nbytes)
            torch.cuda.synchronize()
            check_close(ho, want[k], "step_host scale %d" % k)


@pytest.mark.parametrize("path", [B.PATH_AUTO, B.PATH_TENSOR, B.PATH_TENSOR_PAIR], ids=lambda p: PATH_NAMES[p])
def test_many_units_per_cta_with_partly_idle_query_tiles(path):
    """More work units than resident CTAs, and query tiles whose upper warps have no rows
    (169 = 128 + 41 queries), so persistent CTAs walk several units each."""
    _need(path)
    sides = (2, 5, 13)
    rows, heads, D = 10, 70, 64
    qkv = make_qkv(rows, heads, sides, D, seed=91)
    with Cache(2, heads, D, rows, sides, [(1, 1, False), (1, 1, True)]) as cache:
        outs = run_pass(cache, qkv, path)
        for layer, pol in enumerate(cache.policies):
            want = oracle_outputs(qkv, pol, 1.0 / math.sqrt(D))
            for k in range(len(sides)):
                check_close(outs[layer][k], want[k], "layer %d scale %d" % (layer, k))


@pytest.mark.parametrize("path", [B.PATH_AUTO, B.PATH_TENSOR, B.PATH_TENSOR_PAIR], ids=lambda p: PATH_NAMES[p])
@pytest.mark.parametrize("D", [64, 128])
def test_odd_number_of_query_tiles_and_many_key_tiles(path, D):
    """289 = 2 * 128 + 33 query tokens: three query tiles, so the last pair of every item has a single
    stream, and enough key/value tiles (6 and more) that a stage held back would stall the ring."""
    _need(path, D)
    sides = (4, 17)
    rows, heads = 10, 40      # 400 items x 2 pairs: several pairs per persistent CTA
    qkv = make_qkv(rows, heads, sides, D, seed=17)
    with Cache(1, heads, D, rows, sides, [(0, 9, True)]) as cache:
        outs = run_pass(cache, qkv, path)
        want = oracle_outputs(qkv, cache.policies[0], 1.0 / math.sqrt(D))
        for k in range(len(sides)):
            check_close(outs[0][k], want[k], "scale %d" % k)


@pytest.mark.parametrize("D", [64, 128])
def test_bulk_copy_append_gives_the_same_cache(D):
    """The bulk-copy form of append (for appends that run underneath attention on a side stream) fills the
    cache exactly like the default copy kernel: outputs of a whole pass are bit-equal."""
    _need(B.PATH_AUTO, D)
    sides = (1, 3, 6, 8, 13)
    rows, heads = 3, 7
    qkv = make_qkv(rows, heads, sides, D, seed=23)
    pols = [(1, 2, False), (1, 2, True)]
    with Cache(2, heads, D, rows, sides, pols) as a, Cache(2, heads, D, rows, sides, pols, flags=B.FLAG_BULK_APPEND) as b:
        oa, ob = run_pass(a, qkv), run_pass(b, qkv)
        for layer in range(2):
            want = oracle_outputs(qkv, pols[layer], 1.0 / math.sqrt(D))
            for k in range(len(sides)):
                assert torch.equal(oa[layer][k], ob[layer][k]), (layer, k)
                check_close(ob[layer][k], want[k], "bulk append layer %d scale %d" % (layer, k))


def test_full_size_rows_sampled_against_oracle():
    """The VAR-d30 launch shape (512 rows x 30 heads, 680-token schedule) on one cache-efficient and one
    cache-demanding layer; sampled (row, head) items are compared with the oracle at every scale."""
    wl = synth.WORKLOADS["var_d30"]
    free_b, _ = torch.cuda.mem_get_info()
    if free_b < 12e9:
        pytest.skip("needs about 10 GB of device memory")
    qkv = make_qkv(wl.rows, wl.heads, wl.sides, wl.head_dim, wl.seed)
    pols = [(wl.n_condensed, wl.n_local, False), (wl.n_condensed, wl.n_local, True)]
    items = wl.rows * wl.heads
    g = torch.Generator().manual_seed(7)
    sample = sorted(set([0, wl.heads - 1, items - wl.heads, items - 1] +
                        torch.randint(0, items, (60,), generator=g).tolist()))
    with Cache(2, wl.heads, wl.head_dim, wl.rows, wl.sides, pols) as cache:
        outs = run_pass(cache, qkv, B.PATH_AUTO)
        idx = torch.tensor(sample, device="cuda")

        def pick(x):
            r, h, t, d = x.shape
            return x.reshape(r * h, t, d)[idx].reshape(len(sample), 1, t, d)

        small = [(pick(q), pick(k), pick(v)) for q, k, v in qkv]
        for layer, pol in enumerate(pols):
            want = oracle_outputs(small, pol, 1.0 / math.sqrt(wl.head_dim))
            for k in range(len(wl.sides)):
                check_close(pick(outs[layer][k]), want[k], "full-size layer %d scale %d" % (layer, k))
        # resident KV bytes equal the closed form for these two layers
        assert B.amskv_cache_bytes(cache.h)[1] == oracle.kv_bytes(wl.sides, pols, wl.rows, wl.heads, wl.head_dim)
