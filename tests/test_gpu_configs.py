"""GPU parity at the workload configurations' full shapes, on sampled (row, head) items and sampled
query rows: the launch shapes are the real ones, the oracle only computes what is sampled."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

from gpu_common import Cache, check_close, make_qkv, run_pass, to_items

pytestmark = pytest.mark.gpu


def _query_rows(T, g, n=96):
    """Sampled query tokens of a scale: ends, 128-row tile boundaries and random ones."""
    if T <= n:
        return list(range(T))
    fixed = {0, T - 1}
    for b in range(128, T, 128):
        fixed |= {b - 1, b}
    rnd = torch.randint(0, T, (n,), generator=g).tolist()
    return sorted(fixed | set(rnd))[: n + len(fixed)]


def _check_sampled(wl, pols, n_items, seed, path=B.PATH_AUTO, need_gb=4.0, fused=False):
    free_b, _ = torch.cuda.mem_get_info()
    if free_b < need_gb * 1e9:
        pytest.skip("needs about %.0f GB of device memory" % need_gb)
    qkv = make_qkv(wl.rows, wl.heads, wl.sides, wl.head_dim, wl.seed)
    items = wl.rows * wl.heads
    g = torch.Generator().manual_seed(seed)
    sample = sorted(set([0, wl.heads - 1, items - wl.heads, items - 1][: max(1, min(4, n_items))] +
                        torch.randint(0, items, (n_items,), generator=g).tolist()))
    idx = torch.tensor(sample, device="cuda")

    def pick(x):
        r, h, t, d = x.shape
        return x.reshape(r * h, t, d)[idx]

    scale = 1.0 / math.sqrt(wl.head_dim)
    with Cache(len(pols), wl.heads, wl.head_dim, wl.rows, wl.sides, pols) as cache:
        outs = run_pass(cache, qkv, path, fused=fused)
        Ks = [pick(k).cpu().double().numpy() for _, k, _ in qkv]
        Vs = [pick(v).cpu().double().numpy() for _, _, v in qkv]
        for k, (q, _, _) in enumerate(qkv):
            rows_k = _query_rows(q.shape[2], g)
            ridx = torch.tensor(rows_k, device="cuda")
            Qs = pick(q)[:, ridx].cpu().double().numpy()
            for layer, (c, w, dem) in enumerate(pols):
                want = oracle.attend_selected(Qs, Ks, Vs, oracle.keep_set(k, c, w, dem), scale)
                got = pick(outs[layer][k])[:, ridx].cpu().double()
                check_close(got, want, "%s layer %d scale %d" % (wl.name, layer, k))
                assert B.amskv_kept_segments(cache.h, layer, k) == oracle.keep_set(k, c, w, dem)
        assert B.amskv_cache_bytes(cache.h)[1] == oracle.kv_bytes(wl.sides, pols, wl.rows, wl.heads, wl.head_dim)


def test_var_d16_shape_sampled():
    """16 heads x 64, 128 rows (batch 64 doubled), condensed 2 / local 2, one layer of each class."""
    wl = synth.WORKLOADS["var_d16"]
    _check_sampled(wl, [(wl.n_condensed, wl.n_local, False), (wl.n_condensed, wl.n_local, True)], 48, seed=11)


def test_text_to_image_1024_shape_sampled():
    """16 heads x 128, 16 rows, 13 scales up to 64 x 64 (10 521 tokens), condensed 3 / local 2: the
    tensor-bound regime, 32 query tiles per item at the last scale."""
    wl = synth.WORKLOADS["t2i_1024"]
    _check_sampled(wl, [(wl.n_condensed, wl.n_local, False), (wl.n_condensed, wl.n_local, True)], 3, seed=12, need_gb=3.0)


def test_var_d30_full_shape_sampled_fused():
    """The shape the benchmark times, through the call it times: 512 rows x 30 heads x 64, amskv_append_attend at
    every scale, one layer of each class, sampled items and query rows."""
    wl = synth.WORKLOADS["var_d30"]
    _check_sampled(wl, [(wl.n_condensed, wl.n_local, False), (wl.n_condensed, wl.n_local, True)], 40, seed=15,
                   need_gb=12.0, fused=True)


def test_text_to_image_1024_shape_sampled_fused():
    """The 1024 x 1024-shaped workload (16 rows, 128 channels) through amskv_append_attend."""
    wl = synth.WORKLOADS["t2i_1024"]
    _check_sampled(wl, [(wl.n_condensed, wl.n_local, False), (wl.n_condensed, wl.n_local, True)], 3, seed=16,
                   need_gb=3.0, fused=True)


@pytest.mark.parametrize("fraction", [0.25, 1.0])
def test_sweep_points_at_batch_64(fraction):
    """Sweep points of the VAR-d30 head layout at batch 64 (128 rows): a quarter of the layers, and all of
    them, cache-demanding (the seeded mask decides which); fused calls, sampled items."""
    wl = synth.WORKLOADS["var_d30"].replace(batch=64, layers=4, demanding_fraction=fraction)
    pols = wl.policies()
    assert sum(1 for p in pols if p[2]) == (1 if fraction == 0.25 else 4)
    _check_sampled(wl, pols, 16, seed=17, need_gb=4.0, fused=True)


@pytest.mark.parametrize("fused", [False, True], ids=["separate", "fused"])
def test_depth_36_512_shape_sampled(fused):
    """36 heads x 64 (dim 2304), ten scales up to 32 x 32 (2 240 tokens): head_dim 64 with eight query
    tiles per item at the last scale (the tensor-bound launches take the one-CTA-per-SM form of the paired
    kernel), one layer of each class, sampled items and query rows."""
    wl = synth.WORKLOADS["var_d36_512"].replace(batch=8)
    _check_sampled(wl, [(wl.n_condensed, wl.n_local, False), (wl.n_condensed, wl.n_local, True)], 6, seed=14, need_gb=3.0,
                   fused=fused)


@pytest.mark.parametrize("batch", [1, 16, 64])
def test_policy_sweep_on_var_d30_shape(batch):
    """The VAR-d30 head layout at small batches with a mix of condensed / local settings and layer
    classes in one cache (the sweep's corner points)."""
    wl = synth.WORKLOADS["var_d30"].replace(batch=batch)
    pols = [(1, 1, False), (3, 3, False), (1, 3, False), (3, 1, False), (2, 2, True), (0, 2, False)]
    _check_sampled(wl, pols, 12, seed=13 + batch)
