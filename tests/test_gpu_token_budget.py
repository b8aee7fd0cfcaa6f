"""GPU parity of the token-budget policy (Algorithm 1 with Algorithm 2 as its roll, capacities in
tokens): append + attend through the C ABI against the oracle's attention over the token list that
its literal simulation of the two algorithms leaves."""
import math

import pytest
import torch

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

from gpu_common import Cache, check_close, make_qkv, run_pass, tensor_path_available, to_items

pytestmark = pytest.mark.gpu

PATHS = {"auto": B.PATH_AUTO, "simt": B.PATH_SIMT, "pair": B.PATH_TENSOR_PAIR, "tensor": B.PATH_TENSOR}


def _check_all(rows, heads, D, sides, budgets, path, seed, flags=0):
    if path != B.PATH_SIMT and not tensor_path_available(D):
        pytest.skip("tensor-core path not available")
    qkv = make_qkv(rows, heads, sides, D, seed)
    scale = 1.0 / math.sqrt(D)
    Ks = [to_items(k) for _, k, _ in qkv]
    Vs = [to_items(v) for _, _, v in qkv]
    pols = [(2, 2, False)] * len(budgets)
    with Cache(len(budgets), heads, D, rows, sides, pols, token_budgets=budgets, flags=flags) as cache:
        outs = run_pass(cache, qkv, path)
        for layer, (b, c) in enumerate(budgets):
            for k, (q, _, _) in enumerate(qkv):
                want = oracle.attend_tokens(to_items(q), Ks, Vs, oracle.attended_tokens(sides, k, b, c), scale)
                check_close(outs[layer][k], want, "budget %d/%d scale %d" % (b, c, k))
        resident = sum(len(oracle.algorithm1_tokens(list(sides), b, b, c, False)[-1]) for b, c in budgets)
        assert B.amskv_cache_bytes(cache.h)[1] == resident * 2 * 2 * rows * heads * D


@pytest.mark.parametrize("path", list(PATHS), ids=list(PATHS))
def test_small_schedule_every_element(path):
    """Budgets that never roll, roll through the middle of a scale, cut a scale by its own roll,
    leave no ring at all, and skip scales larger than the budget."""
    budgets = [(500, 5), (100, 5), (40, 5), (70, 0), (13, 3), (5, 5), (64, 14), (1, 0)]
    _check_all(3, 5, 64, (1, 2, 3, 4, 5, 6, 8), budgets, PATHS[path], seed=31)


@pytest.mark.parametrize("path", ["auto", "simt"])
def test_paper_setting_every_element(path):
    """C_cds = the first two scales (5 tokens), C_min = C_cds + the penultimate scale (174),
    C_max = C_cds + the last two scales (430), on the 680-token schedule."""
    _check_all(2, 6, 64, synth.SIDES_256, [(174, 5), (430, 5)], PATHS[path], seed=32)


def test_head_dim_128_and_bulk_append():
    _check_all(2, 3, 128, (1, 2, 4, 6, 9, 12), [(120, 5), (60, 0)], B.PATH_AUTO, seed=33)
    _check_all(2, 3, 64, (1, 2, 4, 6, 9, 12), [(120, 5), (60, 0)], B.PATH_AUTO, seed=34, flags=B.FLAG_BULK_APPEND)


def test_paper_setting_on_var_d30_shape_sampled():
    """The VAR-d30 head layout at 64 rows with the paper's budgets, on sampled items and query rows."""
    wl = synth.WORKLOADS["var_d30"].replace(batch=32)
    if not tensor_path_available(64):
        pytest.skip("tensor-core path not available")
    budgets = [(174, 5), (430, 5)]
    qkv = make_qkv(wl.rows, wl.heads, wl.sides, wl.head_dim, wl.seed)
    items = wl.rows * wl.heads
    g = torch.Generator().manual_seed(35)
    sample = sorted(set([0, items - 1] + torch.randint(0, items, (24,), generator=g).tolist()))
    idx = torch.tensor(sample, device="cuda")

    def pick(x):
        r, h, t, d = x.shape
        return x.reshape(r * h, t, d)[idx]

    scale = 1.0 / math.sqrt(wl.head_dim)
    with Cache(2, wl.heads, wl.head_dim, wl.rows, wl.sides, [(2, 2, False)] * 2, token_budgets=budgets) as cache:
        outs = run_pass(cache, qkv)
        Ks = [pick(k).cpu().double().numpy() for _, k, _ in qkv]
        Vs = [pick(v).cpu().double().numpy() for _, _, v in qkv]
        for k, (q, _, _) in enumerate(qkv):
            Qs = pick(q).cpu().double().numpy()
            for layer, (b, c) in enumerate(budgets):
                want = oracle.attend_tokens(Qs, Ks, Vs, oracle.attended_tokens(wl.sides, k, b, c), scale)
                check_close(pick(outs[layer][k]).cpu().double(), want, "layer %d scale %d" % (layer, k))
