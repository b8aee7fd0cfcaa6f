"""GPU parity: amskv_layer_similarity through the C ABI against the fp64 oracle."""
import pytest
import torch

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

from gpu_common import to_items

pytestmark = pytest.mark.gpu


def _gpu_ss(kp, sp, kc, sc, rows, heads, D, ws=None):
    n = B.amskv_similarity_workspace_bytes()
    ws = torch.empty(n, dtype=torch.uint8, device="cuda") if ws is None else ws
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    B.amskv_layer_similarity(kp, sp, kc, sc, rows, heads, D, out, ws, n)
    torch.cuda.synchronize()
    return float(out.item())


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("rho", [0.0, 0.9])
def test_similarity_matches_oracle_on_adjacent_scales(D, rho):
    rows, heads = 3, 5
    sides = (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)
    keys = synth.smooth_field_keys(rows, heads, sides, D, seed=77, rho=rho, device="cuda")
    for i in range(1, len(sides)):
        got = _gpu_ss(keys[i - 1], sides[i - 1], keys[i], sides[i], rows, heads, D)
        want = oracle.similarity_ss(to_items(keys[i - 1]), sides[i - 1], to_items(keys[i]), sides[i])
        assert abs(got - want) <= 1e-5 * max(want, 1e-30), (i, got, want)


def test_identity_is_zero_and_result_is_reproducible():
    rows, heads, D, s = 2, 4, 64, 9
    k = synth.normal_bf16((rows, heads, s * s, D), 3, "cuda")
    assert _gpu_ss(k, s, k, s, rows, heads, D) == 0.0
    k2 = synth.normal_bf16((rows, heads, 144, D), 4, "cuda")
    a = _gpu_ss(k, s, k2, 12, rows, heads, D)
    b = _gpu_ss(k, s, k2, 12, rows, heads, D)
    assert a == b and a > 0


def test_large_problem_uses_grid_stride_and_fixed_partials():
    rows, heads, D = 64, 16, 64           # 1024 items x 256 tokens: more chunks than the partial slots
    kp = synth.normal_bf16((rows, heads, 169, D), 5, "cuda")
    kc = synth.normal_bf16((rows, heads, 256, D), 6, "cuda")
    got = _gpu_ss(kp, 13, kc, 16, rows, heads, D)
    want = oracle.similarity_ss(to_items(kp), 13, to_items(kc), 16)
    assert abs(got - want) <= 1e-5 * want


@pytest.mark.parametrize("D", [64, 128])
def test_few_items_with_long_sides_are_split_into_parts(D):
    """Two items of 48 x 48 tokens: each item is cut into many block-sized parts (with a ragged last one);
    also a larger previous scale than current one (downsampling), which the bilinear rule covers as well."""
    rows, heads = 1, 2
    kp = synth.normal_bf16((rows, heads, 40 * 40, D), 7, "cuda")
    kc = synth.normal_bf16((rows, heads, 48 * 48, D), 8, "cuda")
    for a, sa, b, sb in ((kp, 40, kc, 48), (kc, 48, kp, 40)):
        got = _gpu_ss(a, sa, b, sb, rows, heads, D)
        want = oracle.similarity_ss(to_items(a), sa, to_items(b), sb)
        assert abs(got - want) <= 1e-5 * want


def test_correlated_layers_rank_above_independent_ones():
    rows, heads, D = 4, 8, 64
    sides = (4, 5, 6, 8, 10)
    scores = []
    for layer in range(6):
        rho = 0.9 if layer % 2 == 0 else 0.0
        keys = synth.smooth_field_keys(rows, heads, sides, D, seed=200 + layer, rho=rho, device="cuda")
        ss = sum(_gpu_ss(keys[i - 1], sides[i - 1], keys[i], sides[i], rows, heads, D) for i in range(1, len(sides)))
        scores.append(-(ss ** 0.5))
    # the three independent layers have the lowest similarity -> cache-demanding
    assert B.amskv_classify_lowest(scores, 3) == [False, True, False, True, False, True]


def test_argument_errors():
    k = synth.normal_bf16((1, 1, 4, 64), 1, "cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    n = B.amskv_similarity_workspace_bytes()
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    f = B.lib.amskv_layer_similarity
    assert f(k.data_ptr(), 2, k.data_ptr(), 2, 1, 1, 64, out.data_ptr(), ws.data_ptr(), n - 1, None) == B.ERR_NOMEM
    assert f(k.data_ptr(), 2, k.data_ptr(), 2, 1, 1, 96, out.data_ptr(), ws.data_ptr(), n, None) == B.ERR_UNSUPPORTED
    assert f(None, 2, k.data_ptr(), 2, 1, 1, 64, out.data_ptr(), ws.data_ptr(), n, None) == B.ERR_INVALID
    assert f(k.data_ptr(), 0, k.data_ptr(), 2, 1, 1, 64, out.data_ptr(), ws.data_ptr(), n, None) == B.ERR_INVALID
