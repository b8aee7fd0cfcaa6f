"""GPU test of amskv_layer_similarity_static, the similarity call that allocates nothing.

Some users of the library cannot hand it a workspace: they run inside a fixed memory pool, or
as a plug-in that only receives its tensors, or in a loop where cudaMalloc is not allowed.
For them the library keeps the scratch for the partial sums in a small array of its own.
This file checks that call against amskv_layer_similarity (the workspace-taking call it
mirrors) through the C ABI, twice in a row with different inputs, because both calls reuse
the one array and the second must not be disturbed by what the first left behind.

The file name sorts last on purpose: a run that stops at the first failure has then already
gone through every other test.
"""
import pytest
import torch

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

pytestmark = pytest.mark.gpu

REL_TOL = 1e-5   # the tolerance the similarity parity tests use (the two calls are in fact bit-equal)


def _with_workspace(kp, sp, kc, sc, rows, heads, D):
    n = B.amskv_similarity_workspace_bytes()
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    B.amskv_layer_similarity(kp, sp, kc, sc, rows, heads, D, out, ws, n)
    torch.cuda.synchronize()
    return float(out.item())


def _static(kp, sp, kc, sc, rows, heads, D):
    out = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    B.amskv_layer_similarity_static(kp, sp, kc, sc, rows, heads, D, out)
    torch.cuda.synchronize()
    return float(out.item())


def test_static_scratch_matches_workspace_call_twice_in_a_row():
    # first call: 2048 (row, head) items, one block each, so every one of the 2048 partial slots is written;
    # second call: a small problem that uses only a few of them, so stale partials of the first call sit right
    # behind the live ones
    cases = [
        (128, 16, 64, 13, 16, 11),
        (2, 3, 128, 5, 6, 12),
    ]
    for rows, heads, D, sp, sc, seed in cases:
        kp = synth.normal_bf16((rows, heads, sp * sp, D), seed, "cuda")
        kc = synth.normal_bf16((rows, heads, sc * sc, D), seed + 100, "cuda")
        want = _with_workspace(kp, sp, kc, sc, rows, heads, D)
        got = _static(kp, sp, kc, sc, rows, heads, D)
        assert want > 0
        assert abs(got - want) <= REL_TOL * want, (rows, heads, D, got, want)
        # and against the definition (fp64 CPU oracle), so that the pair of calls is not only self-consistent
        ref = oracle.similarity_ss(kp.cpu().double().reshape(rows * heads, sp * sp, D).numpy(), sp,
                                   kc.cpu().double().reshape(rows * heads, sc * sc, D).numpy(), sc)
        assert abs(got - ref) <= REL_TOL * ref, (rows, heads, D, got, ref)


def test_static_scratch_at_its_stated_maximum():
    """Exactly 2^30 sixteen-byte chunks of current-scale keys (16 GiB) is accepted and agrees with the
    workspace call; one more (row, head) item is refused before anything is launched."""
    free_b, _ = torch.cuda.mem_get_info()
    if free_b < 24e9:
        pytest.skip("needs about 17 GB of device memory")
    rows, heads, D, sp, sc = 1024, 16, 128, 2, 64          # 1024 * 16 * 64^2 * 128 / 8 = 2^30
    assert rows * heads * sc * sc * D // 8 == 1 << 30
    kp = synth.normal_bf16((rows, heads + 1, sp * sp, D), 21, "cuda")
    kc = torch.zeros((rows, heads + 1, sc * sc, D), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    f = B.lib.amskv_layer_similarity_static
    assert f(kp.data_ptr(), sp, kc.data_ptr(), sc, rows, heads + 1, D, out.data_ptr(), None) == B.ERR_UNSUPPORTED
    want = _with_workspace(kp, sp, kc, sc, rows, heads, D)
    got = _static(kp, sp, kc, sc, rows, heads, D)
    assert want > 0 and got == want
    del kc
    torch.cuda.empty_cache()


def test_static_scratch_argument_errors():
    k = synth.normal_bf16((1, 1, 4, 64), 1, "cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    f = B.lib.amskv_layer_similarity_static
    assert f(None, 2, k.data_ptr(), 2, 1, 1, 64, out.data_ptr(), None) == B.ERR_INVALID
    assert f(k.data_ptr(), 2, k.data_ptr(), 2, 1, 1, 96, out.data_ptr(), None) == B.ERR_UNSUPPORTED
    # beyond the stated maximum of 2^30 sixteen-byte chunks: refused before anything is launched
    assert f(k.data_ptr(), 2, k.data_ptr(), 4096, 1 << 10, 1 << 4, 128, out.data_ptr(), None) == B.ERR_UNSUPPORTED
