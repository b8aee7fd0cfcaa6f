"""GPU parity for kernel branches that ordinary inputs reach rarely or never: the rescale of the running
softmax reference (both head sizes, fused and separate calls), the give-up path of a bounded wait, and
argument checks that need a device cache."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

from gpu_common import Cache, check_close, make_qkv, oracle_outputs, run_pass, tensor_path_available, to_items

pytestmark = pytest.mark.gpu

PATHS = {"pair": B.PATH_TENSOR_PAIR, "auto": B.PATH_AUTO, "tensor": B.PATH_TENSOR, "simt": B.PATH_SIMT}


def _need(D):
    if not tensor_path_available(D):
        pytest.skip("tensor-core path not available for head_dim %d" % D)


@pytest.mark.parametrize("fused", [False, True], ids=["separate", "fused"])
@pytest.mark.parametrize("path", ["pair", "auto"])
def test_peaked_softmax_rows_head_dim_128(path, fused):
    """Logit spread of several units with 128 channels: the wide form of the paired kernel, whose rescale
    waits for the previous P V on a barrier of its own."""
    _need(128)
    sides = (2, 5, 9, 14, 18)
    rows, heads, D = 2, 3, 128
    qkv = make_qkv(rows, heads, sides, D, seed=81, peaked=True)
    with Cache(2, heads, D, rows, sides, [(1, 2, True), (1, 2, False)]) as cache:
        outs = run_pass(cache, qkv, PATHS[path], fused=fused)
        for layer, pol in enumerate(cache.policies):
            want = oracle_outputs(qkv, pol, 1.0 / math.sqrt(D))
            for k in range(len(sides)):
                check_close(outs[layer][k], want[k], "peaked D=128 layer %d scale %d" % (layer, k), max_abs=4e-2)


@pytest.mark.parametrize("fused", [False, True], ids=["separate", "fused"])
@pytest.mark.parametrize("path", ["pair", "auto", "tensor", "simt"])
@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("step", [8, 48])
def test_reference_maximum_moves_in_every_key_tile(D, path, fused, step):
    """Keys built so that every row's largest logit grows by `step` from one 64-token tile to the next.
    step 8 (11.5 in base-2 units, above the rescale threshold of 2^8): a kernel that takes every tile's
    maximum brings the accumulator and the row sum to a new reference in every tile of every row.
    step 48 (69 in base-2 units, above the 2^64 limit on a tile's sum): a kernel that only takes the first
    tile's maximum finds every later tile out of range and has to form each of them a second time."""
    _need(D)
    sides = (8, 18)                      # 64 + 324 keys: seven key tiles at the last scale, three query tiles
    rows, heads = 3, 5
    scale = 1.0 / 8 if D == 64 else 1.0 / 16
    qkv, level = [], 0
    for k, s in enumerate(sides):
        qkv.append(synth.growing_logit_qkv(rows, heads, s * s, D, 82, k, first_level=level, step=step, device="cuda"))
        level += (s * s + 63) // 64
    # the inputs do what they are meant to: per-tile maxima of the true logits climb by more than 2^8 (base 2)
    q, kk = to_items(qkv[1][0])[0], np.concatenate([to_items(qkv[0][1])[0], to_items(qkv[1][1])[0]], 0)
    z = scale * (q @ kk.T) * math.log2(math.e)
    tile_max = np.stack([z[:, t:t + 64].max(axis=1) for t in range(0, 320, 64)], 1)
    assert (np.diff(tile_max, axis=1) > 8.0).all()
    with Cache(1, heads, D, rows, sides, [(0, 9, True)], softmax_scale=scale) as cache:
        outs = run_pass(cache, qkv, PATHS[path], fused=fused)
        want = oracle_outputs(qkv, (0, 9, True), scale)
        for k in range(len(sides)):
            check_close(outs[0][k], want[k], "D=%d scale %d" % (D, k), max_abs=2e-2)


def test_a_wait_that_runs_out_is_reported_and_the_cache_stays_usable():
    """A bounded wait nothing ever satisfies: the kernel gives up after its iteration limit, records its
    code and returns; amskv_status reports it once; an ordinary pass on the same cache then succeeds."""
    _need(64)
    sides, rows, heads, D = (2, 9), 2, 3, 64
    qkv = make_qkv(rows, heads, sides, D, seed=83)
    with Cache(1, heads, D, rows, sides, [(1, 1, True)]) as cache:
        assert B.amskv_status(cache.h) == 0
        B.amskv_selftest_wait_timeout(cache.h, 1000)
        w = B.ctypes.c_int(0)
        assert B.lib.amskv_status(cache.h, B.ctypes.byref(w)) == B.ERR_DEVICE_TIMEOUT
        assert w.value == 3
        assert B.lib.amskv_status(cache.h, B.ctypes.byref(w)) == B.OK and w.value == 0     # read and cleared
        outs = run_pass(cache, qkv, B.PATH_TENSOR_PAIR)                                     # asserts status 0
        want = oracle_outputs(qkv, (1, 1, True), 1.0 / math.sqrt(D))
        for k in range(len(sides)):
            check_close(outs[0][k], want[k], "after the timeout, scale %d" % k)
        # limits of the diagnostic itself
        assert B.lib.amskv_selftest_wait_timeout(cache.h, 0, None) == B.ERR_INVALID
        assert B.lib.amskv_selftest_wait_timeout(cache.h, (1 << 20) + 1, None) == B.ERR_INVALID
        assert B.lib.amskv_selftest_wait_timeout(None, 10, None) == B.ERR_INVALID


def test_status_word_written_by_hand_is_reported_with_its_code():
    """The reporting chain without any kernel: a code stored in the status word of a caller-owned arena."""
    with Cache(1, 2, 64, 2, (1, 2), [(1, 1, False)]) as cache:
        word = cache.arena[:4].view(torch.int32)
        for code in (1, 2, 3):
            word.fill_(code)
            torch.cuda.synchronize()
            w = B.ctypes.c_int(0)
            assert B.lib.amskv_status(cache.h, B.ctypes.byref(w)) == B.ERR_DEVICE_TIMEOUT and w.value == code
            assert int(word.item()) == 0
        B.amskv_cache_reset(cache.h)
        assert B.amskv_status(cache.h) == 0


def test_broadcast_strides_are_refused():
    """A zero row or head stride (an expanded view) cannot be described to the copy engine: refused for every
    tensor where the dimension has more than one entry, and always for the output."""
    rows, heads, D = 2, 3, 64
    with Cache(1, heads, D, rows, (2, 3), [(1, 1, False)]) as cache:
        q, k, v = synth.qkv_for_scale(rows, heads, 4, D, 5, 0, "cuda")
        o = torch.empty_like(q)
        k_b = k[:, :1].expand(rows, heads, 4, D)          # head-broadcast keys
        v_r = v[:1].expand(rows, heads, 4, D)             # row-broadcast values
        i64 = B.ctypes.c_int64

        def st(t):
            return (i64 * 3)(*t.stride()[:3])

        assert B.lib.amskv_append(cache.h, 0, 0, k_b.data_ptr(), v.data_ptr(), st(k_b), None) == B.ERR_INVALID
        assert B.lib.amskv_append(cache.h, 0, 0, k.data_ptr(), v_r.data_ptr(), st(v_r), None) == B.ERR_INVALID
        assert B.lib.amskv_append_attend(cache.h, 0, 0, k_b.data_ptr(), v.data_ptr(), st(k_b), q.data_ptr(), o.data_ptr(),
                                         None, None, None) == B.ERR_INVALID
        B.amskv_append(cache.h, 0, 0, k, v)
        q_b = q[:, :1].expand(rows, heads, 4, D)
        assert B.lib.amskv_attend(cache.h, 0, 0, q_b.data_ptr(), o.data_ptr(), st(q_b), None, None) == B.ERR_INVALID
        o_b = o[:1].expand(rows, heads, 4, D)
        assert B.lib.amskv_attend(cache.h, 0, 0, q.data_ptr(), o_b.data_ptr(), None, st(o_b), None) == B.ERR_INVALID
        B.amskv_attend(cache.h, 0, 0, q, o)
        torch.cuda.synchronize()
        assert B.amskv_status(cache.h) == 0
    # one row: a zero row stride on an input addresses nothing else and is accepted; on the output it is not
    with Cache(1, heads, D, 1, (2,), [(1, 1, False)]) as cache:
        q, k, v = synth.qkv_for_scale(1, heads, 4, D, 6, 0, "cuda")
        o = torch.empty_like(q)
        strides = (B.ctypes.c_int64 * 3)(0, 4 * D, D)
        assert B.lib.amskv_append(cache.h, 0, 0, k.data_ptr(), v.data_ptr(), strides, None) == B.OK
        assert B.lib.amskv_attend(cache.h, 0, 0, q.data_ptr(), o.data_ptr(), strides, strides, None) == B.ERR_INVALID
        assert B.lib.amskv_attend(cache.h, 0, 0, q.data_ptr(), o.data_ptr(), strides, None, None) == B.OK
        torch.cuda.synchronize()
        want = oracle.attend_selected(to_items(q), [to_items(k)], [to_items(v)], [0], 1.0 / math.sqrt(D))
        check_close(o, want, "one row, zero row stride")


def test_nvtx_ranges_change_nothing():
    """AMSKV_FLAG_NVTX wraps every call in a named range for timeline tools; outputs are bit-equal with and without."""
    sides, rows, heads, D = (1, 2, 4, 9), 2, 3, 64
    qkv = make_qkv(rows, heads, sides, D, seed=84)
    with Cache(1, heads, D, rows, sides, [(1, 2, False)]) as a, Cache(1, heads, D, rows, sides, [(1, 2, False)], flags=B.FLAG_NVTX) as b:
        for fused in (False, True):
            oa, ob = run_pass(a, qkv, fused=fused), run_pass(b, qkv, fused=fused)
            for x, y in zip(oa[0], ob[0]):
                assert torch.equal(x, y)
    d, keep = B.make_desc(1, heads, D, rows, sides, [(1, 2, False)], flags=16)
    with pytest.raises(B.AmskvError) as e:
        B.amskv_cache_create(d)
    assert e.value.code == B.ERR_INVALID


@pytest.mark.parametrize("fused", [False, True], ids=["separate", "fused"])
def test_longest_schedule_many_ranges(fused):
    """32 scales (the most a cache takes), a window of 7 and of 31 rotating slots: many short resident ranges per
    call, every scale compared with the oracle."""
    sides = tuple(1 + (i % 4) for i in range(B.MAX_SCALES))
    rows, heads, D = 2, 3, 64
    pols = [(3, 7, False), (0, 31, False), (5, 1, True)]
    qkv = make_qkv(rows, heads, sides, D, seed=85)
    with Cache(len(pols), heads, D, rows, sides, pols) as cache:
        outs = run_pass(cache, qkv, fused=fused)
        for layer, pol in enumerate(pols):
            want = oracle_outputs(qkv, pol, 1.0 / math.sqrt(D))
            for k in range(len(sides)):
                check_close(outs[layer][k], want[k], "layer %d scale %d" % (layer, k))
