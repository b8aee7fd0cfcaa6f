"""Host-side logic of the C ABI against the oracle; no GPU needed (plan-only caches)."""
import itertools
import os
import re

import pytest

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _plan(sides, policies, heads=2, head_dim=64, rows=2):
    d, keep = B.make_desc(len(policies), heads, head_dim, rows, sides, policies, flags=B.FLAG_PLAN_ONLY)
    return B.amskv_cache_create(d), d, keep


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "amskv.h")).read()
    declared = set(re.findall(r"AMSKV_API[^;(]*?\b(amskv_\w+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(B.lib, name), name


def test_kept_and_evicted_match_oracle_bruteforce():
    for K in (1, 2, 3, 5, 8):
        sides = list(range(1, K + 1))
        combos = list(itertools.product(range(0, K + 2), range(1, K + 2), (False, True)))
        cache, d, keep = _plan(sides, combos)
        for layer, (c, w, dem) in enumerate(combos):
            for k in range(K):
                assert B.amskv_kept_segments(cache, layer, k) == oracle.keep_set(k, c, w, dem)
                assert B.amskv_evicted_at(cache, layer, k) == oracle.evicted_at(k, c, w, dem)
        B.amskv_cache_destroy(cache)


@pytest.mark.parametrize("sides", [synth.SIDES_256, synth.SIDES_1024, (3, 1, 4, 1, 5, 9, 2, 6)])
def test_layout_is_collision_free_and_ranges_cover_exactly_the_kept_tokens(sides):
    K = len(sides)
    tokens = [s * s for s in sides]
    combos = list(itertools.product(range(0, 4), range(1, 5), (False, True)))
    cache, d, keep = _plan(sides, combos)
    for layer, (c, w, dem) in enumerate(combos):
        owner = {}     # token position -> segment currently stored there
        home = {}      # segment -> start, discovered from the ranges when it is appended
        for k in range(K):
            ranges = B.amskv_resident_ranges(cache, layer, k)
            kept = oracle.keep_set(k, c, w, dem)
            assert sum(n for _, n in ranges) == sum(tokens[s] for s in kept)
            # ranges are sorted, disjoint and non-adjacent (merged)
            for (a, n), (b, _) in zip(ranges, ranges[1:]):
                assert a + n < b
            covered = set()
            for a, n in ranges:
                covered |= set(range(a, a + n))
            prev_cover = home.get("cover", set())
            new_positions = covered - {p for p in prev_cover if owner.get(p) in kept}
            # the newly appended segment occupies exactly T_k fresh positions
            assert len(new_positions) == tokens[k]
            for p in new_positions:
                owner[p] = k
            # every covered position belongs to a kept segment
            assert {owner[p] for p in covered} == set(kept)
            for s in kept:
                assert sum(1 for p in covered if owner[p] == s) == tokens[s]
            home["cover"] = covered
    B.amskv_cache_destroy(cache)


def test_single_contiguous_range_for_window_up_to_two():
    for c, w in itertools.product(range(0, 4), (1, 2)):
        cache, d, keep = _plan(synth.SIDES_256, [(c, w, False)])
        for k in range(len(synth.SIDES_256)):
            assert len(B.amskv_resident_ranges(cache, 0, k)) == 1
        B.amskv_cache_destroy(cache)


def test_required_bytes_match_closed_form():
    wl = synth.WORKLOADS["var_d30"]
    pol = wl.policies()
    d, keep = B.make_desc(wl.layers, wl.heads, wl.head_dim, wl.rows, wl.sides, pol, flags=B.FLAG_PLAN_ONLY)
    need = B.amskv_cache_required_bytes(d)
    exact = oracle.kv_bytes(wl.sides, pol, wl.rows, wl.heads, wl.head_dim)
    assert exact == 2 * 2 * 512 * 30 * 64 * (9 * 680 + 21 * 430)
    assert exact <= need <= exact + 256 * (wl.layers + 1)
    full, keep2 = B.make_desc(wl.layers, wl.heads, wl.head_dim, wl.rows, wl.sides, wl.policies(True),
                              flags=B.FLAG_PLAN_ONLY)
    assert B.amskv_cache_required_bytes(full) > need


def test_resident_bytes_follow_the_policy():
    wl = synth.WORKLOADS["single"]
    pol = [(2, 2, False), (2, 2, True)]
    cache, d, keep = _plan(wl.sides, pol, heads=wl.heads, rows=wl.rows)
    per_token = 2 * 2 * wl.rows * wl.heads * 64
    for k in range(len(wl.sides)):
        for layer in range(2):
            B.lib.amskv_append(cache, layer, k, None, None, None, None)
        _, now, peak = B.amskv_cache_bytes(cache)
        expect = sum(oracle.kept_tokens(wl.sides, oracle.keep_set(k, c, w, dem)) for c, w, dem in pol) * per_token
        assert now == expect
        assert peak >= now
    assert now == oracle.kv_bytes(wl.sides, pol, wl.rows, wl.heads, 64)
    B.amskv_cache_reset(cache)
    assert B.amskv_cache_bytes(cache)[1] == 0
    B.amskv_cache_destroy(cache)


def test_order_contract_and_argument_errors():
    cache, d, keep = _plan((1, 2, 3), [(1, 1, False)])
    assert B.lib.amskv_append(cache, 0, 1, None, None, None, None) == B.ERR_ORDER
    assert B.lib.amskv_append(cache, 0, 0, None, None, None, None) == B.OK
    assert B.lib.amskv_append(cache, 0, 0, None, None, None, None) == B.ERR_ORDER
    assert B.lib.amskv_append(cache, 1, 0, None, None, None, None) == B.ERR_INVALID
    assert B.lib.amskv_append(cache, 0, 3, None, None, None, None) == B.ERR_INVALID
    assert B.lib.amskv_attend(cache, 0, 0, None, None, None, None, None) == B.ERR_UNSUPPORTED  # plan-only
    assert B.lib.amskv_set_attend_path(cache, 7) == B.ERR_INVALID
    assert B.lib.amskv_set_attend_path(cache, B.PATH_TENSOR) == B.ERR_UNSUPPORTED
    B.amskv_cache_destroy(cache)
    # descriptor validation
    for kw in (dict(head_dim=96), dict(rows=0), dict(heads=0)):
        args = dict(layers=1, heads=2, head_dim=64, rows=2)
        args.update(kw)
        d, keep = B.make_desc(args["layers"], args["heads"], args["head_dim"], args["rows"], (1, 2), [(1, 1, False)],
                              flags=B.FLAG_PLAN_ONLY)
        with pytest.raises(B.AmskvError):
            B.amskv_cache_create(d)
    d, keep = B.make_desc(1, 2, 64, 2, (1, 2), [(1, 0, False)], flags=B.FLAG_PLAN_ONLY)   # window of zero
    with pytest.raises(B.AmskvError) as e:
        B.amskv_cache_create(d)
    assert e.value.code == B.ERR_INVALID
    d, keep = B.make_desc(1, 2, 64, 2, (1, 0), [(1, 1, False)], flags=B.FLAG_PLAN_ONLY)   # empty scale
    with pytest.raises(B.AmskvError):
        B.amskv_cache_create(d)
    assert B.strerror(B.ERR_ORDER) == "call out of order"


def test_classification_matches_oracle():
    scores = [-3.0, -1.0, -2.0, -1.0, -2.0]
    assert B.amskv_classify_by_threshold(scores, -2.0) == oracle.classify_layers(scores, -2.0)
    for n in range(0, 6):
        assert B.amskv_classify_lowest(scores, n) == oracle.lowest_similarity_layers(scores, n)


def test_compute_calls_fail_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    d, keep = B.make_desc(1, 2, 64, 2, (1, 2), [(1, 1, False)])
    with pytest.raises(B.AmskvError) as e:
        B.amskv_cache_create(d)
    assert e.value.code == B.ERR_CUDA


def test_longest_schedule_and_its_limits():
    """AMSKV_MAX_SCALES scales are accepted (kept sets equal the oracle's at every step, window larger than a
    handful of slots), one more is refused, and so are sides outside 1 .. 4096."""
    import oracle
    sides = tuple(1 + (i % 3) for i in range(B.MAX_SCALES))
    pols = [(3, 7, False), (0, 31, False), (5, 1, True)]
    d, keep = B.make_desc(len(pols), 2, 64, 2, sides, pols, flags=B.FLAG_PLAN_ONLY)
    cache = B.amskv_cache_create(d)
    for k in range(len(sides)):
        for layer, (c, w, dem) in enumerate(pols):
            assert B.lib.amskv_append(cache, layer, k, None, None, None, None) == B.OK
            assert B.amskv_kept_segments(cache, layer, k) == oracle.keep_set(k, c, w, dem)
            ranges = B.amskv_resident_ranges(cache, layer, k)
            assert sum(n for _, n in ranges) == oracle.kept_tokens(sides, oracle.keep_set(k, c, w, dem))
    B.amskv_cache_destroy(cache)
    for bad in (sides + (1,), (0, 1), (1, 4097)):
        d, keep = B.make_desc(1, 2, 64, 2, bad, [(1, 1, False)], flags=B.FLAG_PLAN_ONLY)
        with pytest.raises(B.AmskvError) as e:
            B.amskv_cache_create(d)
        assert e.value.code == B.ERR_INVALID
