"""On-line promotion of a live cache (Algorithm 1: the budget becomes C_max when the similarity test passes at
the first overflow): the library's host-side plan against the oracle.  No GPU needed (plan-only caches)."""
import itertools

import pytest

import oracle
from paper_2511_16047_b200 import binding as B

SIDES_680 = (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)


def _expand(runs):
    return [(s, t) for s, first, count in runs for t in range(first, first + count)]


def _plan(sides, policies, budgets=None, heads=2, rows=2, flags=0):
    d, keep = B.make_desc(len(policies), heads, 64, rows, sides, policies, flags=B.FLAG_PLAN_ONLY | flags,
                          token_budgets=budgets)
    return B.amskv_cache_create(d), d, keep


def _append(cache, layer, k):
    assert B.lib.amskv_append(cache, layer, k, None, None, None, None) == B.OK


def test_token_budget_layer_promoted_at_its_first_overflow():
    """The paper's setting: 5 / 174 / 430 tokens.  The first overflow is scale 7 (255 > 174); promoted there, the
    layer behaves as Algorithm 1 with the test passing at scale 7; left alone, as a C_min layer."""
    cache, d, keep = _plan(SIDES_680, [(2, 2, False)] * 2, budgets=[(174, 5, 430), (174, 5, 430)])
    assert B.amskv_first_overflow_scale(cache, 0) == 7
    pass_at_7 = [False] * 7 + [True] * 3
    for k in range(len(SIDES_680)):
        if k == 7:
            B.amskv_promote_layer(cache, 0)          # layer 0: S < theta at the overflow; layer 1: not
        for layer in (0, 1):
            _append(cache, layer, k)
        want0 = oracle.attended_tokens(SIDES_680, k, 174, 5, c_max=430, below_theta=pass_at_7)
        want1 = oracle.attended_tokens(SIDES_680, k, 174, 5, c_max=430, below_theta=False)
        assert sorted(_expand(B.amskv_attended_tokens(cache, 0, k))) == sorted(want0), k
        assert sorted(_expand(B.amskv_attended_tokens(cache, 1, k))) == sorted(want1), k
        caches0, budgets0 = oracle.algorithm1_trace(SIDES_680[:k + 1], 174, 430, 5, pass_at_7)
        assert B.amskv_kept_segments(cache, 0, k) == sorted({s for s, _ in caches0[k]})
    # end states of Sec. 5.1: condensed + last two scales (430 tokens) / condensed + penultimate (174)
    assert B.amskv_kept_segments(cache, 0, 9) == [0, 1, 8, 9] and B.amskv_kept_segments(cache, 1, 9) == [0, 1, 8]
    per_token = 2 * 2 * 2 * 2 * 64
    assert B.amskv_cache_bytes(cache)[1] == (430 + 174) * per_token
    # both regions are sized for the larger layout (C_max = 430 against C_min + a transient slot of 256)
    assert B.amskv_cache_required_bytes(d) == 256 + 2 * max(430, 174 + 256) * per_token
    B.amskv_cache_destroy(cache)


def test_promotion_is_refused_after_the_first_eviction_and_for_ordinary_layers():
    cache, d, keep = _plan(SIDES_680, [(2, 2, False)] * 2, budgets=[(174, 5, 430), (174, 5)])
    for k in range(8):
        _append(cache, 0, k)
    assert B.lib.amskv_promote_layer(cache, 0) == B.ERR_ORDER          # scale 7 has overflowed and rolled
    assert B.lib.amskv_promote_layer(cache, 1) == B.ERR_UNSUPPORTED    # created without a promoted budget
    assert B.lib.amskv_promote_layer(cache, 2) == B.ERR_INVALID
    # a new batch starts every layer in the class it was created with, promotable again
    B.amskv_cache_reset(cache)
    B.amskv_promote_layer(cache, 0)
    B.amskv_promote_layer(cache, 0)                                    # twice is harmless
    for k in range(10):
        _append(cache, 0, k)
    assert B.amskv_kept_segments(cache, 0, 9) == [0, 1, 8, 9]
    B.amskv_cache_reset(cache)
    for k in range(10):
        _append(cache, 0, k)
    assert B.amskv_kept_segments(cache, 0, 9) == [0, 1, 8]
    B.amskv_cache_destroy(cache)
    # a promoted budget below the budget is a bad descriptor
    d, keep = B.make_desc(1, 2, 64, 2, (1, 2), [(2, 2, False)], flags=B.FLAG_PLAN_ONLY, token_budgets=[(10, 2, 5)])
    with pytest.raises(B.AmskvError) as e:
        B.amskv_cache_create(d)
    assert e.value.code == B.ERR_INVALID


def test_token_budget_promotion_bruteforce_against_algorithm_1():
    """Every small schedule and budget pair: promoting at the first overflow equals Algorithm 1 with the test
    passing there, token by token, and the copies of every append stay inside the region and never overlap."""
    schedules = [(1, 2, 3, 4), (2, 1, 3, 1, 2), (1, 2, 2, 3, 3), (3, 2, 4, 1, 3)]
    for sides in schedules:
        total = sum(s * s for s in sides)
        combos = [(lo, cds, hi) for lo in (1, 4, 5, 9, 14) for hi in (lo + 1, lo + 9, total)
                  for cds in (0, 1, 5) if cds <= lo]
        pols = [(2, 2, False)] * len(combos)
        for promote in (True, False):
            cache, d, keep = _plan(sides, pols, budgets=combos)
            need_tokens = (B.amskv_cache_required_bytes(d) - 256) // (2 * 2 * 2 * 2 * 64)
            for layer, (lo, cds, hi) in enumerate(combos):
                first = B.amskv_first_overflow_scale(cache, layer)
                outcomes = [promote] * len(sides)
                trace, budgets = oracle.algorithm1_trace(sides, lo, hi, cds, outcomes)
                # the oracle's budget changes exactly at the library's first overflow (if there is one)
                changed = [k for k in range(len(sides)) if budgets[k] != lo]
                assert (changed[0] if changed else None) == (first if promote and first < len(sides) else None)
                owner = {}
                for k in range(len(sides)):
                    if promote and k == first:
                        B.amskv_promote_layer(cache, layer)
                    written = set()
                    for src, dst, n in B.amskv_append_copies(cache, layer, k):
                        span = set(range(dst, dst + n))
                        assert not (span & written) and dst >= 0
                        written |= span
                        for j in range(n):
                            owner[dst + j] = (k, src + j)
                    _append(cache, layer, k)
                    want = oracle.attended_tokens(sides, k, lo, cds, c_max=hi, below_theta=outcomes)
                    read = [owner[p] for a, n in B.amskv_resident_ranges(cache, layer, k) for p in range(a, a + n)]
                    assert sorted(read) == sorted(want), (sides, lo, cds, hi, promote, k)
                    assert sorted(_expand(B.amskv_attended_tokens(cache, layer, k))) == sorted(want)
                assert max(owner) < need_tokens
            B.amskv_cache_destroy(cache)


def test_scale_granular_promotable_layer():
    """A promotable whole-scale layer: cache-efficient sets until promoted, every scale afterwards; the segments
    sit back to back either way, so no slot is reused and nothing moves."""
    for sides, c, w in [((1, 2, 3, 4, 5, 6, 8), 2, 2), ((1, 2, 3, 4, 5, 6), 1, 1), ((2, 3, 4, 5, 6), 0, 3)]:
        for promote in (True, False):
            cache, d, keep = _plan(sides, [(c, w, B.LAYER_PROMOTABLE), (c, w, True)])
            first = B.amskv_first_overflow_scale(cache, 0)
            assert first == c + w and B.amskv_first_overflow_scale(cache, 1) == len(sides)
            for k in range(len(sides)):
                if promote and k == first:
                    B.amskv_promote_layer(cache, 0)
                if k > first:
                    assert B.lib.amskv_promote_layer(cache, 0) in ((B.OK,) if promote else (B.ERR_ORDER,))
                # same place as in the cache-demanding layer beside it
                assert B.amskv_append_copies(cache, 0, k) == B.amskv_append_copies(cache, 1, k)
                _append(cache, 0, k)
                _append(cache, 1, k)
                dem = promote and k >= first
                assert B.amskv_kept_segments(cache, 0, k) == oracle.keep_set(k, c, w, dem)
                assert B.amskv_evicted_at(cache, 0, k) == oracle.evicted_at(k, c, w, promote)
            assert B.amskv_cache_required_bytes(d) == 256 + 2 * sum(s * s for s in sides) * 2 * 2 * 2 * 2 * 64
            B.amskv_cache_destroy(cache)
    # a promotable layer whose window already covers the schedule has nothing to be promoted to
    cache, d, keep = _plan((1, 2, 3), [(2, 2, B.LAYER_PROMOTABLE)])
    assert B.lib.amskv_promote_layer(cache, 0) == B.ERR_UNSUPPORTED
    B.amskv_cache_destroy(cache)
    d, keep = B.make_desc(1, 2, 64, 2, (1, 2), [(2, 2, 3)], flags=B.FLAG_PLAN_ONLY)
    with pytest.raises(B.AmskvError):
        B.amskv_cache_create(d)
