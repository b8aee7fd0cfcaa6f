"""A cache that never stores its last scale (no later scale reads it): host-side plan.  No GPU needed."""
import itertools

import pytest

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

FLAGS = B.FLAG_PLAN_ONLY | B.FLAG_TRANSIENT_LAST_SCALE


def _plan(sides, policies, budgets=None, heads=2, rows=2):
    d, keep = B.make_desc(len(policies), heads, 64, rows, sides, policies, flags=FLAGS, token_budgets=budgets)
    return B.amskv_cache_create(d), d, keep


def _expand(runs):
    return [(s, t) for s, first, count in runs for t in range(first, first + count)]


def test_arena_has_no_room_for_the_last_scale():
    sides = synth.SIDES_256
    per_token = 2 * 2 * 2 * 2 * 64
    # whole scales: 2 condensed + 2 local keeps 5 + 169 + 100 tokens of homes, full retention 680 - 256
    cache, d, keep = _plan(sides, [(2, 2, False), (2, 2, True)])
    assert B.amskv_cache_required_bytes(d) == 256 + (274 + 424) * per_token
    B.amskv_cache_destroy(cache)
    # token budgets of the paper's setting: neither layer class needs the 256-token transient slot any more
    cache, d, keep = _plan(sides, [(2, 2, False)] * 2, budgets=[(174, 5), (430, 5)])
    assert B.amskv_cache_required_bytes(d) == 256 + (174 + 424) * per_token
    B.amskv_cache_destroy(cache)


def test_what_is_attended_does_not_change():
    for sides in [(1, 2, 3, 4, 5), (3, 1, 4, 1, 5), (2,), synth.SIDES_256]:
        K = len(sides)
        pols = [(c, w, dem) for c, w, dem in itertools.product((0, 1, 2), (1, 2, 3), (False, True))]
        cache, d, keep = _plan(sides, pols)
        for layer, (c, w, dem) in enumerate(pols):
            for k in range(K):
                want = [(s, t) for s in oracle.keep_set(k, c, w, dem) for t in range(sides[s] ** 2)]
                assert _expand(B.amskv_attended_tokens(cache, layer, k)) == want
                kept = oracle.keep_set(k, c, w, dem)
                if k == K - 1:
                    kept = [s for s in kept if s != k]      # attended, but never held
                    assert k in B.amskv_evicted_at(cache, layer, k)
                assert B.amskv_kept_segments(cache, layer, k) == kept
        B.amskv_cache_destroy(cache)
    sides = (1, 2, 3, 4, 5, 6)
    budgets = [(b, c) for b in (3, 10, 20, 40, 100) for c in (0, 3, 5) if c <= b]
    cache, d, keep = _plan(sides, [(2, 2, False)] * len(budgets), budgets=budgets)
    for layer, (b, c) in enumerate(budgets):
        for k in range(len(sides)):
            assert sorted(_expand(B.amskv_attended_tokens(cache, layer, k))) == sorted(oracle.attended_tokens(sides, k, b, c))
    B.amskv_cache_destroy(cache)


def test_last_scale_reads_only_older_positions_and_is_never_copied():
    sides = synth.SIDES_256
    last = len(sides) - 1
    cache, d, keep = _plan(sides, [(2, 2, False), (2, 2, True)])
    for layer, n_older in ((0, 5 + 169), (1, 424)):
        assert B.amskv_append_copies(cache, layer, last) == []
        assert sum(n for _, n in B.amskv_resident_ranges(cache, layer, last)) == n_older
    B.amskv_cache_destroy(cache)


def test_order_contract_and_resident_bytes():
    sides = (1, 2, 3, 4)
    cache, d, keep = _plan(sides, [(1, 2, False)], heads=3, rows=4)
    per_token = 2 * 2 * 4 * 3 * 64
    for k in range(3):
        assert B.lib.amskv_append(cache, 0, k, None, None, None, None) == B.OK
    assert B.amskv_cache_bytes(cache)[1] == (1 + 4 + 9) * per_token
    # the last scale has no place in the arena: append refuses it, append_attend takes it
    assert B.lib.amskv_append(cache, 0, 3, None, None, None, None) == B.ERR_UNSUPPORTED
    assert B.lib.amskv_append_attend(cache, 0, 3, None, None, None, None, None, None, None, None) == B.OK
    assert B.lib.amskv_append_attend(cache, 0, 3, None, None, None, None, None, None, None, None) == B.ERR_ORDER
    # its step rolled the window (scale 1 left it) and stored nothing
    assert B.amskv_cache_bytes(cache)[1] == (1 + 9) * per_token
    B.amskv_cache_destroy(cache)
