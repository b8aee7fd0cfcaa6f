"""Token budgets (Algorithm 1 with Algorithm 2 as its roll, capacities in tokens): the library's
host-side plan against the oracle's literal list simulation.  No GPU needed (plan-only caches)."""
import itertools
import os

import pytest

import oracle
from paper_2511_16047_b200 import binding as B
from paper_2511_16047_b200 import synth

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "paper_680_schedule.txt")


def _golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            key, val = line.split("=")
            out[key.strip()] = [int(x) for x in val.split()]
    return out


def _plan(sides, budgets, policies=None, heads=2, rows=2):
    policies = policies or [(2, 2, False)] * len(budgets)
    d, keep = B.make_desc(len(budgets), heads, 64, rows, sides, policies, flags=B.FLAG_PLAN_ONLY,
                          token_budgets=budgets)
    return B.amskv_cache_create(d), d, keep


def _expand(runs):
    return [(s, t) for s, first, count in runs for t in range(first, first + count)]


def _check_layer(cache, layer, sides, c_bgt, c_cds, capacity):
    """Replays the library's copies on a model of the per-item region and compares what attend
    would read, position by position, with the oracle's token list."""
    owner = {}
    tokens = [s * s for s in sides]
    prev_cached = set()
    for k in range(len(sides)):
        copies = B.amskv_append_copies(cache, layer, k)
        written = set()
        for src, dst, n in copies:
            assert 0 <= src and src + n <= tokens[k] and n > 0
            assert 0 <= dst and dst + n <= capacity
            span = set(range(dst, dst + n))
            assert not (span & written), "two copies of one append overlap"
            written |= span
            for j in range(n):
                owner[dst + j] = (k, src + j)
        want = oracle.attended_tokens(sides, k, c_bgt, c_cds)
        assert len(set(want)) == len(want)
        ranges = B.amskv_resident_ranges(cache, layer, k)
        for (a, n), (b, _) in zip(ranges, ranges[1:]):
            assert a + n < b, "ranges must be sorted, disjoint and merged"
        read = [owner[p] for a, n in ranges for p in range(a, a + n)]
        assert len(read) == len(want) and set(read) == set(want), (sides, c_bgt, c_cds, k)
        runs = B.amskv_attended_tokens(cache, layer, k)
        assert sorted(_expand(runs)) == sorted(want)
        assert [r[0] for r in runs] == sorted(r[0] for r in runs)
        # what stays cached (the transient copy of a scale that is not resident in full does not count)
        hist = oracle.algorithm1_tokens(list(sides[:k + 1]), c_bgt, c_bgt, c_cds, below_theta=False)[k]
        cached = {s for s, _ in hist}
        assert B.amskv_kept_segments(cache, layer, k) == sorted(cached)
        assert B.amskv_evicted_at(cache, layer, k) == sorted((prev_cached | {k}) - cached)
        prev_cached = cached
        B.lib.amskv_append(cache, layer, k, None, None, None, None)


def test_plan_matches_algorithm_1_and_2_bruteforce():
    schedules = [(1, 2, 3), (1, 2, 3, 4, 5), (2, 1, 3, 1, 2), (1, 1, 1, 1, 1, 1), (3, 2, 4, 1, 3), (1, 2, 2, 3, 3, 4)]
    for sides in schedules:
        total = sum(s * s for s in sides)
        combos = [(b, c) for b in list(range(1, 14)) + [total - 1, total, total + 5]
                  for c in (0, 1, 2, 3, 5, 8, b) if 0 < b and c <= b]
        combos = sorted(set(combos))
        cache, d, keep = _plan(sides, combos)
        for layer, (b, c) in enumerate(combos):
            # the region never exceeds the budget plus a transient slot for the largest scale
            _check_layer(cache, layer, sides, b, c, b + max(s * s for s in sides))
        B.amskv_cache_destroy(cache)


def test_resident_bytes_follow_the_budget():
    sides = synth.SIDES_256
    budgets = [(174, 5), (430, 5), (50, 0)]
    cache, d, keep = _plan(sides, budgets, heads=3, rows=4)
    per_token = 2 * 2 * 4 * 3 * 64
    for k in range(len(sides)):
        for layer in range(3):
            B.lib.amskv_append(cache, layer, k, None, None, None, None)
        expect = sum(len(oracle.algorithm1_tokens(list(sides[:k + 1]), b, b, c, False)[k]) for b, c in budgets)
        assert B.amskv_cache_bytes(cache)[1] == expect * per_token
    B.amskv_cache_destroy(cache)


def test_paper_setting_on_the_680_token_schedule():
    g = _golden()
    sides = g["sides"]
    c_max, c_min, c_cds = g["c_max_tokens"][0], g["c_min_tokens"][0], g["c_cds_tokens"][0]
    cache, d, keep = _plan(sides, [(c_min, c_cds), (c_max, c_cds)])
    last = len(sides) - 1
    # cache-efficient layer: ends with the condensed scales and the penultimate scale cached; the last
    # scale is larger than C_min, is never cached and is attended from the transient slot
    assert B.amskv_kept_segments(cache, 0, last) == g["c_min_end_scales"]
    runs = B.amskv_attended_tokens(cache, 0, last)
    assert runs == [(0, 0, 1), (1, 0, 4), (8, 0, 169), (9, 0, 256)]
    assert B.amskv_resident_ranges(cache, 0, last) == [(0, c_min + 256)]
    # at scale 7 the tail cuts through scale 5: five of its tokens survive
    assert B.amskv_attended_tokens(cache, 0, 7) == [(0, 0, 1), (1, 0, 4), (5, 31, 5), (6, 0, 64), (7, 0, 100)]
    # cache-demanding layer: condensed scales plus the last two scales, whole
    assert B.amskv_kept_segments(cache, 1, last) == g["c_max_end_scales"]
    assert B.amskv_attended_tokens(cache, 1, last) == [(0, 0, 1), (1, 0, 4), (8, 0, 169), (9, 0, 256)]
    assert B.amskv_resident_ranges(cache, 1, last) == [(0, c_max)]
    # arena: C_min + the transient slot of the last scale, and C_max
    per_token = 2 * 2 * 2 * 2 * 64
    need = B.amskv_cache_required_bytes(d)
    assert need == 256 + (c_min + 256) * per_token + c_max * per_token
    B.amskv_cache_destroy(cache)


def test_promotion_at_first_overflow_equals_starting_at_c_max():
    # why a static per-layer budget is enough: nothing is evicted before the first overflow
    for sides in [(1, 2, 3, 4, 5), (2, 1, 3, 1, 2), (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)]:
        total = sum(s * s for s in sides)
        for c_min, extra, c_cds in itertools.product((1, 5, 14, 30, 174), (0, 3, 26, 256), (0, 1, 5)):
            c_max = c_min + extra
            if c_cds > c_min or c_min > total:
                continue
            a = oracle.algorithm1_tokens(sides, c_min, c_max, c_cds, below_theta=True)
            b = oracle.algorithm1_tokens(sides, c_max, c_max, c_cds, below_theta=False)
            assert a == b
            a = oracle.algorithm1_tokens(sides, c_min, c_max, c_cds, below_theta=False)
            b = oracle.algorithm1_tokens(sides, c_min, c_min, c_cds, below_theta=False)
            # without promotion a scale between C_min and C_max is skipped either way
            assert a == b


def test_token_and_scale_layers_mix_in_one_cache():
    sides = (1, 2, 3, 4, 5)
    d, keep = B.make_desc(3, 2, 64, 2, sides, [(1, 1, False), (2, 2, False), (0, 1, True)], flags=B.FLAG_PLAN_ONLY,
                          token_budgets=[(0, 0), (20, 5), (0, 0)])
    cache = B.amskv_cache_create(d)
    for k in range(len(sides)):
        assert B.amskv_kept_segments(cache, 0, k) == oracle.keep_set(k, 1, 1, False)
        assert B.amskv_kept_segments(cache, 2, k) == oracle.keep_set(k, 0, 1, True)
        assert B.amskv_append_copies(cache, 0, k)[0][0::2] == (0, sides[k] ** 2)
        assert sorted(_expand(B.amskv_attended_tokens(cache, 1, k))) == sorted(oracle.attended_tokens(sides, k, 20, 5))
    B.amskv_cache_destroy(cache)


def test_bad_budgets_are_refused():
    for bad in [(-1, 0), (5, -1)]:
        d, keep = B.make_desc(1, 2, 64, 2, (1, 2), [(2, 2, False)], flags=B.FLAG_PLAN_ONLY, token_budgets=[bad])
        with pytest.raises(B.AmskvError) as e:
            B.amskv_cache_create(d)
        assert e.value.code == B.ERR_INVALID
