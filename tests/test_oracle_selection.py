"""Pins for the oracle's selection rule (integers only, no GPU)."""
import itertools
import os

import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_680_schedule.txt")


def _golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = [p.strip() for p in line.split("=")]
            out[k] = [int(x) for x in v.split()]
    return out


def test_predicate_equals_list_simulation_bruteforce():
    # every schedule length K <= 8, every c in 0..K, every w in 1..K, both layer classes
    for K in range(1, 9):
        for c, w, dem in itertools.product(range(0, K + 1), range(1, K + 1), (False, True)):
            for k in range(K):
                assert oracle.keep_set(k, c, w, dem) == oracle.keep_set_simulated(k, c, w, dem), (K, c, w, dem, k)


def test_within_budget_keeps_everything():
    # Algorithm 2: no rolling while the cache is within budget
    for c, w in itertools.product(range(0, 4), range(1, 4)):
        for k in range(c + w):
            assert oracle.keep_set(k, c, w, False) == list(range(k + 1))
        # the first eviction happens at k = c + w and removes segment c
        assert oracle.evicted_at(c + w, c, w, False) == [c]
        for k in range(c + w):
            assert oracle.evicted_at(k, c, w, False) == []


def test_demanding_is_full_retention_and_current_scale_always_kept():
    for k in range(12):
        assert oracle.keep_set(k, 2, 2, True) == list(range(k + 1))
        assert oracle.evicted_at(k, 2, 2, True) == []
        for c, w in itertools.product(range(0, 4), range(1, 4)):
            assert k in oracle.keep_set(k, c, w, False)


def test_evicted_segments_never_return():
    for c, w in itertools.product(range(0, 4), range(1, 5)):
        gone = set()
        for k in range(13):
            gone |= set(oracle.evicted_at(k, c, w, False))
            assert not (gone & set(oracle.keep_set(k, c, w, False)))
            assert sorted(gone | set(oracle.keep_set(k, c, w, False))) == list(range(k + 1))


def test_condensed_ablation_variants_are_legal():
    # CDS = {}, {0}, {0,1} (Appendix A)
    assert oracle.keep_set(9, 0, 2, False) == [8, 9]
    assert oracle.keep_set(9, 1, 2, False) == [0, 8, 9]
    assert oracle.keep_set(9, 2, 2, False) == [0, 1, 8, 9]
    with pytest.raises(ValueError):
        oracle.keep_set(3, 2, 0, False)


def test_paper_worked_example_token_counts():
    g = _golden()
    sides = g["sides"]
    assert sum(s * s for s in sides) == g["total_tokens"][0]
    assert oracle.kept_tokens(sides, [0, 1]) == g["c_cds_tokens"][0]
    # scale-granular rule, c=2 w=2, end state == the paper's C_max layer
    keep = oracle.keep_set(len(sides) - 1, 2, 2, False)
    assert keep == g["c_max_end_scales"]
    assert oracle.kept_tokens(sides, keep) == g["c_max_tokens"][0]
    assert oracle.kept_tokens(sides, g["c_min_end_scales"]) == g["c_min_tokens"][0]


def test_token_level_algorithms_reproduce_paper_end_states():
    g = _golden()
    sides = g["sides"]
    c_max, c_min, c_cds = g["c_max_tokens"][0], g["c_min_tokens"][0], g["c_cds_tokens"][0]
    # a promoted (cache-demanding) layer ends with scales {0,1,8,9}
    hist = oracle.algorithm1_tokens(sides, c_min, c_max, c_cds, below_theta=True)
    assert sorted({s for s, _ in hist[-1]}) == g["c_max_end_scales"]
    assert len(hist[-1]) == c_max
    # whole scales only in that end state
    for s in g["c_max_end_scales"]:
        assert sum(1 for e in hist[-1] if e[0] == s) == sides[s] ** 2
    # an unpromoted layer: the last scale is larger than C_min, so it is never cached
    hist = oracle.algorithm1_tokens(sides, c_min, c_max, c_cds, below_theta=False)
    assert sorted({s for s, _ in hist[-1]}) == g["c_min_end_scales"]
    assert len(hist[-1]) == c_min
    # budgets are respected after every scale, and the condensed prefix is always resident
    for h in hist:
        assert len(h) <= c_min
    for h in hist[1:]:
        assert h[:c_cds] == [(0, 0), (1, 0), (1, 1), (1, 2), (1, 3)]
    # while within budget nothing is rolled
    assert len(hist[6]) == sum(s * s for s in sides[:7])


def test_clru_literal_slicing():
    cache = [(0, i) for i in range(10)]
    assert oracle.clru_tokens(cache, 10, 2) == cache
    assert oracle.clru_tokens(cache, 5, 2) == cache[:2] + cache[-3:]
    assert oracle.clru_tokens(cache, 2, 2) == cache[:2]


def test_kv_bytes_closed_form():
    sides = (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)
    # d30 shape: 9 demanding (680 tokens) + 21 efficient (430 tokens), rows 512, 30 heads x 64
    pol = [(2, 2, True)] * 9 + [(2, 2, False)] * 21
    b = oracle.kv_bytes(sides, pol, 512, 30, 64)
    assert b == 2 * 2 * 512 * 30 * 64 * (9 * 680 + 21 * 430)
    full = oracle.kv_bytes(sides, [(2, 2, True)] * 30, 512, 30, 64)
    assert full == 2 * 2 * 512 * 30 * 64 * 30 * 680
    # Eq. 5's bracket: saving = total - retained, in tokens x layers
    saved_tokens = 680 * 30 - 680 * 9 - 430 * 21
    assert full - b == 2 * 2 * 512 * 30 * 64 * saved_tokens


ROLLS = os.path.join(os.path.dirname(__file__), "golden", "paper_680_token_rolls.txt")
SIDES_680 = (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)


def _rolls():
    out = {}
    with open(ROLLS) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                key, val = [p.strip() for p in line.split("=")]
                runs = [tuple(int(x) for x in r.split(":")) for r in val.split()]
                out[key] = [(s, t) for s, first, count in runs for t in range(first, first + count)]
    return out


def test_token_budget_caches_equal_hand_worked_lists():
    """Algorithm 1 + 2 with the paper's 5 / 174 / 430-token setting against states written out by hand."""
    g = _rolls()
    fixed_min = oracle.algorithm1_tokens(SIDES_680, 174, 174, 5, below_theta=False)
    for k in (6, 7, 8, 9):
        assert fixed_min[k] == g["cmin_cache_after_%d" % k], k
    fixed_max = oracle.algorithm1_tokens(SIDES_680, 430, 430, 5, below_theta=False)
    for k in (8, 9):
        assert fixed_max[k] == g["cmax_cache_after_%d" % k], k


def test_attended_tokens_equal_hand_worked_lists():
    """attended_tokens = the cache after the scale's own step plus the scale's tokens the cache lacks."""
    g = _rolls()
    for k in (6, 7, 8):     # the scale is resident in full: attended = cache
        assert oracle.attended_tokens(SIDES_680, k, 174, 5) == g["cmin_cache_after_%d" % k], k
    assert oracle.attended_tokens(SIDES_680, 9, 174, 5) == g["cmin_attended_at_9"]
    assert oracle.attended_tokens(SIDES_680, 9, 430, 5) == g["cmax_cache_after_9"]
    assert oracle.attended_tokens(SIDES_680, 8, 430, 5) == g["cmax_cache_after_8"]
    # a scale cut by its own roll: sides (1, 2, 3), budget 10, head 3 -> after scale 2 (9 tokens, 14 in all) the
    # cache is the first 3 entries + the newest 7 tokens of scale 2; its queries also see tokens 0 and 1 of scale 2
    assert oracle.attended_tokens((1, 2, 3), 2, 10, 3) == ([(0, 0), (1, 0), (1, 1)] + [(2, t) for t in range(2, 9)]
                                                          + [(2, 0), (2, 1)])
    # a scale larger than the budget is skipped: the cache is carried over and the scale sees itself
    assert oracle.attended_tokens((1, 2, 3), 2, 8, 1) == ([(0, 0)] + [(1, t) for t in range(4)]
                                                         + [(2, t) for t in range(9)])
    # with a promotion outcome list: the layer of `late8` at scales 8 and 9
    late = [False] * 8 + [True, True]
    assert oracle.attended_tokens(SIDES_680, 8, 174, 5, c_max=430, below_theta=late) == g["late8_cache_after_8"]
    assert oracle.attended_tokens(SIDES_680, 9, 174, 5, c_max=430, below_theta=late) == g["late8_cache_after_9"]


def test_similarity_test_is_taken_again_at_every_overflow_until_promotion():
    """Algorithm 1 evaluates the test whenever the budget is still C_min at an overflow, so a layer can be
    promoted after evictions; that is NOT the same as starting at C_max."""
    g = _rolls()
    caches, budgets = oracle.algorithm1_trace(SIDES_680, 174, 430, 5, [False] * 8 + [True, False])
    assert budgets == [174] * 8 + [430, 430]
    for k in (7, 8, 9):
        assert caches[k] == g["late8_cache_after_%d" % k], k
    assert caches[8] != oracle.algorithm1_tokens(SIDES_680, 430, 430, 5, False)[8]
    caches, budgets = oracle.algorithm1_trace(SIDES_680, 174, 430, 5, [False] * 9 + [True])
    assert budgets == [174] * 9 + [430]
    assert caches[8] == g["late9_cache_after_8"] and caches[9] == g["late9_cache_after_9"]
    # outcomes at scales that do not overflow are never looked at
    caches, budgets = oracle.algorithm1_trace(SIDES_680, 174, 430, 5, [True] * 7 + [False] * 3)
    assert budgets == [174] * 10
    # passing at the first overflow (scale 7) equals starting at C_max
    assert (oracle.algorithm1_tokens(SIDES_680, 174, 430, 5, [False] * 7 + [True] * 3)
            == oracle.algorithm1_tokens(SIDES_680, 430, 430, 5, False))
