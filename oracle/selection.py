"""AMS-KV oracle, selection part: which KV segments a layer keeps (integers only).

TEST INFRASTRUCTURE ONLY: the product path never imports this module, and this module
imports nothing from the product.  Scales are 0-based here (the appendix's condensed-scale
ablation also writes CDS={0,1}); the main text counts from 1.

Reading of the paper taken here (the text is ambiguous on the first point):
  * the local window counts the just-appended scale: Algorithm 1 appends scale i before it
    rolls the cache and Algorithm 2 keeps the tail of that cache, so the newest entry of the
    tail is the current scale;
  * the scale-granular rule keeps whole scales: `n_condensed` leading scales are pinned and
    the `n_local` most recent scales form the FIFO tail;
  * a cache-demanding layer keeps every scale (full retention);
  * with token budgets (Algorithm 1 and 2 taken literally) the queries of a scale attend to the
    cache as it stands after that scale's step plus every token of the scale itself: the paper
    does not say what a scale that Algorithm 1 skips, or that its own roll cuts, attends to, and
    without its own keys it could not see itself.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def keep_set_simulated(k: int, n_condensed: int, n_local: int, cache_demanding: bool) -> List[int]:
    """Resident segment ids after scale k was appended, by literal list simulation.

    Algorithm 1 (append, then roll when over budget) with Algorithm 2 as the roll
    (pinned prefix plus FIFO tail), both at scale granularity: the budget is
    n_condensed + n_local entries, the prefix is the first n_condensed entries and the
    tail is the last n_local entries.
    """
    if n_local < 1:
        raise ValueError("n_local must be >= 1: a scale always attends to itself")
    if n_condensed < 0:
        raise ValueError("n_condensed must be >= 0")
    cache: List[int] = []
    for i in range(k + 1):
        cache = cache + [i]  # Algorithm 1: append the i-th scale
        if cache_demanding:
            continue  # full retention: never rolled
        budget = n_condensed + n_local
        if len(cache) <= budget:
            continue  # Algorithm 2: no rolling if within budget
        prefix = cache[:n_condensed]
        tail = cache[-n_local:]
        cache = prefix + [s for s in tail if s not in prefix]
    return cache


def keep_set(k: int, n_condensed: int, n_local: int, cache_demanding: bool) -> List[int]:
    """Same set by the closed-form predicate: s is kept iff s < c or s > k - w."""
    if n_local < 1 or n_condensed < 0:
        raise ValueError("need n_local >= 1 and n_condensed >= 0")
    if cache_demanding:
        return list(range(k + 1))
    return [s for s in range(k + 1) if s < n_condensed or s > k - n_local]


def evicted_at(k: int, n_condensed: int, n_local: int, cache_demanding: bool) -> List[int]:
    """Segments dropped by the append of scale k: (resident(k-1) + {k}) minus resident(k)."""
    before = keep_set(k - 1, n_condensed, n_local, cache_demanding) if k > 0 else []
    after = set(keep_set(k, n_condensed, n_local, cache_demanding))
    return [s for s in before + [k] if s not in after]


def kept_tokens(sides: Sequence[int], keep: Sequence[int]) -> int:
    """Number of key tokens in a kept set; a scale of side s has s*s tokens."""
    return sum(int(sides[s]) ** 2 for s in keep)


def clru_tokens(cache: List[Tuple[int, int]], c_bgt: int, c_cds: int) -> List[Tuple[int, int]]:
    """Algorithm 2 literally, on a list of tokens.

    `cache` is an ordered list of (scale, token) entries; c_bgt and c_cds are token counts.
    Within budget the cache is returned unchanged; otherwise the first c_cds entries and the
    last (c_bgt - c_cds) entries survive.
    """
    if len(cache) <= c_bgt:
        return cache
    head = cache[:c_cds]
    k = c_bgt - c_cds
    tail = cache[-k:] if k > 0 else []
    seen = set(head)
    return head + [e for e in tail if e not in seen]


def algorithm1_tokens(sides: Sequence[int], c_min: int, c_max: int, c_cds: int,
                      promote_at_overflow: bool) -> List[List[Tuple[int, int]]]:
    """Algorithm 1 literally with token budgets; returns the cache after every scale.

    `promote_at_overflow` stands for the outcome of the similarity test S < theta at the
    first overflow (the test itself needs key values; here only its outcome matters).
    A scale larger than c_max, or larger than the budget after the promotion decision, is
    not cached and the cache stays as it was.
    """
    cache: List[Tuple[int, int]] = []
    c_bgt = c_min
    history: List[List[Tuple[int, int]]] = []
    for i, side in enumerate(sides):
        seg = [(i, t) for t in range(side * side)]
        if len(seg) > c_max:
            history.append(list(cache))
            continue
        grown = cache + seg
        if len(grown) > c_bgt:
            if c_bgt == c_min and promote_at_overflow:
                c_bgt = c_max
            if len(seg) > c_bgt:
                history.append(list(cache))
                continue
            grown = clru_tokens(grown, c_bgt, c_cds)
        cache = grown
        history.append(list(cache))
    return history


def attended_tokens(sides: Sequence[int], k: int, c_bgt: int, c_cds: int) -> List[Tuple[int, int]]:
    """(scale, token) pairs the queries of scale k attend to in a layer whose budget is fixed at c_bgt.

    The cache Algorithm 1 leaves after scale k (budget c_bgt from the start: see
    `algorithm1_tokens`, whose promotion happens before anything was evicted), followed by the
    tokens of scale k that the cache does not hold.
    """
    cache = algorithm1_tokens(list(sides[:k + 1]), c_bgt, c_bgt, c_cds, promote_at_overflow=False)[k]
    have = set(cache)
    return cache + [(k, t) for t in range(int(sides[k]) ** 2) if (k, t) not in have]


def kv_bytes(sides: Sequence[int], policies: Sequence[Tuple[int, int, bool]], rows: int,
             heads: int, head_dim: int, bytes_per_value: int = 2) -> int:
    """KV bytes resident after the last append, summed over layers.

    The bracket of the memory-saving formula (Appendix D, Eq. 5) counts, per layer, the
    tokens of the scales that layer retains; here that count is turned into bytes as
    2 (K and V) * bytes_per_value * rows * heads * head_dim * tokens.
    `policies` holds (n_condensed, n_local, cache_demanding) per layer.
    """
    last = len(sides) - 1
    tokens = 0
    for (c, w, dem) in policies:
        tokens += kept_tokens(sides, keep_set(last, c, w, dem))
    return 2 * bytes_per_value * rows * heads * head_dim * tokens
