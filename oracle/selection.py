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
        cache = cache + [i]  # the new scale joins the cache first (Algorithm 1)
        if cache_demanding:
            continue  # full retention: never rolled
        budget = n_condensed + n_local
        if len(cache) <= budget:
            continue  # a cache that fits its budget is left alone (Algorithm 2)
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
    """The eviction rule of Algorithm 2 (Appendix F) on an ordered list of (scale, token) entries.

    Budgets are token counts.  Stated by position: a cache of n entries that fits the budget is
    left alone; a longer one keeps position p exactly when p lies in the pinned head (p < c_cds)
    or among the newest c_bgt - c_cds positions (p >= n - (c_bgt - c_cds)).  Because
    n > c_bgt = c_cds + (c_bgt - c_cds), the two position sets cannot meet.
    """
    n = len(cache)
    if n <= c_bgt:
        return list(cache)
    newest = max(c_bgt - c_cds, 0)
    return [entry for p, entry in enumerate(cache) if p < c_cds or p >= n - newest]


def _outcome(below_theta, scale: int) -> bool:
    """Outcome of the similarity test S(k_i, resized k_{i-1}) < theta if it is evaluated at `scale`:
    one boolean for every scale, or a sequence indexed by scale."""
    if isinstance(below_theta, (bool, int)):
        return bool(below_theta)
    return bool(below_theta[scale])


def algorithm1_trace(sides: Sequence[int], c_min: int, c_max: int, c_cds: int, below_theta):
    """Algorithm 1 (Sec. 4.3) with budgets in tokens: (cache after every scale, budget after every scale).

    The layer starts cache-efficient with budget C_min.  For each scale, in order:
      1. a scale with more tokens than C_max is never cached: the cache is carried over;
      2. otherwise the scale's tokens join the end of the cache;
      3. if that exceeds the current budget: while the budget is still C_min the similarity test
         decides -- at THIS overflow, with this scale's keys, and again at every later overflow as
         long as the layer has not been promoted -- whether the budget becomes C_max; a scale with
         more tokens than the (possibly raised) budget is dropped again, leaving the cache as it
         was; otherwise the cache is rolled by `clru_tokens`.
    `below_theta` supplies the outcomes of the similarity test (the test itself needs key values):
    a single boolean, or a sequence indexed by scale so that a layer can fail the test at its
    first overflow and pass it at a later one, i.e. be promoted after evictions have happened.
    """
    cache: List[Tuple[int, int]] = []
    budget = c_min
    caches: List[List[Tuple[int, int]]] = []
    budgets: List[int] = []
    for i, side in enumerate(sides):
        own = [(i, t) for t in range(int(side) * int(side))]
        if len(own) <= c_max:
            joined = cache + own
            if len(joined) <= budget:
                cache = joined
            else:
                if budget == c_min and _outcome(below_theta, i):
                    budget = c_max
                if len(own) <= budget:
                    cache = clru_tokens(joined, budget, c_cds)
        caches.append(list(cache))
        budgets.append(budget)
    return caches, budgets


def algorithm1_tokens(sides: Sequence[int], c_min: int, c_max: int, c_cds: int,
                      below_theta) -> List[List[Tuple[int, int]]]:
    """The caches of `algorithm1_trace` (one per scale)."""
    return algorithm1_trace(sides, c_min, c_max, c_cds, below_theta)[0]


def attended_tokens(sides: Sequence[int], k: int, c_bgt: int, c_cds: int, c_max: int = None,
                    below_theta=False) -> List[Tuple[int, int]]:
    """(scale, token) pairs the queries of scale k attend to in a token-budget layer.

    The cache Algorithm 1 leaves after scale k, followed by the tokens of scale k that the cache
    does not hold (the reading taken for a scale that is skipped or cut by its own roll: it still
    sees itself).  With c_max left out the budget is fixed at c_bgt from the start; otherwise the
    layer starts at c_bgt (= C_min) and `below_theta` gives the promotion outcomes per scale.
    """
    top = c_bgt if c_max is None else c_max
    cache = algorithm1_tokens(list(sides[:k + 1]), c_bgt, top, c_cds, below_theta)[k]
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
